// C-ABI entry points of libpf: argument validation, workspace layout, path selection
// (tensor-core kernels for bf16 inside their envelope, FMA kernels otherwise) and launches.
// Nothing here allocates or synchronises; see include/pf.h for the contract.
#include <atomic>
#include <cstring>

#include "pf_internal.h"
#include "pf_tc.h"

namespace pf {
namespace {

__device__ unsigned int g_device_status;  // 0 = fine; kernels store a PF_ERR_* code here

struct PerDevice {
    unsigned int* status_ptr;
    bool ready;
};
PerDevice g_dev[64];

bool elem_aligned(const void* p, int dtype) {
    return (reinterpret_cast<uintptr_t>(p) % dtype_size(dtype)) == 0;
}
bool valid_dtype(int dtype) { return dtype == PF_F32 || dtype == PF_BF16; }

int check_ws(const void* ws, size_t have, size_t need) {
    if (need == 0) return PF_OK;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || have < need)
        return PF_ERR_WORKSPACE;
    return PF_OK;
}

#define PF_CUDA(expr)                                   \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) return PF_ERR_CUDA;     \
    } while (0)

MatA plainA(const void* p, int64_t s_row, int64_t s_col) {
    MatA a;
    std::memset(&a, 0, sizeof(a));
    a.p = p; a.s_row = s_row; a.s_col = s_col; a.kind = A_PLAIN; a.l_fast = (s_col == 1);
    return a;
}
MatB plainB(const void* p, int64_t s_row, int64_t s_col) {
    MatB b;
    std::memset(&b, 0, sizeof(b));
    b.p = p; b.s_row = s_row; b.s_col = s_col; b.kind = B_PLAIN; b.l_fast = (s_col != 1);
    return b;
}
SimtGemm mk(const MatA& A, const MatB& B, void* C, int64_t ldc, int64_t M, int64_t N, int64_t K,
            int dtype, int splits = 1, float* partial = nullptr) {
    SimtGemm g;
    g.A = A; g.B = B; g.C = C; g.ldc = ldc; g.M = M; g.N = N; g.K = K;
    g.splits = splits; g.partial = partial; g.dtype = dtype;
    return g;
}

// ------------------------------------------------------------------------------ linear
struct LinearWs {
    size_t off_T, off_G, off_partial, off_gtmp, off_tc, total;
    int splits_dU, splits_dV;
};

LinearWs linear_ws(int64_t m, int64_t k, int64_t n, int64_t r, int dtype, bool bwd) {
    LinearWs w;
    std::memset(&w, 0, sizeof(w));
    const size_t s = dtype_size(dtype);
    size_t off = 0;
    w.off_T = off; off += align_up(static_cast<size_t>(m) * r * s, 256);
    if (bwd) {
        w.off_G = off; off += align_up(static_cast<size_t>(m) * r * s, 256);
        w.splits_dU = simt_pick_splits(k, r, m);
        w.splits_dV = simt_pick_splits(n, r, m);
        size_t pu = w.splits_dU > 1 ? static_cast<size_t>(w.splits_dU) * k * r * 4 : 0;
        size_t pv = w.splits_dV > 1 ? static_cast<size_t>(w.splits_dV) * n * r * 4 : 0;
        w.off_partial = off; off += align_up(pu > pv ? pu : pv, 256);
        // plain dU and dV of a call that wants them in fp32 or accumulated, on the paths that cannot
        // write them that way directly
        w.off_gtmp = off; off += align_up(static_cast<size_t>(k) * r * s, 256) + align_up(static_cast<size_t>(n) * r * s, 256);
    }
    w.off_tc = off;
    if (dtype == PF_BF16) off += align_up(tc::linear_extra_workspace(m, k, n, r, bwd), 256);
    w.total = off;
    return w;
}

int validate_linear_common(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                           int64_t ldv, int64_t m, int64_t k, int64_t n, int64_t r, int dtype) {
    if (!valid_dtype(dtype)) return PF_ERR_INVALID_ARG;
    if (m < 0 || k < 1 || n < 1 || r < 1) return PF_ERR_INVALID_ARG;
    if ((!x && m > 0) || !U || !V) return PF_ERR_INVALID_ARG;   // an empty batch may be a null pointer
    if (ldx < k || ldu < r || ldv < r) return PF_ERR_INVALID_ARG;
    if (!elem_aligned(x, dtype) || !elem_aligned(U, dtype) || !elem_aligned(V, dtype))
        return PF_ERR_INVALID_ARG;
    if (m > (1LL << 40) || k > (1LL << 31) || n > (1LL << 31) || r > (1LL << 20)) return PF_ERR_UNSUPPORTED;
    return PF_OK;
}

}  // namespace

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

unsigned int* device_status_ptr() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!g_dev[dev].ready) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        g_dev[dev].status_ptr = static_cast<unsigned int*>(p);
        g_dev[dev].ready = true;
    }
    return g_dev[dev].status_ptr;
}

}  // namespace pf

using namespace pf;

extern "C" {

const char* pf_status_string(int status) {
    switch (status) {
        case PF_OK: return "PF_OK";
        case PF_ERR_INVALID_ARG: return "PF_ERR_INVALID_ARG";
        case PF_ERR_UNSUPPORTED: return "PF_ERR_UNSUPPORTED";
        case PF_ERR_WORKSPACE: return "PF_ERR_WORKSPACE";
        case PF_ERR_CUDA: return "PF_ERR_CUDA";
        case PF_ERR_TIMEOUT: return "PF_ERR_TIMEOUT";
        default: return "PF_ERR_UNKNOWN";
    }
}

int pf_version(void) { return 100; }

long long pf_launch_count(void) { return launches_so_far(); }

int pf_last_device_status(void) {
    unsigned int* p = device_status_ptr();
    if (!p) return PF_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return PF_ERR_CUDA;
    unsigned int v = 0;
    if (cudaMemcpy(&v, p, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return PF_ERR_CUDA;
    if (v != 0) {
        const unsigned int zero = 0;
        if (cudaMemcpy(p, &zero, sizeof(zero), cudaMemcpyHostToDevice) != cudaSuccess) return PF_ERR_CUDA;
        tc::reset_fix_counters();
    }
    return v == 0 ? PF_OK : PF_ERR_TIMEOUT;
}

size_t pf_lowrank_linear_workspace(int64_t m, int64_t k, int64_t n, int64_t r, int dtype, int is_bwd) {
    if (!valid_dtype(dtype) || m < 0 || k < 1 || n < 1 || r < 1) return 0;
    return linear_ws(m, k, n, r, dtype, is_bwd != 0).total;
}

}  // extern "C"

namespace pf {
// The forward behind both entry points.  `exact_need`: instead of the public query's bound (which
// reserves for every path the call could take), require only the bytes that the path chosen for
// these pointers will touch; the workspace layout is the same either way.
int linear_fwd_impl(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                    int64_t ldv, void* y, int64_t ldy, void* T_stash, int64_t ldt,
                    int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                    void* workspace, size_t workspace_bytes, void* cuda_stream, bool exact_need, const void* bias,
                    int act) {
    int st = validate_linear_common(x, ldx, U, ldu, V, ldv, m, k, n, r, dtype);
    if (st != PF_OK) return st;
    if ((act != PF_ACT_NONE && act != PF_ACT_RELU) || (bias && !elem_aligned(bias, dtype))) return PF_ERR_INVALID_ARG;
    if ((!y && m > 0) || ldy < n || !elem_aligned(y, dtype)) return PF_ERR_INVALID_ARG;
    if (T_stash && (ldt < r || !elem_aligned(T_stash, dtype))) return PF_ERR_INVALID_ARG;
    const LinearWs w = linear_ws(m, k, n, r, dtype, false);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    tc::LinearArgs a;
    a.x = x; a.ldx = ldx; a.U = U; a.ldu = ldu; a.V = V; a.ldv = ldv;
    a.y = y; a.ldy = ldy; a.T = T_stash; a.ldt = ldt;
    a.m = m; a.k = k; a.n = n; a.r = r;
    a.ws = ws + w.off_tc; a.ws_T = ws + w.off_T; a.stream = stream;
    a.bias = bias; a.act = act;
    size_t need = w.total;
    if (exact_need) {
        bool tc_handles = false;
        const size_t tc_need = dtype == PF_BF16 ? tc::linear_fwd_need(a, &tc_handles) : 0;
        if (tc_handles) need = tc_need ? w.off_tc + tc_need : 0;
        else need = T_stash ? 0 : w.off_T + static_cast<size_t>(m) * r * dtype_size(dtype);   // FMA kernels: x U only
    }
    st = check_ws(workspace, workspace_bytes, need);
    if (st != PF_OK) return st;
    if (m == 0) return PF_OK;

    if (dtype == PF_BF16) {
        int handled = 0;
        st = tc::linear_fwd(a, &handled);
        if (st != PF_OK || handled) return st;
    }
    void* T = T_stash ? T_stash : static_cast<void*>(ws + w.off_T);
    const int64_t ldT = T_stash ? ldt : r;
    PF_CUDA(simt_gemm(mk(plainA(x, ldx, 1), plainB(U, ldu, 1), T, ldT, m, r, k, dtype), stream));
    PF_CUDA(simt_gemm(mk(plainA(T, ldT, 1), plainB(V, 1, ldv), y, ldy, m, n, r, dtype), stream));
    PF_CUDA(bias_act_inplace(y, ldy, m, n, bias, act, dtype, stream));
    return PF_OK;
}
}  // namespace pf

extern "C" {

int pf_lowrank_linear_fwd(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                          int64_t ldv, void* y, int64_t ldy, void* T_stash, int64_t ldt,
                          int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return linear_fwd_impl(x, ldx, U, ldu, V, ldv, y, ldy, T_stash, ldt, m, k, n, r, dtype, workspace, workspace_bytes,
                           cuda_stream, false);
}

int pf_lowrank_linear_fwd_act(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                              int64_t ldv, const void* bias, int act, void* y, int64_t ldy, void* T_stash, int64_t ldt,
                              int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return linear_fwd_impl(x, ldx, U, ldu, V, ldv, y, ldy, T_stash, ldt, m, k, n, r, dtype, workspace, workspace_bytes,
                           cuda_stream, false, bias, act);
}

size_t pf_bias_act_bwd_workspace(int64_t m, int64_t n) {
    if (m <= 0 || n <= 0) return 0;
    return align_up(static_cast<size_t>(act_bwd_chunks(m)) * n * 4, 256);
}

int pf_bias_act_bwd(const void* y, int64_t ldy, void* dY, int64_t lddy, void* dbias, int64_t m, int64_t n, int act,
                    int dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!valid_dtype(dtype) || m < 0 || n < 1) return PF_ERR_INVALID_ARG;
    if (act != PF_ACT_NONE && act != PF_ACT_RELU) return PF_ERR_INVALID_ARG;
    if ((m > 0 && !dY) || lddy < n || !elem_aligned(dY, dtype)) return PF_ERR_INVALID_ARG;
    if (act == PF_ACT_RELU && ((m > 0 && !y) || ldy < n || !elem_aligned(y, dtype))) return PF_ERR_INVALID_ARG;
    if (dbias && !elem_aligned(dbias, dtype)) return PF_ERR_INVALID_ARG;
    const size_t need = dbias ? pf_bias_act_bwd_workspace(m, n) : 0;
    int st = check_ws(workspace, workspace_bytes, need);
    if (st != PF_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (m == 0) {
        if (dbias) PF_CUDA(cudaMemsetAsync(dbias, 0, static_cast<size_t>(n) * dtype_size(dtype), stream));
        return PF_OK;
    }
    PF_CUDA(act_bwd(y, ldy, dY, lddy, dbias, m, n, act, dtype, static_cast<float*>(workspace), stream));
    return PF_OK;
}

int pf_lowrank_linear_bwd(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                          int64_t ldv, const void* dY, int64_t lddy, const void* T_stash, int64_t ldt,
                          void* dX, int64_t lddx, void* dU, int64_t lddu, void* dV, int64_t lddv,
                          int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return pf_lowrank_linear_bwd_ex(x, ldx, U, ldu, V, ldv, dY, lddy, T_stash, ldt, dX, lddx, dU, lddu, dV, lddv, m, k, n, r,
                                    dtype, 0u, workspace, workspace_bytes, cuda_stream);
}

int pf_lowrank_linear_bwd_ex(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V,
                             int64_t ldv, const void* dY, int64_t lddy, const void* T_stash, int64_t ldt,
                             void* dX, int64_t lddx, void* dU, int64_t lddu, void* dV, int64_t lddv,
                             int64_t m, int64_t k, int64_t n, int64_t r, int dtype, unsigned flags,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int st = validate_linear_common(x, ldx, U, ldu, V, ldv, m, k, n, r, dtype);
    if (st != PF_OK) return st;
    if (flags & ~static_cast<unsigned>(PF_GRAD_ACCUMULATE | PF_GRAD_F32)) return PF_ERR_INVALID_ARG;
    const bool g_acc = (flags & PF_GRAD_ACCUMULATE) != 0, g_f32 = (flags & PF_GRAD_F32) != 0;
    const int gdtype = g_f32 ? PF_F32 : dtype;          // storage type of dU and dV
    if ((!dY && m > 0) || lddy < n || !elem_aligned(dY, dtype)) return PF_ERR_INVALID_ARG;
    if (!dU || lddu < r || !elem_aligned(dU, gdtype)) return PF_ERR_INVALID_ARG;
    if (!dV || lddv < r || !elem_aligned(dV, gdtype)) return PF_ERR_INVALID_ARG;
    if (dX && (lddx < k || !elem_aligned(dX, dtype))) return PF_ERR_INVALID_ARG;
    if (T_stash && (ldt < r || !elem_aligned(T_stash, dtype))) return PF_ERR_INVALID_ARG;
    const LinearWs w = linear_ws(m, k, n, r, dtype, true);
    st = check_ws(workspace, workspace_bytes, w.total);
    if (st != PF_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t s = dtype_size(dtype);
    if (m == 0) {  // empty sums: zero, or nothing to add
        if (g_acc) return PF_OK;
        const size_t gs = dtype_size(gdtype);
        PF_CUDA(cudaMemset2DAsync(dU, lddu * gs, 0, r * gs, k, stream));
        PF_CUDA(cudaMemset2DAsync(dV, lddv * gs, 0, r * gs, n, stream));
        return PF_OK;
    }
    char* ws = static_cast<char*>(workspace);
    // A call with gradient flags that no kernel can honour directly computes plain dU and dV into the
    // workspace and adds / widens them into the caller's matrices in a pass of its own.
    void* const user_dU = dU;
    void* const user_dV = dV;
    const int64_t user_lddu = lddu, user_lddv = lddv;
    bool indirect = false;

    if (dtype == PF_BF16) {
        tc::LinearArgs a;
        a.x = x; a.ldx = ldx; a.U = U; a.ldu = ldu; a.V = V; a.ldv = ldv;
        a.dY = dY; a.lddy = lddy; a.T = const_cast<void*>(T_stash); a.ldt = ldt;
        a.dX = dX; a.lddx = lddx; a.dU = dU; a.lddu = lddu; a.dV = dV; a.lddv = lddv;
        a.m = m; a.k = k; a.n = n; a.r = r;
        a.ws = ws + w.off_tc; a.ws_T = ws + w.off_T; a.ws_G = ws + w.off_G; a.stream = stream;
        tc::LinearArgs::Slices su_info, sv_info;
        if (flags) {
            // plain gradients go to the workspace; where a reduction was split, its fp32 slices are still
            // there afterwards and are summed once more, unrounded, into the caller's matrix
            indirect = true;
            dU = ws + w.off_gtmp; lddu = r;
            dV = ws + w.off_gtmp + align_up(static_cast<size_t>(k) * r * s, 256); lddv = r;
            a.dU = dU; a.lddu = lddu; a.dV = dV; a.lddv = lddv;
            a.du_slices = &su_info; a.dv_slices = &sv_info;
        }
        int handled = 0;
        st = tc::linear_bwd(a, &handled);
        if (st != PF_OK) return st;
        if (handled && flags) {
            SliceSums jobs[2];
            int nj = 0;
            if (su_info.splits > 1)
                jobs[nj++] = SliceSums{su_info.partial, user_dU, user_lddu, static_cast<int>(k), static_cast<int>(r), su_info.splits,
                                       su_info.bn, su_info.tiles_x, su_info.tiles_y, g_f32, g_acc};
            else
                PF_CUDA(grad_combine(user_dU, user_lddu, gdtype, dU, lddu, dtype, k, r, g_acc, stream));
            if (sv_info.splits > 1)
                jobs[nj++] = SliceSums{sv_info.partial, user_dV, user_lddv, static_cast<int>(n), static_cast<int>(r), sv_info.splits,
                                       sv_info.bn, sv_info.tiles_x, sv_info.tiles_y, g_f32, g_acc};
            else
                PF_CUDA(grad_combine(user_dV, user_lddv, gdtype, dV, lddv, dtype, n, r, g_acc, stream));
            if (nj) PF_CUDA(slices_to_gradients(jobs, nj, stream));
            return PF_OK;
        }
        if (handled) return PF_OK;
    } else if (flags) {
        indirect = true;
        dU = ws + w.off_gtmp; lddu = r;
        dV = ws + w.off_gtmp + align_up(static_cast<size_t>(k) * r * s, 256); lddv = r;
    }
    const void* T = T_stash;
    int64_t ldT = ldt;
    if (!T) {
        void* Tw = ws + w.off_T;
        PF_CUDA(simt_gemm(mk(plainA(x, ldx, 1), plainB(U, ldu, 1), Tw, r, m, r, k, dtype), stream));
        T = Tw; ldT = r;
    }
    void* G = ws + w.off_G;
    float* partial = reinterpret_cast<float*>(ws + w.off_partial);
    PF_CUDA(simt_gemm(mk(plainA(dY, lddy, 1), plainB(V, ldv, 1), G, r, m, r, n, dtype), stream));
    if (dX) PF_CUDA(simt_gemm(mk(plainA(G, r, 1), plainB(U, 1, ldu), dX, lddx, m, k, r, dtype), stream));
    PF_CUDA(simt_gemm(mk(plainA(x, 1, ldx), plainB(G, r, 1), dU, lddu, k, r, m, dtype, w.splits_dU, partial), stream));
    PF_CUDA(simt_gemm(mk(plainA(dY, 1, lddy), plainB(T, ldT, 1), dV, lddv, n, r, m, dtype, w.splits_dV, partial), stream));
    if (indirect) {
        PF_CUDA(grad_combine(user_dU, user_lddu, gdtype, dU, lddu, dtype, k, r, g_acc, stream));
        PF_CUDA(grad_combine(user_dV, user_lddv, gdtype, dV, lddv, dtype, n, r, g_acc, stream));
    }
    return PF_OK;
}

// ------------------------------------------------------------------------------ grouped linear
namespace {
struct GroupedWs {
    size_t off_tc, off_acc, off_dx, off_single, total;
};
// Workspace of the grouped calls: the tensor-core path's buffers, then (for the path that runs group by
// group) an fp32 accumulator and one per-group dX for layers whose groups share x, then the workspace
// of one ungrouped call.
GroupedWs grouped_ws(int groups, int64_t m, int64_t k, int64_t n, int64_t r, int dtype, bool bwd) {
    GroupedWs w;
    size_t off = 0;
    w.off_tc = off;
    if (dtype == PF_BF16) off += align_up(tc::grouped_workspace(groups, m, k, n, r, bwd), 256);
    w.off_acc = off;
    if (bwd) off += align_up(static_cast<size_t>(m) * k * 4, 256);
    w.off_dx = off;
    if (bwd) off += align_up(static_cast<size_t>(m) * k * dtype_size(dtype), 256);
    w.off_single = off;
    off += linear_ws(m, k, n, r, dtype, bwd).total;
    w.total = off;
    return w;
}
const void* at_c(const void* p, int64_t stride, int g, int dtype) {
    return p ? static_cast<const char*>(p) + static_cast<size_t>(g) * stride * dtype_size(dtype) : nullptr;
}
void* at_m(void* p, int64_t stride, int g, int dtype) {
    return p ? static_cast<char*>(p) + static_cast<size_t>(g) * stride * dtype_size(dtype) : nullptr;
}
}  // namespace

size_t pf_lowrank_linear_grouped_workspace(int groups, int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                                           int is_bwd) {
    if (!valid_dtype(dtype) || groups < 1 || m < 0 || k < 1 || n < 1 || r < 1) return 0;
    return grouped_ws(groups, m, k, n, r, dtype, is_bwd != 0).total;
}

int pf_lowrank_linear_grouped_fwd(int groups, const void* x, int64_t ldx, int64_t sx, const void* U, int64_t ldu,
                                  int64_t su, const void* V, int64_t ldv, int64_t sv, void* y, int64_t ldy, int64_t sy,
                                  void* T_stash, int64_t ldt, int64_t st, int64_t m, int64_t k, int64_t n, int64_t r,
                                  int dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (groups < 1 || sx < 0 || su < 0 || sv < 0 || sy < 0 || st < 0) return PF_ERR_INVALID_ARG;
    int rc = validate_linear_common(x, ldx, U, ldu, V, ldv, m, k, n, r, dtype);
    if (rc != PF_OK) return rc;
    if ((!y && m > 0) || ldy < n || !elem_aligned(y, dtype)) return PF_ERR_INVALID_ARG;
    if (T_stash && (ldt < r || !elem_aligned(T_stash, dtype))) return PF_ERR_INVALID_ARG;
    // every group has its own factors and outputs; only x may be shared (sx == 0)
    if (groups > 1 && (su < k * ldu - (ldu - r) || sv < n * ldv - (ldv - r) || (m > 0 && sy < (m - 1) * ldy + n) ||
                       (T_stash && m > 0 && st < (m - 1) * ldt + r) || (sx != 0 && m > 0 && sx < (m - 1) * ldx + k)))
        return PF_ERR_INVALID_ARG;
    const GroupedWs w = grouped_ws(groups, m, k, n, r, dtype, false);
    rc = check_ws(workspace, workspace_bytes, w.total);
    if (rc != PF_OK) return rc;
    if (m == 0) return PF_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    if (dtype == PF_BF16) {
        tc::GroupedArgs a;
        a.groups = groups; a.x = x; a.ldx = ldx; a.sx = sx; a.U = U; a.ldu = ldu; a.su = su; a.V = V; a.ldv = ldv; a.sv = sv;
        a.y = y; a.ldy = ldy; a.sy = sy; a.T = T_stash; a.ldt = ldt; a.st = st;
        a.m = m; a.k = k; a.n = n; a.r = r; a.ws = ws + w.off_tc; a.stream = stream;
        int handled = 0;
        rc = tc::linear_grouped_fwd(a, &handled);
        if (rc != PF_OK || handled) return rc;
    }
    // group by group through the ungrouped entry (fp32, and bf16 operands TMA cannot describe)
    const size_t single = linear_ws(m, k, n, r, dtype, false).total;
    for (int g = 0; g < groups; ++g) {
        rc = linear_fwd_impl(at_c(x, sx, g, dtype), ldx, at_c(U, su, g, dtype), ldu, at_c(V, sv, g, dtype), ldv, at_m(y, sy, g, dtype),
                             ldy, at_m(T_stash, st, g, dtype), ldt, m, k, n, r, dtype, ws + w.off_single, single, cuda_stream,
                             false);
        if (rc != PF_OK) return rc;
    }
    return PF_OK;
}

int pf_lowrank_linear_grouped_bwd(int groups, const void* x, int64_t ldx, int64_t sx, const void* U, int64_t ldu,
                                  int64_t su, const void* V, int64_t ldv, int64_t sv, const void* dY, int64_t lddy,
                                  int64_t sdy, const void* T_stash, int64_t ldt, int64_t st, void* dX, int64_t lddx,
                                  int64_t sdx, void* dU, int64_t lddu, int64_t sdu, void* dV, int64_t lddv, int64_t sdv,
                                  int64_t m, int64_t k, int64_t n, int64_t r, int dtype, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
    if (groups < 1 || sx < 0 || su < 0 || sv < 0 || sdy < 0 || st < 0 || sdx < 0 || sdu < 0 || sdv < 0) return PF_ERR_INVALID_ARG;
    int rc = validate_linear_common(x, ldx, U, ldu, V, ldv, m, k, n, r, dtype);
    if (rc != PF_OK) return rc;
    if ((!dY && m > 0) || lddy < n || !elem_aligned(dY, dtype)) return PF_ERR_INVALID_ARG;
    if (!dU || lddu < r || !elem_aligned(dU, dtype) || !dV || lddv < r || !elem_aligned(dV, dtype)) return PF_ERR_INVALID_ARG;
    if (dX && (lddx < k || !elem_aligned(dX, dtype))) return PF_ERR_INVALID_ARG;
    if (T_stash && (ldt < r || !elem_aligned(T_stash, dtype))) return PF_ERR_INVALID_ARG;
    const bool shared_x = sx == 0 && groups > 1;
    if (groups > 1 && (su < k * ldu - (ldu - r) || sv < n * ldv - (ldv - r) || sdu < k * lddu - (lddu - r) ||
                       sdv < n * lddv - (lddv - r) || (m > 0 && sdy < (m - 1) * lddy + n) ||
                       (T_stash && m > 0 && st < (m - 1) * ldt + r) || (sx != 0 && m > 0 && sx < (m - 1) * ldx + k) ||
                       (dX && !shared_x && m > 0 && sdx < (m - 1) * lddx + k)))
        return PF_ERR_INVALID_ARG;
    const GroupedWs w = grouped_ws(groups, m, k, n, r, dtype, true);
    rc = check_ws(workspace, workspace_bytes, w.total);
    if (rc != PF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    if (dtype == PF_BF16 && m > 0) {
        tc::GroupedArgs a;
        a.groups = groups; a.x = x; a.ldx = ldx; a.sx = sx; a.U = U; a.ldu = ldu; a.su = su; a.V = V; a.ldv = ldv; a.sv = sv;
        a.dY = dY; a.lddy = lddy; a.sdy = sdy; a.T = const_cast<void*>(T_stash); a.ldt = ldt; a.st = st;
        a.dX = dX; a.lddx = lddx; a.sdx = sdx; a.dU = dU; a.lddu = lddu; a.sdu = sdu; a.dV = dV; a.lddv = lddv; a.sdv = sdv;
        a.m = m; a.k = k; a.n = n; a.r = r; a.ws = ws + w.off_tc; a.stream = stream;
        int handled = 0;
        rc = tc::linear_grouped_bwd(a, &handled);
        if (rc != PF_OK || handled) return rc;
    }
    // group by group; groups that share x add their input gradients in an fp32 accumulator
    const size_t single = linear_ws(m, k, n, r, dtype, true).total;
    float* acc = reinterpret_cast<float*>(ws + w.off_acc);
    void* dx_one = ws + w.off_dx;
    for (int g = 0; g < groups; ++g) {
        void* dx_g = !dX ? nullptr : shared_x ? dx_one : at_m(dX, sdx, g, dtype);
        rc = pf_lowrank_linear_bwd(at_c(x, sx, g, dtype), ldx, at_c(U, su, g, dtype), ldu, at_c(V, sv, g, dtype), ldv,
                                   at_c(dY, sdy, g, dtype), lddy, at_c(T_stash, st, g, dtype), ldt, dx_g, shared_x ? k : lddx,
                                   at_m(dU, sdu, g, dtype), lddu, at_m(dV, sdv, g, dtype), lddv, m, k, n, r, dtype,
                                   ws + w.off_single, single, cuda_stream);
        if (rc != PF_OK) return rc;
        if (dX && shared_x && m > 0) PF_CUDA(accumulate_f32(acc, dx_one, k, m, k, dtype, g == 0, stream));
    }
    if (dX && shared_x && m > 0) PF_CUDA(round_out_f32(acc, dX, lddx, m, k, dtype, stream));
    return PF_OK;
}

// ------------------------------------------------------------------------------ conv
namespace {
struct ConvWs {
    size_t off_T, off_dT, off_partial, off_gtmp, off_tc, total;
    int splits_dU, splits_dV;
    int Ho, Wo;
    int64_t P, Pin;
};
ConvWs conv_ws(int N, int H, int W, int C, int R, int O, int kh, int kw, int stride, int pad,
               int dtype, bool bwd) {
    ConvWs w;
    std::memset(&w, 0, sizeof(w));
    w.Ho = (H + 2 * pad - kh) / stride + 1;
    w.Wo = (W + 2 * pad - kw) / stride + 1;
    if (w.Ho < 0) w.Ho = 0;
    if (w.Wo < 0) w.Wo = 0;
    w.P = static_cast<int64_t>(N) * w.Ho * w.Wo;
    w.Pin = static_cast<int64_t>(N) * H * W;
    const size_t s = dtype_size(dtype);
    size_t off = 0;
    w.off_T = off; off += align_up(static_cast<size_t>(w.P) * R * s, 256);
    if (bwd) {
        w.off_dT = off; off += align_up(static_cast<size_t>(w.P) * R * s, 256);
        const int64_t Keff = static_cast<int64_t>(kh) * kw * C;
        w.splits_dU = simt_pick_splits(Keff, R, w.P);
        w.splits_dV = simt_pick_splits(O, R, w.P);
        size_t pu = w.splits_dU > 1 ? static_cast<size_t>(w.splits_dU) * Keff * R * 4 : 0;
        size_t pv = w.splits_dV > 1 ? static_cast<size_t>(w.splits_dV) * O * R * 4 : 0;
        w.off_partial = off; off += align_up(pu > pv ? pu : pv, 256);
        // plain dU and dV of a call that wants them in fp32 or accumulated
        w.off_gtmp = off; off += align_up(static_cast<size_t>(Keff) * R * s, 256) + align_up(static_cast<size_t>(O) * R * s, 256);
    }
    w.off_tc = off;
    if (dtype == PF_BF16) off += align_up(tc::conv_extra_workspace(N, H, W, C, R, O, kh, kw, stride, pad, bwd), 256);
    w.total = off;
    return w;
}
int validate_conv_common(const void* x, const void* U, const void* V, int N, int H, int W, int C,
                         int R, int O, int kh, int kw, int stride, int pad, int dtype) {
    if (!valid_dtype(dtype)) return PF_ERR_INVALID_ARG;
    if (N < 0 || H < 1 || W < 1 || C < 1 || R < 1 || O < 1 || kh < 1 || kw < 1 || pad < 0)
        return PF_ERR_INVALID_ARG;
    if (stride < 1 || kh != kw) return PF_ERR_UNSUPPORTED;
    if (H + 2 * pad < kh || W + 2 * pad < kw) return PF_ERR_INVALID_ARG;
    if ((!x && N > 0) || !U || !V) return PF_ERR_INVALID_ARG;   // an empty batch may be a null pointer
    if (!elem_aligned(x, dtype) || !elem_aligned(U, dtype) || !elem_aligned(V, dtype))
        return PF_ERR_INVALID_ARG;
    return PF_OK;
}
ConvGeom geom(int N, int H, int W, int C, int R, int kh, int kw, int stride, int pad, const ConvWs& w) {
    ConvGeom g;
    g.N = N; g.H = H; g.W = W; g.C = C; g.Ho = w.Ho; g.Wo = w.Wo; g.kh = kh; g.kw = kw;
    g.st = stride; g.pad = pad; g.R = R;
    return g;
}
}  // namespace

size_t pf_lowrank_conv_workspace(int N, int H, int W, int C, int R, int O, int kh, int kw,
                                 int stride, int pad, int dtype, int is_bwd) {
    if (!valid_dtype(dtype) || N < 0 || H < 1 || W < 1 || C < 1 || R < 1 || O < 1 || kh < 1 ||
        kw < 1 || pad < 0 || stride < 1 || H + 2 * pad < kh || W + 2 * pad < kw)
        return 0;
    return conv_ws(N, H, W, C, R, O, kh, kw, stride, pad, dtype, is_bwd != 0).total;
}

int pf_lowrank_conv_fwd(const void* x, const void* U, const void* V, void* y, void* T_stash,
                        int N, int H, int W, int C, int R, int O, int kh, int kw, int stride,
                        int pad, int dtype, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    int st = validate_conv_common(x, U, V, N, H, W, C, R, O, kh, kw, stride, pad, dtype);
    if (st != PF_OK) return st;
    if ((!y && N > 0) || !elem_aligned(y, dtype) || (T_stash && !elem_aligned(T_stash, dtype)))
        return PF_ERR_INVALID_ARG;
    const ConvWs w = conv_ws(N, H, W, C, R, O, kh, kw, stride, pad, dtype, false);
    st = check_ws(workspace, workspace_bytes, w.total);
    if (st != PF_OK) return st;
    if (w.P == 0) return PF_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);

    if (dtype == PF_BF16) {
        tc::ConvArgs a;
        std::memset(&a, 0, sizeof(a));
        a.x = x; a.U = U; a.V = V; a.y = y; a.T = T_stash;
        a.N = N; a.H = H; a.W = W; a.C = C; a.R = R; a.O = O; a.kh = kh; a.kw = kw;
        a.stride = stride; a.pad = pad; a.Ho = w.Ho; a.Wo = w.Wo;
        a.ws = ws + w.off_tc; a.ws_T = ws + w.off_T; a.stream = stream;
        int handled = 0;
        st = tc::conv_fwd(a, &handled);
        if (st != PF_OK || handled) return st;
    }
    void* T = T_stash ? T_stash : static_cast<void*>(ws + w.off_T);
    MatA A;
    std::memset(&A, 0, sizeof(A));
    A.p = x; A.kind = A_IM2COL; A.l_fast = 1; A.g = geom(N, H, W, C, R, kh, kw, stride, pad, w);
    const int64_t Keff = static_cast<int64_t>(kh) * kw * C;
    PF_CUDA(simt_gemm(mk(A, plainB(U, R, 1), T, R, w.P, R, Keff, dtype), stream));
    PF_CUDA(simt_gemm(mk(plainA(T, R, 1), plainB(V, 1, R), y, O, w.P, O, R, dtype), stream));
    return PF_OK;
}

int pf_lowrank_conv_bwd(const void* x, const void* U, const void* V, const void* dY,
                        const void* T_stash, void* dX, void* dU, void* dV,
                        int N, int H, int W, int C, int R, int O, int kh, int kw, int stride,
                        int pad, int dtype, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    return pf_lowrank_conv_bwd_ex(x, U, V, dY, T_stash, dX, dU, dV, N, H, W, C, R, O, kh, kw, stride, pad, dtype, 0u,
                                  workspace, workspace_bytes, cuda_stream);
}

int pf_lowrank_conv_bwd_ex(const void* x, const void* U, const void* V, const void* dY,
                           const void* T_stash, void* dX, void* dU, void* dV,
                           int N, int H, int W, int C, int R, int O, int kh, int kw, int stride,
                           int pad, int dtype, unsigned flags, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
    int st = validate_conv_common(x, U, V, N, H, W, C, R, O, kh, kw, stride, pad, dtype);
    if (st != PF_OK) return st;
    if (flags & ~static_cast<unsigned>(PF_GRAD_ACCUMULATE | PF_GRAD_F32)) return PF_ERR_INVALID_ARG;
    const bool g_acc = (flags & PF_GRAD_ACCUMULATE) != 0, g_f32 = (flags & PF_GRAD_F32) != 0;
    const int gdtype = g_f32 ? PF_F32 : dtype;
    if ((!dY && N > 0) || !dU || !dV) return PF_ERR_INVALID_ARG;
    if (!elem_aligned(dY, dtype) || !elem_aligned(dU, gdtype) || !elem_aligned(dV, gdtype) ||
        (dX && !elem_aligned(dX, dtype)) || (T_stash && !elem_aligned(T_stash, dtype)))
        return PF_ERR_INVALID_ARG;
    const ConvWs w = conv_ws(N, H, W, C, R, O, kh, kw, stride, pad, dtype, true);
    st = check_ws(workspace, workspace_bytes, w.total);
    if (st != PF_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t s = dtype_size(dtype);
    const int64_t Keff = static_cast<int64_t>(kh) * kw * C;
    if (w.P == 0) {
        if (!g_acc) {
            PF_CUDA(cudaMemsetAsync(dU, 0, Keff * R * dtype_size(gdtype), stream));
            PF_CUDA(cudaMemsetAsync(dV, 0, static_cast<size_t>(O) * R * dtype_size(gdtype), stream));
        }
        if (dX && w.Pin > 0) PF_CUDA(cudaMemsetAsync(dX, 0, w.Pin * C * s, stream));
        return PF_OK;
    }
    char* ws = static_cast<char*>(workspace);
    // with gradient flags: plain dU, dV into the workspace, then one pass into the caller's matrices
    void* const user_dU = dU;
    void* const user_dV = dV;
    if (flags) {
        dU = ws + w.off_gtmp;
        dV = ws + w.off_gtmp + align_up(static_cast<size_t>(Keff) * R * s, 256);
    }
    tc::LinearArgs::Slices su_info, sv_info;
    auto finish = [&]() -> int {
        if (!flags) return PF_OK;
        SliceSums jobs[2];
        int nj = 0;
        if (su_info.splits > 1)
            jobs[nj++] = SliceSums{su_info.partial, user_dU, R, static_cast<int>(Keff), R, su_info.splits, su_info.bn,
                                   su_info.tiles_x, su_info.tiles_y, g_f32, g_acc};
        else
            PF_CUDA(grad_combine(user_dU, R, gdtype, dU, R, dtype, Keff, R, g_acc, stream));
        if (sv_info.splits > 1)
            jobs[nj++] = SliceSums{sv_info.partial, user_dV, R, O, R, sv_info.splits, sv_info.bn, sv_info.tiles_x,
                                   sv_info.tiles_y, g_f32, g_acc};
        else
            PF_CUDA(grad_combine(user_dV, R, gdtype, dV, R, dtype, O, R, g_acc, stream));
        if (nj) PF_CUDA(slices_to_gradients(jobs, nj, stream));
        return PF_OK;
    };

    if (dtype == PF_BF16) {
        tc::ConvArgs a;
        std::memset(&a, 0, sizeof(a));
        a.x = x; a.U = U; a.V = V; a.dY = dY; a.T = const_cast<void*>(T_stash);
        a.dX = dX; a.dU = dU; a.dV = dV;
        a.N = N; a.H = H; a.W = W; a.C = C; a.R = R; a.O = O; a.kh = kh; a.kw = kw;
        a.stride = stride; a.pad = pad; a.Ho = w.Ho; a.Wo = w.Wo;
        a.ws = ws + w.off_tc; a.ws_T = ws + w.off_T; a.ws_G = ws + w.off_dT; a.stream = stream;
        a.du_slices = &su_info; a.dv_slices = &sv_info;
        int handled = 0;
        st = tc::conv_bwd(a, &handled);
        if (st != PF_OK) return st;
        if (handled) return finish();
        su_info = tc::LinearArgs::Slices();
        sv_info = tc::LinearArgs::Slices();
    }
    MatA Aim;
    std::memset(&Aim, 0, sizeof(Aim));
    Aim.p = x; Aim.kind = A_IM2COL; Aim.l_fast = 1; Aim.g = geom(N, H, W, C, R, kh, kw, stride, pad, w);
    const void* T = T_stash;
    if (!T) {
        void* Tw = ws + w.off_T;
        PF_CUDA(simt_gemm(mk(Aim, plainB(U, R, 1), Tw, R, w.P, R, Keff, dtype), stream));
        T = Tw;
    }
    void* dT = ws + w.off_dT;
    float* partial = reinterpret_cast<float*>(ws + w.off_partial);
    PF_CUDA(simt_gemm(mk(plainA(dY, O, 1), plainB(V, R, 1), dT, R, w.P, R, O, dtype), stream));
    PF_CUDA(simt_gemm(mk(plainA(dY, 1, O), plainB(T, R, 1), dV, R, O, R, w.P, dtype, w.splits_dV, partial), stream));
    MatA At = Aim;
    At.kind = A_IM2COL_T; At.l_fast = 0;
    PF_CUDA(simt_gemm(mk(At, plainB(dT, R, 1), dU, R, Keff, R, w.P, dtype, w.splits_dU, partial), stream));
    if (dX) {
        MatA Ac = Aim;
        Ac.p = dT; Ac.kind = A_COL2IM; Ac.l_fast = 1;
        MatB Bt;
        std::memset(&Bt, 0, sizeof(Bt));
        Bt.p = U; Bt.kind = B_TAPSPLIT; Bt.l_fast = 1; Bt.R = R; Bt.CR = C * R;
        PF_CUDA(simt_gemm(mk(Ac, Bt, dX, C, w.Pin, C, static_cast<int64_t>(kh) * kw * R, dtype), stream));
    }
    return finish();
}

// ------------------------------------------------------------------------------ pack
int pf_pack_factor_grads(const void* const* grads, const int64_t* numels, int count, int dtype,
                         void* flat, int64_t flat_capacity_elems, int64_t* offsets_out,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
    (void)workspace; (void)workspace_bytes;
    if (!valid_dtype(dtype) || count < 0 || !offsets_out || flat_capacity_elems < 0)
        return PF_ERR_INVALID_ARG;
    if (count > 0 && (!grads || !numels)) return PF_ERR_INVALID_ARG;
    offsets_out[0] = 0;
    for (int i = 0; i < count; ++i) {
        if (numels[i] < 0) return PF_ERR_INVALID_ARG;
        if (numels[i] > 0 && (!grads[i] || !elem_aligned(grads[i], dtype))) return PF_ERR_INVALID_ARG;
        if (numels[i] > (1LL << 46)) return PF_ERR_UNSUPPORTED;
        offsets_out[i + 1] = offsets_out[i] + numels[i];
    }
    const int64_t total = offsets_out[count];
    if (total > flat_capacity_elems) return PF_ERR_WORKSPACE;
    if (total == 0) return PF_OK;
    if (!flat || !elem_aligned(flat, dtype)) return PF_ERR_INVALID_ARG;
    PF_CUDA(pack_launch(grads, numels, offsets_out, count, static_cast<int>(dtype_size(dtype)), flat,
                        static_cast<cudaStream_t>(cuda_stream)));
    return PF_OK;
}

int pf_unpack_factor_grads(const void* flat, int64_t flat_elems, void* const* grads, const int64_t* numels, int count,
                           int dtype, int64_t* offsets_out, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
    (void)workspace; (void)workspace_bytes;
    if (!valid_dtype(dtype) || count < 0 || !offsets_out || flat_elems < 0) return PF_ERR_INVALID_ARG;
    if (count > 0 && (!grads || !numels)) return PF_ERR_INVALID_ARG;
    offsets_out[0] = 0;
    for (int i = 0; i < count; ++i) {
        if (numels[i] < 0) return PF_ERR_INVALID_ARG;
        if (numels[i] > 0 && (!grads[i] || !elem_aligned(grads[i], dtype))) return PF_ERR_INVALID_ARG;
        if (numels[i] > (1LL << 46)) return PF_ERR_UNSUPPORTED;
        offsets_out[i + 1] = offsets_out[i] + numels[i];
    }
    const int64_t total = offsets_out[count];
    if (total > flat_elems) return PF_ERR_WORKSPACE;
    if (total == 0) return PF_OK;
    if (!flat || !elem_aligned(flat, dtype)) return PF_ERR_INVALID_ARG;
    PF_CUDA(unpack_launch(flat, grads, numels, offsets_out, count, static_cast<int>(dtype_size(dtype)),
                          static_cast<cudaStream_t>(cuda_stream)));
    return PF_OK;
}

}  // extern "C"
