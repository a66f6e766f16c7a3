// Internal declarations shared by the translation units of libpf (not part of the ABI).
#ifndef PF_INTERNAL_H_
#define PF_INTERNAL_H_

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "pf.h"

namespace pf {

// Streaming multiprocessors of the current device (148 on B200), asked once per device: grids that
// must be resident at once (split reductions whose thread blocks meet at counters) and persistent
// schedules are sized by it.
inline int num_sms() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t dtype_size(int dtype) { return dtype == PF_BF16 ? 2 : 4; }

// ---------------------------------------------------------------------------------------
// Generic strided / implicit matrix views consumed by the FMA (SIMT) GEMM.  The FMA path
// serves fp32 storage and every bf16 shape outside the tensor-core envelope.
// ---------------------------------------------------------------------------------------
enum AKind : int {
    A_PLAIN = 0,     // A(i,l) = p[i*s_row + l*s_col]
    A_IM2COL = 1,    // i = output pixel (n,ho,wo), l = (a,b,c):  x[n, ho*st-pad+a, wo*st-pad+b, c] or 0
    A_IM2COL_T = 2,  // i = (a,b,c), l = output pixel: same value, roles swapped (for dU)
    A_COL2IM = 3     // i = input pixel (n,h,w), l = (a,b,j): dT[n,(h+pad-a)/st,(w+pad-b)/st,j] or 0
};
enum BKind : int {
    B_PLAIN = 0,    // B(l,j) = p[l*s_row + j*s_col]
    B_TAPSPLIT = 1  // l = (tap, q), q < R:  p[tap*C*R + j*R + q]   (U[tap][j][q] read as (tap,q) x j)
};

struct ConvGeom {
    int N, H, W, C, Ho, Wo, kh, kw, st, pad, R;
};

struct MatA {
    const void* p;
    int64_t s_row, s_col;
    int kind;
    int l_fast;  // 1 if consecutive l are contiguous in memory, else consecutive i are
    ConvGeom g;
};
struct MatB {
    const void* p;
    int64_t s_row, s_col;
    int kind;
    int l_fast;
    int R, CR;  // B_TAPSPLIT only
};

struct SimtGemm {
    MatA A;
    MatB B;
    void* C;          // [M, N] row-major, ldc, storage dtype
    int64_t ldc;
    int64_t M, N, K;
    int splits;       // > 1: fp32 partials go to `partial` [splits, M, N], then a fixed-order sum
    float* partial;
    int dtype;
};

cudaError_t simt_gemm(const SimtGemm& g, cudaStream_t stream);
int simt_pick_splits(int64_t M, int64_t N, int64_t K);
// C[M,N] (storage dtype, ldc) = sum over z < splits of partial[z][M][N], in increasing z.
cudaError_t splitk_reduce(const float* partial, void* C, int64_t ldc, int64_t M, int64_t N, int splits,
                          int dtype, cudaStream_t stream);

// Strided 2-D copy with zero fill (repack to a padded pitch), elements of 2 bytes.
cudaError_t repack_rows_bf16(const void* src, int64_t ld_src, void* dst, int64_t ld_dst,
                             int64_t rows, int64_t cols, int64_t cols_padded, cudaStream_t stream);

// acc (fp32, dense [rows, cols]) = (first ? 0 : acc) + src; dst = acc rounded once to the storage dtype.
cudaError_t accumulate_f32(float* acc, const void* src, int64_t ld_src, int64_t rows, int64_t cols, int dtype, bool first,
                           cudaStream_t stream);
cudaError_t round_out_f32(const float* acc, void* dst, int64_t ld_dst, int64_t rows, int64_t cols, int dtype,
                          cudaStream_t stream);
// out (fp32 or the storage dtype, pitch ld_out) = (accumulate ? out : 0) + src (storage dtype src_dtype).
cudaError_t grad_combine(void* out, int64_t ld_out, int out_dtype, const void* src, int64_t ld_src, int src_dtype,
                         int64_t rows, int64_t cols, bool accumulate, cudaStream_t stream);
// out = (accumulate ? out : 0) + the sum, in slice order, of the fp32 slices a split tensor-core reduction
// left at `partial` ([tile][slice][128][bn], see pf_simt.cu); one launch for up to two matrices.
struct SliceSums {
    const float* partial;
    void* out;          // fp32 (out_f32) or bf16 matrix, pitch ld in its own elements
    long long ld;
    int M, N, splits, bn, tiles_x, tiles_y;
    bool out_f32, accumulate;
};
cudaError_t slices_to_gradients(const SliceSums* jobs, int count, cudaStream_t stream);
// Backward of y = act(z + bias): dY becomes dZ in place, db (optional) its column sums.  `part` holds
// act_bwd_chunks(rows) * cols floats.
int act_bwd_chunks(int64_t rows);
cudaError_t act_bwd(const void* y, int64_t ldy, void* dY, int64_t lddy, void* db, int64_t rows, int64_t cols, int act,
                    int dtype, float* part, cudaStream_t stream);
// y = act(y + bias) in place: bias [cols] of the storage dtype or null, act 0 = identity, 1 = max(0, .)
cudaError_t bias_act_inplace(void* y, int64_t ld, int64_t rows, int64_t cols, const void* bias, int act, int dtype,
                             cudaStream_t stream);

// Several such copies in one launch (row counts and widths below 2^31).
struct RepackJob {
    const void* src;
    int64_t ld_src;
    void* dst;
    int64_t ld_dst;
    int64_t rows, cols, cols_padded;
};
cudaError_t repack_rows_bf16_multi(const RepackJob* jobs, int count, cudaStream_t stream);

// pack
cudaError_t pack_launch(const void* const* grads, const int64_t* numels, const int64_t* offsets,
                        int count, int elem_bytes, void* flat, cudaStream_t stream);
cudaError_t unpack_launch(const void* flat, void* const* grads, const int64_t* numels, const int64_t* offsets,
                          int count, int elem_bytes, cudaStream_t stream);

// The factorized linear forward behind pf_lowrank_linear_fwd and pf_lowrank_linear_fwd_static.
// exact_need = false: the workspace must satisfy the public query; true: only the bytes the path
// chosen for these pointers and pitches will touch.
int linear_fwd_impl(const void* x, int64_t ldx, const void* U, int64_t ldu, const void* V, int64_t ldv, void* y,
                    int64_t ldy, void* T_stash, int64_t ldt, int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                    void* workspace, size_t workspace_bytes, void* cuda_stream, bool exact_need,
                    const void* bias = nullptr, int act = 0);

// host-side count of kernels launched by this library
void count_launch(int n = 1);

// device status word (bounded waits report here)
cudaError_t read_and_clear_device_status(unsigned int* out);

}  // namespace pf
#endif
