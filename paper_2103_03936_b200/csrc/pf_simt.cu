// FMA (CUDA-core) GEMM with implicit-matrix views.
//
// Serves the fp32 storage path (single-pass TF32 cannot reach 1e-4 after two chained
// products) and every bf16 shape outside the tensor-core envelope.  One kernel, templated on
// how operand A is addressed: plain strided, im2col of an NHWC image (convolution forward
// and dU), or the gather form of the transposed convolution (dX).  Products accumulate in
// fp32; a reduction split over K writes fp32 partials that a second kernel sums in a fixed
// order, so results are bit-reproducible run to run.
#include "pf_internal.h"

namespace pf {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

template <typename T> __device__ __forceinline__ float ldf(const void* p, int64_t idx);
template <> __device__ __forceinline__ float ldf<float>(const void* p, int64_t idx) {
    return __ldg(reinterpret_cast<const float*>(p) + idx);
}
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const void* p, int64_t idx) {
    const unsigned short raw = __ldg(reinterpret_cast<const unsigned short*>(p) + idx);
    return __uint_as_float(static_cast<unsigned int>(raw) << 16);
}
template <typename T> __device__ __forceinline__ void stf(void* p, int64_t idx, float v);
template <> __device__ __forceinline__ void stf<float>(void* p, int64_t idx, float v) {
    reinterpret_cast<float*>(p)[idx] = v;
}
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(void* p, int64_t idx, float v) {
    reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
}

template <typename T, int AK>
__device__ __forceinline__ float load_a(const MatA& A, int64_t i, int64_t l) {
    if (AK == A_PLAIN) {
        return ldf<T>(A.p, i * A.s_row + l * A.s_col);
    } else if (AK == A_IM2COL || AK == A_IM2COL_T) {
        const int64_t pix = (AK == A_IM2COL) ? i : l;
        const int64_t q = (AK == A_IM2COL) ? l : i;
        const ConvGeom& g = A.g;
        const int c = static_cast<int>(q % g.C);
        const int tap = static_cast<int>(q / g.C);
        const int b = tap % g.kw, a = tap / g.kw;
        const int wo = static_cast<int>(pix % g.Wo);
        const int64_t t = pix / g.Wo;
        const int ho = static_cast<int>(t % g.Ho);
        const int64_t n = t / g.Ho;
        const int h = ho * g.st - g.pad + a, w = wo * g.st - g.pad + b;
        if (h < 0 || h >= g.H || w < 0 || w >= g.W) return 0.f;
        return ldf<T>(A.p, ((n * g.H + h) * g.W + w) * g.C + c);
    } else {  // A_COL2IM
        const ConvGeom& g = A.g;
        const int j = static_cast<int>(l % g.R);
        const int tap = static_cast<int>(l / g.R);
        const int b = tap % g.kw, a = tap / g.kw;
        const int w = static_cast<int>(i % g.W);
        const int64_t t = i / g.W;
        const int h = static_cast<int>(t % g.H);
        const int64_t n = t / g.H;
        const int hn = h + g.pad - a, wn = w + g.pad - b;
        if (hn < 0 || wn < 0 || hn % g.st != 0 || wn % g.st != 0) return 0.f;
        const int ho = hn / g.st, wo = wn / g.st;
        if (ho >= g.Ho || wo >= g.Wo) return 0.f;
        return ldf<T>(A.p, ((n * g.Ho + ho) * g.Wo + wo) * g.R + j);
    }
}

template <typename T, int BKD>
__device__ __forceinline__ float load_b(const MatB& B, int64_t l, int64_t j) {
    if (BKD == B_PLAIN) return ldf<T>(B.p, l * B.s_row + j * B.s_col);
    const int64_t tap = l / B.R, q = l % B.R;
    return ldf<T>(B.p, tap * B.CR + j * B.R + q);
}

template <typename T, int AK, int BKD>
__global__ void __launch_bounds__(NT)
simt_gemm_kernel(const SimtGemm g) {
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN + 1];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t i0 = static_cast<int64_t>(blockIdx.x) * BM;
    const int64_t j0 = static_cast<int64_t>(blockIdx.y) * BN;
    const int64_t kchunk = (g.K + g.splits - 1) / g.splits;
    const int64_t kbeg = static_cast<int64_t>(blockIdx.z) * kchunk;
    const int64_t kend = kbeg + kchunk < g.K ? kbeg + kchunk : g.K;

    float acc[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.f;

    for (int64_t l0 = kbeg; l0 < kend; l0 += BK) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int li, ii;
            if (g.A.l_fast) { li = tid % BK; ii = tid / BK + (NT / BK) * q; }
            else            { ii = tid % BM; li = tid / BM + (NT / BM) * q; }
            const int64_t gi = i0 + ii, gl = l0 + li;
            As[li][ii] = (gi < g.M && gl < kend) ? load_a<T, AK>(g.A, gi, gl) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int li, ji;
            if (g.B.l_fast) { li = tid % BK; ji = tid / BK + (NT / BK) * q; }
            else            { ji = tid % BN; li = tid / BN + (NT / BN) * q; }
            const int64_t gj = j0 + ji, gl = l0 + li;
            Bs[li][ji] = (gj < g.N && gl < kend) ? load_b<T, BKD>(g.B, gl, gj) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int l = 0; l < BK; ++l) {
            float a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = As[l][ty * 4 + u];
#pragma unroll
            for (int v = 0; v < 4; ++v) b[v] = Bs[l][tx * 4 + v];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t gi = i0 + ty * 4 + u;
        if (gi >= g.M) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int64_t gj = j0 + tx * 4 + v;
            if (gj >= g.N) continue;
            if (g.splits > 1) g.partial[(static_cast<int64_t>(blockIdx.z) * g.M + gi) * g.N + gj] = acc[u][v];
            else stf<T>(g.C, gi * g.ldc + gj, acc[u][v]);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ partial, void* C, int64_t ldc, int64_t M, int64_t N,
                     int splits) {
    const int64_t total = M * N;
    for (int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
         e += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        float s = 0.f;
        for (int z = 0; z < splits; ++z) s += partial[static_cast<int64_t>(z) * total + e];
        stf<T>(C, (e / N) * ldc + (e % N), s);
    }
}

template <typename T>
cudaError_t launch_typed(const SimtGemm& g, cudaStream_t stream) {
    dim3 grid(static_cast<unsigned>(ceil_div(g.M, BM)), static_cast<unsigned>(ceil_div(g.N, BN)),
              static_cast<unsigned>(g.splits));
    if (g.A.kind == A_PLAIN && g.B.kind == B_PLAIN)
        simt_gemm_kernel<T, A_PLAIN, B_PLAIN><<<grid, NT, 0, stream>>>(g);
    else if (g.A.kind == A_IM2COL && g.B.kind == B_PLAIN)
        simt_gemm_kernel<T, A_IM2COL, B_PLAIN><<<grid, NT, 0, stream>>>(g);
    else if (g.A.kind == A_IM2COL_T && g.B.kind == B_PLAIN)
        simt_gemm_kernel<T, A_IM2COL_T, B_PLAIN><<<grid, NT, 0, stream>>>(g);
    else if (g.A.kind == A_COL2IM && g.B.kind == B_TAPSPLIT)
        simt_gemm_kernel<T, A_COL2IM, B_TAPSPLIT><<<grid, NT, 0, stream>>>(g);
    else
        return cudaErrorInvalidValue;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    count_launch();
    if (g.splits > 1) {
        const int64_t total = g.M * g.N;
        const int blocks = static_cast<int>(ceil_div(total, 256) < 4 * num_sms() ? ceil_div(total, 256)
                                                                                : 4 * num_sms());
        splitk_reduce_kernel<T><<<blocks, 256, 0, stream>>>(g.partial, g.C, g.ldc, g.M, g.N, g.splits);
        e = cudaGetLastError();
        if (e == cudaSuccess) count_launch();
    }
    return e;
}

__global__ void __launch_bounds__(256)
repack_rows_kernel(const unsigned short* __restrict__ src, int64_t ld_src,
                   unsigned short* __restrict__ dst, int64_t ld_dst, int64_t rows, int64_t cols,
                   int64_t cols_padded) {
    const int64_t total = rows * cols_padded;
    for (int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
         e += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t rr = e / cols_padded, cc = e % cols_padded;
        dst[rr * ld_dst + cc] = cc < cols ? src[rr * ld_src + cc] : static_cast<unsigned short>(0);
    }
}

// Several re-pitch copies in one launch.  A work item is one 16-byte piece (8 elements) of a
// destination row: the destination is 16-byte aligned with a pitch that is a multiple of 8
// elements, the source may start anywhere, so it is read element by element.
constexpr int kRepackJobs = 6;
struct RepackBatchArgs {
    const unsigned short* src[kRepackJobs];
    unsigned short* dst[kRepackJobs];
    long long ld_src[kRepackJobs], ld_dst[kRepackJobs];
    int cols[kRepackJobs], pieces_per_row[kRepackJobs];
    long long item_end[kRepackJobs];   // running total of items up to and including job j
    int count;
};
__global__ void __launch_bounds__(256)
repack_multi_kernel(const RepackBatchArgs a) {
    const long long total = a.item_end[a.count - 1];
    for (long long it = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; it < total;
         it += static_cast<long long>(gridDim.x) * blockDim.x) {
        int j = 0;
        while (j + 1 < a.count && it >= a.item_end[j]) ++j;
        const long long local = it - (j > 0 ? a.item_end[j - 1] : 0);
        const int ppr = a.pieces_per_row[j];
        const long long row = local / ppr;
        const int c0 = static_cast<int>(local - row * ppr) * 8;
        const unsigned short* sp = a.src[j] + row * a.ld_src[j] + c0;
        const int left = a.cols[j] - c0;
        unsigned short v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = e < left ? sp[e] : static_cast<unsigned short>(0);
        uint4 o;
        o.x = v[0] | (static_cast<unsigned int>(v[1]) << 16);
        o.y = v[2] | (static_cast<unsigned int>(v[3]) << 16);
        o.z = v[4] | (static_cast<unsigned int>(v[5]) << 16);
        o.w = v[6] | (static_cast<unsigned int>(v[7]) << 16);
        *reinterpret_cast<uint4*>(a.dst[j] + row * a.ld_dst[j] + c0) = o;
    }
}

}  // namespace

int simt_pick_splits(int64_t M, int64_t N, int64_t K) {
    const int64_t tiles = ceil_div(M, BM) * ceil_div(N, BN);
    int64_t s = ceil_div(2 * num_sms(), tiles);
    const int64_t max_by_k = ceil_div(K, 8 * BK);
    if (s > max_by_k) s = max_by_k;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}

cudaError_t splitk_reduce(const float* partial, void* C, int64_t ldc, int64_t M, int64_t N, int splits,
                          int dtype, cudaStream_t stream) {
    const int64_t total = M * N;
    if (total <= 0) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 4 * num_sms() ? ceil_div(total, 256) : 4 * num_sms());
    if (dtype == PF_BF16) splitk_reduce_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(partial, C, ldc, M, N, splits);
    else splitk_reduce_kernel<float><<<blocks, 256, 0, stream>>>(partial, C, ldc, M, N, splits);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

cudaError_t simt_gemm(const SimtGemm& g, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    if (ceil_div(g.N, BN) > 65535 || ceil_div(g.M, BM) > 2147483647LL) return cudaErrorInvalidConfiguration;
    return g.dtype == PF_BF16 ? launch_typed<__nv_bfloat16>(g, stream) : launch_typed<float>(g, stream);
}

// acc[rows, cols] (fp32, dense) = (first ? 0 : acc) + src (storage dtype, pitch ld_src); and its
// counterpart that rounds the sums to the storage dtype once.  They add up the per-group input
// gradients of a grouped layer whose groups share one input, on the path that runs group by group.
template <typename T>
__global__ void accumulate_kernel(float* acc, const T* src, int64_t ld_src, int64_t rows, int64_t cols, int first) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t rr = i / cols, cc = i - rr * cols;
        const float v = static_cast<float>(src[rr * ld_src + cc]);
        acc[i] = first ? v : acc[i] + v;
    }
}
template <typename T>
__global__ void round_out_kernel(const float* acc, T* dst, int64_t ld_dst, int64_t rows, int64_t cols) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t rr = i / cols, cc = i - rr * cols;
        dst[rr * ld_dst + cc] = static_cast<T>(acc[i]);
    }
}
// out = (accumulate ? out : 0) + src, the sum taken in fp32 and rounded once to out's type.
template <typename TO, typename TS>
__global__ void grad_combine_kernel(TO* out, int64_t ld_out, const TS* src, int64_t ld_src, int64_t rows, int64_t cols,
                                    int accumulate) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t rr = i / cols, cc = i - rr * cols;
        float v = static_cast<float>(src[rr * ld_src + cc]);
        if (accumulate) v += static_cast<float>(out[rr * ld_out + cc]);
        out[rr * ld_out + cc] = static_cast<TO>(v);
    }
}
cudaError_t grad_combine(void* out, int64_t ld_out, int out_dtype, const void* src, int64_t ld_src, int src_dtype,
                         int64_t rows, int64_t cols, bool accumulate, cudaStream_t stream) {
    const int64_t total = rows * cols;
    if (total <= 0) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256) : 8 * num_sms());
    const int acc = accumulate ? 1 : 0;
    if (out_dtype == PF_F32 && src_dtype == PF_BF16)
        grad_combine_kernel<<<blocks, 256, 0, stream>>>(static_cast<float*>(out), ld_out, static_cast<const __nv_bfloat16*>(src), ld_src, rows, cols, acc);
    else if (out_dtype == PF_F32)
        grad_combine_kernel<<<blocks, 256, 0, stream>>>(static_cast<float*>(out), ld_out, static_cast<const float*>(src), ld_src, rows, cols, acc);
    else
        grad_combine_kernel<<<blocks, 256, 0, stream>>>(static_cast<__nv_bfloat16*>(out), ld_out, static_cast<const __nv_bfloat16*>(src), ld_src, rows, cols, acc);
    count_launch();
    return cudaGetLastError();
}

// The fp32 slices a split tensor-core reduction left in the workspace, summed once more in slice order
// (the very sums the reduction rounded to bf16) and written unrounded to an fp32 matrix and / or added to
// the old contents.  Slice layout: [tile][slice][128 rows][bn floats], tile = column tile * tiles_x + row
// tile, the 16-byte pieces of a row XOR-permuted by the row index.
struct SliceSumJob {
    const float* partial;
    void* out;
    long long ld;
    int M, N, S, bn, tiles_x, tiles_y, out_f32, accumulate;
};
__global__ void __launch_bounds__(256) slices_to_gradients_kernel(const SliceSumJob j0, const SliceSumJob j1, int blocks0) {
    const bool first = static_cast<int>(blockIdx.x) < blocks0;
    const SliceSumJob& j = first ? j0 : j1;
    const int b = first ? blockIdx.x : blockIdx.x - blocks0;
    const int nb = first ? blocks0 : gridDim.x - blocks0;
    const int pieces = j.bn / 4;
    const long long total = static_cast<long long>(j.tiles_x) * j.tiles_y * 128 * pieces;
    for (long long i = static_cast<long long>(b) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(nb) * blockDim.x) {
        const int pc = static_cast<int>(i % pieces);
        const long long t = i / pieces;
        const int rin = static_cast<int>(t % 128);
        const int tile = static_cast<int>(t / 128);
        const int bx = tile % j.tiles_x, by = tile / j.tiles_x;
        const int row = bx * 128 + rin, col = by * j.bn + pc * 4;
        if (row >= j.M || col >= j.N) continue;
        const float* src = j.partial + (static_cast<size_t>(tile) * j.S * 128 + rin) * j.bn + ((pc ^ (rin & (pieces - 1))) << 2);
        float4 acc = *reinterpret_cast<const float4*>(src);
        for (int s = 1; s < j.S; ++s) {
            const float4 w = *reinterpret_cast<const float4*>(src + static_cast<size_t>(s) * 128 * j.bn);
            acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
        }
        const float sums[4] = {acc.x, acc.y, acc.z, acc.w};
        const size_t at = static_cast<size_t>(row) * j.ld + col;
        for (int e = 0; e < 4 && col + e < j.N; ++e) {
            if (j.out_f32) {
                float* o = static_cast<float*>(j.out) + at + e;
                *o = j.accumulate ? *o + sums[e] : sums[e];
            } else {
                __nv_bfloat16* o = static_cast<__nv_bfloat16*>(j.out) + at + e;
                *o = __float2bfloat16_rn(j.accumulate ? __bfloat162float(*o) + sums[e] : sums[e]);
            }
        }
    }
}
cudaError_t slices_to_gradients(const SliceSums* jobs, int count, cudaStream_t stream) {
    if (count < 1 || count > 2) return cudaErrorInvalidValue;
    SliceSumJob j[2];
    int blocks[2] = {0, 0};
    for (int i = 0; i < 2; ++i) {
        const SliceSums& s = jobs[i < count ? i : 0];
        j[i] = SliceSumJob{s.partial, s.out, s.ld, s.M, s.N, s.splits, s.bn, s.tiles_x, s.tiles_y, s.out_f32 ? 1 : 0, s.accumulate ? 1 : 0};
        if (i < count) {
            const long long total = static_cast<long long>(s.tiles_x) * s.tiles_y * 128 * (s.bn / 4);
            blocks[i] = static_cast<int>(std::min<long long>(ceil_div(total, 256), 4LL * num_sms()));
            if (blocks[i] < 1) blocks[i] = 1;
        }
    }
    slices_to_gradients_kernel<<<blocks[0] + blocks[1], 256, 0, stream>>>(j[0], j[1], blocks[0]);
    count_launch();
    return cudaGetLastError();
}

// Backward of y = act(z + bias): dZ = dY where y > 0 (act = max(0, .)) or everywhere (identity), written
// over dY; partial column sums of dZ per chunk of rows go to `part` [chunks, cols] (fp32), summed in chunk
// order by the second kernel into db (deterministic).
template <typename T>
__global__ void __launch_bounds__(256) act_bwd_kernel(const T* y, int64_t ldy, T* dY, int64_t lddy, int64_t rows,
                                                      int64_t cols, int act, float* part, int rows_per_chunk) {
    const int64_t col = static_cast<int64_t>(blockIdx.x) * 32 + (threadIdx.x & 31);
    const int64_t r_beg = static_cast<int64_t>(blockIdx.y) * rows_per_chunk;
    const int64_t r_end = r_beg + rows_per_chunk < rows ? r_beg + rows_per_chunk : rows;
    float sum = 0.f;
    if (col < cols) {
        for (int64_t r = r_beg + (threadIdx.x >> 5); r < r_end; r += 8) {
            float g = static_cast<float>(dY[r * lddy + col]);
            if (act == 1 && !(static_cast<float>(y[r * ldy + col]) > 0.f)) {
                g = 0.f;
                dY[r * lddy + col] = static_cast<T>(0.f);
            }
            sum += g;
        }
    }
    __shared__ float red[8][33];
    red[threadIdx.x >> 5][threadIdx.x & 31] = sum;
    __syncthreads();
    if (threadIdx.x < 32 && col < cols && part) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += red[w][threadIdx.x];
        part[static_cast<int64_t>(blockIdx.y) * cols + col] = s;
    }
}
template <typename T>
__global__ void act_bwd_bias_kernel(const float* part, int chunks, int64_t cols, T* db) {
    const int64_t col = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (col >= cols) return;
    float s = 0.f;
    for (int c = 0; c < chunks; ++c) s += part[static_cast<int64_t>(c) * cols + col];
    db[col] = static_cast<T>(s);
}
int act_bwd_chunks(int64_t rows) {
    const int64_t c = ceil_div(rows, 256);
    return static_cast<int>(c < 1 ? 1 : (c > 64 ? 64 : c));
}
cudaError_t act_bwd(const void* y, int64_t ldy, void* dY, int64_t lddy, void* db, int64_t rows, int64_t cols, int act,
                    int dtype, float* part, cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    const int chunks = act_bwd_chunks(rows);
    const int rpc = static_cast<int>(ceil_div(rows, chunks));
    const dim3 grid(static_cast<unsigned>(ceil_div(cols, 32)), static_cast<unsigned>(chunks));
    float* pp = db ? part : nullptr;
    if (dtype == PF_BF16) {
        act_bwd_kernel<<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(y), ldy, static_cast<__nv_bfloat16*>(dY), lddy,
                                                 rows, cols, act, pp, rpc);
        if (db) act_bwd_bias_kernel<<<static_cast<unsigned>(ceil_div(cols, 256)), 256, 0, stream>>>(part, chunks, cols, static_cast<__nv_bfloat16*>(db));
    } else {
        act_bwd_kernel<<<grid, 256, 0, stream>>>(static_cast<const float*>(y), ldy, static_cast<float*>(dY), lddy, rows, cols,
                                                 act, pp, rpc);
        if (db) act_bwd_bias_kernel<<<static_cast<unsigned>(ceil_div(cols, 256)), 256, 0, stream>>>(part, chunks, cols, static_cast<float*>(db));
    }
    count_launch(db ? 2 : 1);
    return cudaGetLastError();
}

// y = act(y + bias) in place (the paths that do not fuse the epilogue into the producing kernel).
template <typename T>
__global__ void bias_act_kernel(T* y, int64_t ld, int64_t rows, int64_t cols, const T* bias, int act) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t rr = i / cols, cc = i - rr * cols;
        float v = static_cast<float>(y[rr * ld + cc]);
        if (bias) v += static_cast<float>(bias[cc]);
        if (act == 1) v = fmaxf(v, 0.f);
        y[rr * ld + cc] = static_cast<T>(v);
    }
}
cudaError_t bias_act_inplace(void* y, int64_t ld, int64_t rows, int64_t cols, const void* bias, int act, int dtype,
                             cudaStream_t stream) {
    const int64_t total = rows * cols;
    if (total <= 0 || (!bias && !act)) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256) : 8 * num_sms());
    if (dtype == PF_BF16)
        bias_act_kernel<<<blocks, 256, 0, stream>>>(static_cast<__nv_bfloat16*>(y), ld, rows, cols,
                                                    static_cast<const __nv_bfloat16*>(bias), act);
    else
        bias_act_kernel<<<blocks, 256, 0, stream>>>(static_cast<float*>(y), ld, rows, cols, static_cast<const float*>(bias), act);
    count_launch();
    return cudaGetLastError();
}
cudaError_t accumulate_f32(float* acc, const void* src, int64_t ld_src, int64_t rows, int64_t cols, int dtype, bool first,
                           cudaStream_t stream) {
    const int64_t total = rows * cols;
    if (total <= 0) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256) : 8 * num_sms());
    if (dtype == PF_BF16)
        accumulate_kernel<<<blocks, 256, 0, stream>>>(acc, static_cast<const __nv_bfloat16*>(src), ld_src, rows, cols, first ? 1 : 0);
    else
        accumulate_kernel<<<blocks, 256, 0, stream>>>(acc, static_cast<const float*>(src), ld_src, rows, cols, first ? 1 : 0);
    count_launch();
    return cudaGetLastError();
}
cudaError_t round_out_f32(const float* acc, void* dst, int64_t ld_dst, int64_t rows, int64_t cols, int dtype,
                          cudaStream_t stream) {
    const int64_t total = rows * cols;
    if (total <= 0) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256) : 8 * num_sms());
    if (dtype == PF_BF16)
        round_out_kernel<<<blocks, 256, 0, stream>>>(acc, static_cast<__nv_bfloat16*>(dst), ld_dst, rows, cols);
    else
        round_out_kernel<<<blocks, 256, 0, stream>>>(acc, static_cast<float*>(dst), ld_dst, rows, cols);
    count_launch();
    return cudaGetLastError();
}

cudaError_t repack_rows_bf16(const void* src, int64_t ld_src, void* dst, int64_t ld_dst,
                             int64_t rows, int64_t cols, int64_t cols_padded, cudaStream_t stream) {
    const int64_t total = rows * cols_padded;
    if (total <= 0) return cudaSuccess;
    const int blocks = static_cast<int>(ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256)
                                                                            : 8 * num_sms());
    repack_rows_kernel<<<blocks, 256, 0, stream>>>(static_cast<const unsigned short*>(src), ld_src,
                                                   static_cast<unsigned short*>(dst), ld_dst, rows, cols,
                                                   cols_padded);
    count_launch();
    return cudaGetLastError();
}

cudaError_t repack_rows_bf16_multi(const RepackJob* jobs, int count, cudaStream_t stream) {
    while (count > 0) {
        RepackBatchArgs a;
        a.count = 0;
        long long total = 0;
        const int n = count < kRepackJobs ? count : kRepackJobs;
        for (int i = 0; i < n; ++i) {
            const RepackJob& j = jobs[i];
            if (j.rows <= 0 || j.cols <= 0) continue;
            const bool fast = (reinterpret_cast<uintptr_t>(j.dst) & 15) == 0 && j.ld_dst % 8 == 0 &&
                              j.cols_padded == (j.cols + 7) / 8 * 8 && j.cols_padded <= j.ld_dst;
            if (!fast) {   // arbitrary destination: the element-wise copy
                cudaError_t e = repack_rows_bf16(j.src, j.ld_src, j.dst, j.ld_dst, j.rows, j.cols, j.cols_padded, stream);
                if (e != cudaSuccess) return e;
                continue;
            }
            const int k = a.count++;
            a.src[k] = static_cast<const unsigned short*>(j.src);
            a.dst[k] = static_cast<unsigned short*>(j.dst);
            a.ld_src[k] = j.ld_src; a.ld_dst[k] = j.ld_dst;
            a.cols[k] = static_cast<int>(j.cols);
            a.pieces_per_row[k] = static_cast<int>(j.cols_padded / 8);
            total += j.rows * (j.cols_padded / 8);
            a.item_end[k] = total;
        }
        if (a.count > 0) {
            for (int k = a.count; k < kRepackJobs; ++k) {
                a.src[k] = a.src[0]; a.dst[k] = a.dst[0]; a.ld_src[k] = 0; a.ld_dst[k] = 0; a.cols[k] = 0;
                a.pieces_per_row[k] = 1; a.item_end[k] = total;
            }
            const long long blocks = ceil_div(total, 256) < 8 * num_sms() ? ceil_div(total, 256) : 8 * num_sms();
            repack_multi_kernel<<<static_cast<int>(blocks), 256, 0, stream>>>(a);
            count_launch();
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return e;
        }
        jobs += n;
        count -= n;
    }
    return cudaSuccess;
}

}  // namespace pf
