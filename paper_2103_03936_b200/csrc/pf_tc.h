// Tensor-core (tcgen05 / TMEM / TMA) path for bf16 storage.  Each entry either handles the
// call (*handled = 1) or declines it (*handled = 0, nothing launched) when the shape lies
// outside its envelope; the caller then uses the FMA kernels.
#ifndef PF_TC_H_
#define PF_TC_H_

#include "pf_internal.h"

namespace pf {

unsigned int* device_status_ptr();  // per-device address of the bounded-wait status word

namespace tc {

struct LinearArgs {
    const void *x = nullptr, *U = nullptr, *V = nullptr, *dY = nullptr;
    void *y = nullptr, *T = nullptr, *dX = nullptr, *dU = nullptr, *dV = nullptr;
    int64_t ldx = 0, ldu = 0, ldv = 0, ldy = 0, ldt = 0, lddy = 0, lddx = 0, lddu = 0, lddv = 0;
    int64_t m = 0, k = 0, n = 0, r = 0;
    char *ws = nullptr, *ws_T = nullptr, *ws_G = nullptr;
    cudaStream_t stream = nullptr;
    const void* bias = nullptr;   // forward: y = act((x U) V^T + bias)
    int act = 0;
    // backward: where the fp32 slices of dU / dV were left in the workspace (filled in when the reduction
    // over the batch was split across thread blocks; splits <= 1 otherwise), for callers that want the
    // unrounded sums
    struct Slices {
        const float* partial = nullptr;
        int splits = 0, bn = 0, tiles_x = 0, tiles_y = 0;
    };
    Slices* du_slices = nullptr;
    Slices* dv_slices = nullptr;
};

struct ConvArgs {
    const void *x, *U, *V, *dY;
    void *y, *T, *dX, *dU, *dV;
    int N, H, W, C, R, O, kh, kw, stride, pad, Ho, Wo;
    char *ws, *ws_T, *ws_G;
    cudaStream_t stream;
    // backward: where the fp32 slices of dU / dV were left (see LinearArgs::Slices); may be null
    LinearArgs::Slices *du_slices, *dv_slices;
};

// Fused chain kernel (pf_tc_chain.cu): out = (A * B1) * B2^T with the intermediate on chip.
struct ChainPlan {
    int r_pad, num_stages, stage_bytes, nsplit, tiles_per_split, row_tiles, boxes_per_stage, staging_off;
    size_t smem;
};
// `max_split` caps the number of column ranges the output is split into (0 = no cap).
bool chain_plan(int64_t M, int64_t K1, int64_t N2, int64_t r, bool has_out, ChainPlan* plan, int rows_tile = 128,
                int max_split = 0);
int conv_box_h(int H, int W, int limit);
// When `conv` is given, A is an NHWC image and phase 1 is the implicit GEMM of a kh x kw, stride-1,
// "same"-padded convolution: M = N*H*W pixels, K1 = kh*kw*C, B1 = U as a (kh*kw*C) x r matrix.
// stride (1 or 2) applies to the k x k convolution: M = N*Ho*Wo output pixels, and the image tile of a tap
// is fetched with that step between pixels (a tensor map with element strides).
struct ChainConv {
    int N, H, W, C, kh, kw, pad;
    int stride = 1;
};
int chain(const void* A, int64_t lda, int64_t M, int64_t K1, const void* B1, int64_t ldb1, int64_t r,
          const void* B2, int64_t ldb2, int64_t N2, void* out, int64_t ldo, void* T, int64_t ldt,
          cudaStream_t stream, const ChainConv* conv = nullptr, int max_split = 0, const void* bias = nullptr,
          int act = 0);   // bias [N2] (bf16) and act (0 identity, 1 max(0, .)) apply to `out`

// Plain product on CTA pairs (pf_tc_pair.cu); PF_ERR_UNSUPPORTED when the output is not 16-byte aligned
// with a pitch that is a multiple of 8 elements.
int gemm_pair_2sm(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb, bool b_mn, int64_t M, int64_t N,
                  int64_t K, void* C, int64_t ldc, cudaStream_t stream);

// Grouped factorized linear layer: `groups` problems of one shape (several factor pairs applied to the
// same or to different inputs) in two launches forward and two backward, whatever the group count.
// Strides s* are in elements between consecutive groups; sx == 0 means one x shared by all groups,
// in which case dX is ONE matrix, the sum over the groups.
struct GroupedArgs {
    int groups = 1;
    const void *x = nullptr, *U = nullptr, *V = nullptr, *dY = nullptr;
    void *y = nullptr, *T = nullptr, *dX = nullptr, *dU = nullptr, *dV = nullptr;
    int64_t ldx = 0, ldu = 0, ldv = 0, ldy = 0, ldt = 0, lddy = 0, lddx = 0, lddu = 0, lddv = 0;
    int64_t sx = 0, su = 0, sv = 0, sy = 0, st = 0, sdy = 0, sdx = 0, sdu = 0, sdv = 0;
    int64_t m = 0, k = 0, n = 0, r = 0;
    char* ws = nullptr;
    cudaStream_t stream = nullptr;
};
size_t grouped_workspace(int groups, int64_t m, int64_t k, int64_t n, int64_t r, bool bwd);
int linear_grouped_fwd(const GroupedArgs& a, int* handled);
int linear_grouped_bwd(const GroupedArgs& a, int* handled);

size_t linear_extra_workspace(int64_t m, int64_t k, int64_t n, int64_t r, bool bwd);
size_t conv_extra_workspace(int N, int H, int W, int C, int R, int O, int kh, int kw, int stride,
                            int pad, bool bwd);
void reset_fix_counters();  // clears the slice-sum counters (after PF_ERR_TIMEOUT)
size_t linear_fwd_need(const LinearArgs& a, bool* handles);   // bytes of a.ws the forward really touches
int linear_fwd(const LinearArgs& a, int* handled);
int linear_bwd(const LinearArgs& a, int* handled);
int conv_fwd(const ConvArgs& a, int* handled);
int conv_bwd(const ConvArgs& a, int* handled);

}  // namespace tc
}  // namespace pf
#endif
