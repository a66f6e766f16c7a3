// Host side of the fused two-GEMM chain (kernel: pf_tc_chain_kernel.cuh): shape envelope, launch
// geometry, tensor maps, and the launch of the single-tile form.
#include <cuda.h>

#include "pf_tc.h"
#include "pf_tc_host.h"
#include "pf_tc_chain_kernel.cuh"

namespace pf {
namespace tc {

// Largest number of full-width image rows (a divisor of H) whose pixels fit in `limit` tile rows.
int conv_box_h(int H, int W, int limit) {
    int best = 1;
    for (int d = 1; d <= H; ++d)
        if (H % d == 0 && d * W <= limit) best = d;
    return best;
}

// Shape envelope of the fused kernel and its launch geometry.
bool chain_plan(int64_t M, int64_t K1, int64_t N2, int64_t r, bool has_out, ChainPlan* plan, int rows_tile, int max_split) {
    const int64_t r_pad = (r + 63) / 64 * 64;
    if (r_pad > 384 || M > 0x7fffffff || K1 > 0x7fffffff || N2 > 0x7fffffff) return false;
    const int64_t stage = kTileBytes + r_pad * 128;
    // Small ranks: dedicated 32 KB store staging, and a whole B2 tile (r_pad / 64 boxes) per stage
    // in phase 2.  Larger ranks: staging lives in the idle B1 part of the stages, one box per stage.
    const bool dedicated = r_pad <= 128;
    const int64_t budget = 227 * 1024 - 2048 - r_pad * 256 - (dedicated ? 32768 : 0);
    int64_t ns = budget / stage;
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns < 2 || (!dedicated && ns * (r_pad / 32) < 8)) return false;
    const int64_t row_tiles = ceil_div(M, rows_tile), nt = ceil_div(N2, 128);
    // Split N2 over blockIdx.y while that shortens the critical path of a CTA (each split repeats
    // phase 1, cost ~ K1; phase 2 costs ~ N2 / split) and the grid still fits one wave.
    int64_t best = 1;
    if (has_out) {
        double best_cost = 1e30;
        for (int64_t s = 1; s <= nt && (s == 1 || row_tiles * s <= num_sms()) && (max_split <= 0 || s <= max_split); ++s) {
            const double waves = static_cast<double>(ceil_div(row_tiles * s, num_sms()));
            const double cost = waves * (static_cast<double>(K1) + 128.0 * ceil_div(nt, s));
            if (cost < best_cost * 0.97) { best_cost = cost; best = s; }
        }
    }
    plan->r_pad = static_cast<int>(r_pad);
    plan->num_stages = static_cast<int>(ns);
    plan->stage_bytes = static_cast<int>(stage);
    plan->nsplit = static_cast<int>(has_out ? best : 1);
    plan->tiles_per_split = has_out ? static_cast<int>(ceil_div(nt, best)) : 0;
    plan->nsplit = has_out ? static_cast<int>(ceil_div(nt, plan->tiles_per_split)) : 1;
    plan->smem = static_cast<size_t>(2048 + r_pad * 256 + ns * stage + (dedicated ? 32768 : 0));
    plan->boxes_per_stage = dedicated ? static_cast<int>(r_pad / 64) : 1;
    plan->staging_off = dedicated ? static_cast<int>(1024 + r_pad * 256 + ns * stage) : 0;
    plan->row_tiles = static_cast<int>(row_tiles);
    return true;
}

// NHWC image map whose boxes take every `stride`-th pixel along W and H: box_w x box_h pixels of 64
// channels are loaded (the box extents are given in traversed elements, i.e. times the stride).
static bool make_map_nhwc_strided(CUtensorMap* map, const void* p, int64_t N, int64_t H, int64_t W, int64_t C, int box_w,
                                  int box_h, int stride) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(H),
                                static_cast<cuuint64_t>(N)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(C) * 2, static_cast<cuuint64_t>(W) * C * 2,
                                   static_cast<cuuint64_t>(H) * W * C * 2};
    const cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(box_w * stride), static_cast<cuuint32_t>(box_h * stride), 1u};
    const cuuint32_t estr[4] = {1u, static_cast<cuuint32_t>(stride), static_cast<cuuint32_t>(stride), 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(p), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// out may be null (phase 1 only: T is written and nothing else).  All pointers must satisfy tma_ok.
int chain(const void* A, int64_t lda, int64_t M, int64_t K1, const void* B1, int64_t ldb1, int64_t r,
          const void* B2, int64_t ldb2, int64_t N2, void* out, int64_t ldo, void* T, int64_t ldt,
          cudaStream_t stream, const ChainConv* conv, int max_split, const void* bias, int act) {
    ChainPlan plan;
    const int cs = conv ? conv->stride : 1;
    const int Ho = conv ? (conv->H + 2 * conv->pad - conv->kh) / cs + 1 : 1;
    const int Wo = conv ? (conv->W + 2 * conv->pad - conv->kw) / cs + 1 : 1;
    const int box_h = conv ? conv_box_h(Ho, Wo, 128) : 1;          // output rows of one tile
    const int rows_tile = conv ? box_h * Wo : 128;
    if (conv && (Wo > 128 || cs * Wo > 256 || cs * box_h > 256)) return PF_ERR_UNSUPPORTED;
    if (!chain_plan(M, K1, N2, r, out != nullptr, &plan, rows_tile, max_split)) return PF_ERR_UNSUPPORTED;
    CUtensorMap ta, tb1, tb2, to, tt;
    bool ok = !conv ? cached_map_2d(&ta, A, M, K1, lda, 128)
              : cs == 1 ? cached_map_nhwc(&ta, A, conv->N, conv->H, conv->W, conv->C, conv->W, box_h)
                        : make_map_nhwc_strided(&ta, A, conv->N, conv->H, conv->W, conv->C, Wo, box_h, cs);
    ok = ok && cached_map_2d(&tb1, B1, K1, r, ldb1, 64) && cached_map_2d(&tb2, B2, N2, r, ldb2, 128);
    if (conv) {   // outputs seen as [tiles][rows_tile][cols] so that partial tiles are clipped per tile
        ok = ok && (out ? cached_map_tiled_rows(&to, out, M / rows_tile, rows_tile, N2, 32)
                        : cached_map_2d(&to, B2, N2, r, ldb2, 32));
        ok = ok && (T ? cached_map_tiled_rows(&tt, T, M / rows_tile, rows_tile, r, rows_tile)
                      : cached_map_2d(&tt, B2, N2, r, ldb2, 128));
    } else {
        ok = ok && (out ? cached_map_2d(&to, out, M, N2, ldo, 32) : cached_map_2d(&to, B2, N2, r, ldb2, 32));
        ok = ok && (T ? cached_map_2d(&tt, T, M, r, ldt, 128) : cached_map_2d(&tt, B2, N2, r, ldb2, 128));
    }
    if (!ok) return PF_ERR_CUDA;
    ChainParams p;
    p.M = static_cast<int>(M); p.K1 = static_cast<int>(K1); p.N2 = static_cast<int>(N2);
    p.r_pad = plan.r_pad; p.num_stages = plan.num_stages; p.stage_bytes = plan.stage_bytes;
    p.tiles_per_split = plan.tiles_per_split; p.store_T = T != nullptr;
    p.boxes_per_stage = plan.boxes_per_stage; p.staging_off = plan.staging_off;
    p.conv_cblks = 0; p.conv_kw = 1; p.conv_pad = 0; p.conv_box_h = 1; p.conv_tiles_per_img = 1;
    if (conv) {
        p.conv_cblks = conv->C / 64; p.conv_kw = conv->kw; p.conv_pad = conv->pad;
        // the kernel places tile i of an image at input row i * conv_box_h - pad: stride x the output rows
        p.conv_box_h = box_h * cs; p.conv_tiles_per_img = Ho / box_h;
    }
    p.rows_tile = rows_tile;
    p.row_tiles = plan.row_tiles;
    // More row tiles than SMs: a persistent grid of equally loaded CTAs whose tiles overlap (phase 1 of
    // the next under the stores of the current), with the output accumulators behind T's in TMEM.
    int grid_x = plan.row_tiles;
    p.acc_base = 0; p.acc_bufs = kAccBufs;
    const bool persistent = plan.r_pad <= 128 && plan.nsplit == 1 && plan.row_tiles > num_sms();
    if (persistent) {
        const int per_cta = static_cast<int>(ceil_div(plan.row_tiles, num_sms()));
        grid_x = static_cast<int>(ceil_div(plan.row_tiles, per_cta));
        p.acc_base = 128; p.acc_bufs = 3;
    }
    p.bias = bias; p.act = act;
    p.status = device_status_ptr();
    dim3 grid(static_cast<unsigned>(grid_x), static_cast<unsigned>(plan.nsplit), 1);
    if (out && (bias || act)) return chain_launch_act(persistent, grid, plan.smem, stream, ta, tb1, tb2, to, tt, p);
    if (persistent && plan.r_pad <= 128) {
        // software-pipelined form: two T accumulators and two T buffers, the ring behind them, then the
        // 32 KB of store staging; output accumulators in what tensor memory the T accumulators leave
        const int64_t stage = plan.stage_bytes, t2 = 2 * static_cast<int64_t>(plan.r_pad) * 256;
        int64_t ns = (227 * 1024 - 2048 - t2 - 32768) / stage;
        if (ns > kMaxStages) ns = kMaxStages;
        if (ns >= 3) {
            p.num_stages = static_cast<int>(ns);
            p.staging_off = static_cast<int>(1024 + t2 + ns * stage);
            p.boxes_per_stage = plan.r_pad / 64;
            p.acc_base = 2 * plan.r_pad;
            p.acc_bufs = (512 - 2 * plan.r_pad) / 128;
            return chain_launch_pipe(grid, static_cast<size_t>(2048 + t2 + ns * stage + 32768), stream, ta, tb1, tb2, to, tt, p);
        }
    }
    if (persistent) return chain_launch_multi(grid, plan.smem, stream, ta, tb1, tb2, to, tt, p);
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_chain_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    if (launch_overlapped(tc_chain_kernel<false>, grid, dim3(kChainThreads), plan.smem, stream, ta, tb1, tb2, to, tt, p) !=
        cudaSuccess)
        return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

}  // namespace tc
}  // namespace pf
