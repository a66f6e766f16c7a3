// Fused two-GEMM chain for sm_100a:   out[M, N2] = (A[M, K1] * B1[K1, r]) * B2[N2, r]^T
// with the M x r intermediate kept on chip (fp32 in tensor memory, then bf16 in shared memory)
// and optionally also written out once (the stash).  It serves both
//   forward   y  = (x  U) V^T      A = x,  B1 = U [k, r],  B2 = V [n, r]
//   backward  dX = (dY V) U^T      A = dY, B1 = V [n, r],  B2 = U [k, r]
// of the factorized linear layer.
//
// One CTA owns one 128-row tile of A (and a contiguous range of 128-column output tiles when the
// grid splits N2 to fill the machine; each split then recomputes the intermediate).
//   phase 1  T = A * B1: TMA ring over K1 in 64-element blocks; A tile is a K-major operand,
//            the B1 tile [64 x r] is an MN-major operand (r contiguous in memory); fp32
//            accumulator of r columns in TMEM.
//   switch   the four epilogue warps read T from TMEM, round to bf16 and lay it out in shared
//            memory as the K-major (128-byte swizzled) A operand of phase 2; the same bytes are
//            what TMA stores as the stash.
//   phase 2  for each 128-column tile: out_tile = T * B2_tile^T with B2 tiles streamed through
//            the same ring; accumulators double-buffered in TMEM so the MMAs of tile j+1 overlap
//            the epilogue of tile j; the epilogue stages bf16 rows in swizzled shared memory and
//            writes them with TMA stores (coalesced, clipped at the matrix edge).
// Shared memory: control block | T (r_pad x 256 B) | ring of stages (16 KB A or B2 tile + r_pad x
// 128 B B1 tile).  In phase 2 the B1 part of every stage is idle and serves as store staging.
#include <cuda.h>

#include "pf_tc.h"
#include "pf_tc_host.h"
#include "pf_tc_prims.cuh"

namespace pf {
namespace tc {
namespace {

constexpr int kMaxStages = 8;
constexpr int kChainThreads = 352;          // A producer, MMA warp, 8 epilogue warps, B producer
constexpr uint32_t kTileBytes = 16384;      // 128 rows x 64 bf16
constexpr int kAccBufs = 4;                 // 4 x 128 TMEM columns of phase-2 accumulators
constexpr int kEarlyTiles = 8;              // tiles of A requested into L2 before the dependency wait

struct ChainCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t t_full;        // phase-1 accumulator complete
    uint64_t t_ready;       // bf16 T is in shared memory (one arrival per epilogue warp)
    uint64_t acc_full[kAccBufs];
    uint64_t acc_empty[kAccBufs];
    uint32_t tmem_base;
    uint32_t abort;
};

struct ChainParams {
    int M, K1, N2;
    int r_pad;              // r rounded up to a multiple of 64, <= 384
    int num_stages;
    int stage_bytes;        // 16384 + r_pad * 128
    int tiles_per_split;    // 128-column output tiles per blockIdx.y (0: phase 1 only)
    int store_T;
    int boxes_per_stage;    // phase 2: B2 boxes (16 KB each) loaded per ring stage
    int staging_off;        // byte offset (from the 1 KB-aligned base) of dedicated store staging, 0 = none
    // Implicit-GEMM convolution as phase 1 (conv_cblks > 0): tmA is a 4-D NHWC map, a row tile is
    // box_h full-width image rows (box_h * W = 128 pixels) and k-block kb = (tap, 64-channel block).
    int conv_cblks, conv_kw, conv_pad, conv_box_h, conv_tiles_per_img;
    int rows_tile;          // rows of A one CTA owns: 128, or box_h * W pixels (<= 128) for the convolution
    unsigned int* status;
};

__device__ __forceinline__ uint4 pack8(const uint32_t* v) {
    uint4 o;
    o.x = pack_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
    o.y = pack_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
    o.z = pack_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
    o.w = pack_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
    return o;
}

// Ring position: stage index, its byte offset and the phase bit, advanced without divisions.
struct RingPos {
    uint32_t s = 0, off = 0, ph = 0;
    __device__ __forceinline__ void advance(uint32_t ns, uint32_t stage_bytes) {
        if (++s == ns) { s = 0; off = 0; ph ^= 1u; } else { off += stage_bytes; }
    }
};

__global__ void __launch_bounds__(kChainThreads, 1)
tc_chain_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB1,
                const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmOut,
                const __grid_constant__ CUtensorMap tmT, const ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    ChainCtl* ctl = reinterpret_cast<ChainCtl*>(smem);
    const uint32_t t_smem = smem_u32(smem + 1024);
    const uint32_t ring = t_smem + static_cast<uint32_t>(p.r_pad) * 256u;
    volatile uint32_t* abort_flag = &ctl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * p.rows_tile;
    const int nt_total = (p.N2 + 127) / 128;
    const int t_beg = blockIdx.y * p.tiles_per_split;
    const int ntile = max(0, min(nt_total, t_beg + p.tiles_per_split) - t_beg);
    const int nkb1 = (p.K1 + 63) / 64;
    const int nkb2 = p.r_pad / 64;
    const uint32_t NS = static_cast<uint32_t>(p.num_stages);
    const uint32_t S = static_cast<uint32_t>(p.stage_bytes);
    const int bps = p.boxes_per_stage;

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2);     // one arrival per producer thread
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->t_full), 1);
        mbar_init(smem_u32(&ctl->t_ready), 8);
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), 8);
        }
        ctl->abort = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB1);
        tma_prefetch_desc(&tmB2);
        tma_prefetch_desc(&tmOut);
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // While the previous kernel of the stream finishes, ask L2 for this block's first tiles.  A prefetch
    // only moves lines into L2, the point of coherence, so it is harmless even if that kernel is
    // still writing the tensor; the loads that consume the data are issued after the wait below.
    if (p.conv_cblks == 0) {
        if (warp == 0 && elect_one()) {
            for (int kb = 0; kb < kEarlyTiles && kb < nkb1; ++kb) tma_prefetch_l2_2d(&tmA, kb * 64, m0);
        } else if (warp == 10 && elect_one()) {
            for (int kb = 0; kb < 2 && kb < nkb1; ++kb)
                for (int q = 0; q < nkb2; ++q) tma_prefetch_l2_2d(&tmB1, q * 64, kb * 64);
        }
    }
    pdl_wait();                 // everything above overlapped the previous kernel's tail
    pdl_launch_dependents();
    const uint32_t tmem = ctl->tmem_base;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);

    // Producer and MMA issuer are each ONE thread chosen with elect.sync, running its whole role.
    // (A thread singled out by a lane-id test issues tcgen05 / TMA instructions several times
    // slower, and the issuing thread's own instruction latency is on the critical path, so the
    // loops below carry running offsets instead of recomputing them.)
    if (warp == 0) {
        if (elect_one()) {
            // -------------------------------------------------------------- TMA producer of A (phase 1)
            RingPos rp;
            const uint32_t txa = static_cast<uint32_t>(p.rows_tile) * 128u;
            // convolution: (tap row, tap column, channel block) advance as counters; integer divisions
            // in this loop would sit on the producer's critical path
            const int cv_img = p.conv_cblks > 0 ? static_cast<int>(blockIdx.x) / p.conv_tiles_per_img : 0;
            const int cv_h0 = (static_cast<int>(blockIdx.x) - cv_img * p.conv_tiles_per_img) * p.conv_box_h - p.conv_pad;
            int cv_cb = 0, cv_ta = 0, cv_tb = 0;
            for (int kb = 0; kb < nkb1; ++kb) {
                if (!mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status)) break;
                const uint32_t full = full0 + 8 * rp.s;
                const uint32_t dst = ring + rp.off;
                mbar_expect_tx(full, txa);
                if (p.conv_cblks > 0) {
                    tma_load_4d(dst, &tmA, full, cv_cb * 64, cv_tb - p.conv_pad, cv_h0 + cv_ta, cv_img);
                    if (++cv_cb == p.conv_cblks) {
                        cv_cb = 0;
                        if (++cv_tb == p.conv_kw) { cv_tb = 0; ++cv_ta; }
                    }
                } else {
                    tma_load_2d(dst, &tmA, full, kb * 64, m0);
                }
                rp.advance(NS, S);
            }
        }
    } else if (warp == 10) {
        if (elect_one()) {
            // -------------------------------------------------------------- TMA producer of B1 and B2
            // (a second thread: a producer spends about 130 ns per stage on its loop, barrier wait and
            // expect_tx and 40 ns per TMA instruction, which paced phase 1 when one thread issued both)
            RingPos rp;
            bool ok = true;
            // Phase 2 streams B2 tiles that nobody has touched yet; have L2 fetch them while phase 1
            // runs.  The CTAs that share these tiles each ask for a different one.
            if (ntile > 0) {
                const int n0 = (t_beg + static_cast<int>(blockIdx.x) % ntile) * 128;
                for (int q = 0; q < nkb2; ++q) tma_prefetch_l2_2d(&tmB2, q * 64, n0);
            }
            const uint32_t txb = static_cast<uint32_t>(p.r_pad) * 128u;
            for (int kb = 0; kb < nkb1; ++kb) {
                ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                if (!ok) break;
                const uint32_t full = full0 + 8 * rp.s;
                const uint32_t dst = ring + rp.off + kTileBytes;
                mbar_expect_tx(full, txb);
                for (int q = 0; q < nkb2; ++q) tma_load_2d(dst + q * 8192, &tmB1, full, q * 64, kb * 64);
                rp.advance(NS, S);
            }
            for (int j = 0; j < ntile && ok; ++j) {
                const int n0 = (t_beg + j) * 128;
                for (int kb = 0; kb < nkb2; kb += bps) {
                    const int nb = min(bps, nkb2 - kb);
                    ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    const uint32_t full = full0 + 8 * rp.s;
                    mbar_arrive(full);                      // stands in for the A producer, idle in phase 2
                    mbar_expect_tx(full, kTileBytes * nb);
                    for (int q = 0; q < nb; ++q)
                        tma_load_2d(ring + rp.off + q * kTileBytes, &tmB2, full, (kb + q) * 64, n0);
                    rp.advance(NS, S);
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            // -------------------------------------------------------------- MMA issuer
            RingPos rp;
            bool ok = true;
            const int n1a = min(256, p.r_pad), n1b = p.r_pad - n1a;
            const uint32_t idesc_a = make_idesc_bf16(128, n1a, 0, 1);
            const uint32_t idesc_b = make_idesc_bf16(128, n1b > 0 ? n1b : 64, 0, 1);
            const uint64_t a_ring = make_smem_desc(ring, 16, 1024);                    // K-major tile at a stage start
            const uint64_t b1_ring = make_smem_desc(ring + kTileBytes, 8192, 1024);   // MN-major B1 tile of a stage
            for (int kb = 0; kb < nkb1; ++kb) {
                ok = mbar_wait(full0 + 8 * rp.s, rp.ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint64_t a_desc = a_ring + (rp.off >> 4), b_desc = b1_ring + (rp.off >> 4);
                const uint32_t acc0 = kb > 0 ? 1u : 0u;
                tc_mma_bf16(tmem, a_desc, b_desc, idesc_a, acc0);
                tc_mma_bf16(tmem, a_desc + 2, b_desc + 128, idesc_a, 1u);
                tc_mma_bf16(tmem, a_desc + 4, b_desc + 256, idesc_a, 1u);
                tc_mma_bf16(tmem, a_desc + 6, b_desc + 384, idesc_a, 1u);
                if (n1b > 0) {
                    const uint64_t b2 = b_desc + (4 * 8192 >> 4);
                    tc_mma_bf16(tmem + 256, a_desc, b2, idesc_b, acc0);
                    tc_mma_bf16(tmem + 256, a_desc + 2, b2 + 128, idesc_b, 1u);
                    tc_mma_bf16(tmem + 256, a_desc + 4, b2 + 256, idesc_b, 1u);
                    tc_mma_bf16(tmem + 256, a_desc + 6, b2 + 384, idesc_b, 1u);
                }
                tc_commit(empty0 + 8 * rp.s);
                rp.advance(NS, S);
            }
            if (ok) tc_commit(smem_u32(&ctl->t_full));
            if (ok) ok = mbar_wait(smem_u32(&ctl->t_ready), 0, abort_flag, p.status);
            tc_fence_after();
            const bool stash = ok && p.store_T && blockIdx.y == 0;
            if (stash) {
                for (int q = 0; q < nkb2; ++q) {
                    if (p.conv_cblks > 0) tma_store_3d(&tmT, t_smem + q * kTileBytes, q * 64, 0, blockIdx.x);
                    else tma_store_2d(&tmT, t_smem + q * kTileBytes, q * 64, m0);
                }
                tma_store_commit();
            }
            const uint32_t idesc2 = make_idesc_bf16(128, 128, 0, 0);
            const uint64_t t_desc = make_smem_desc(t_smem, 16, 1024);
            const uint32_t accf0 = smem_u32(&ctl->acc_full[0]), acce0 = smem_u32(&ctl->acc_empty[0]);
            for (int j = 0; j < ntile && ok; ++j) {
                const uint32_t b = static_cast<uint32_t>(j) & (kAccBufs - 1);
                ok = mbar_wait(acce0 + 8 * b, ((static_cast<uint32_t>(j) / kAccBufs) & 1u) ^ 1u, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem + b * 128;
                for (int kb = 0; kb < nkb2; kb += bps) {
                    const int nb = min(bps, nkb2 - kb);
                    ok = mbar_wait(full0 + 8 * rp.s, rp.ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    for (int q = 0; q < nb; ++q) {
                        const uint64_t a_desc = t_desc + static_cast<uint32_t>((kb + q) * (kTileBytes >> 4));
                        const uint64_t b_desc = a_ring + ((rp.off + q * kTileBytes) >> 4);
                        tc_mma_bf16(d_tmem, a_desc, b_desc, idesc2, (kb + q) > 0 ? 1u : 0u);
                        tc_mma_bf16(d_tmem, a_desc + 2, b_desc + 2, idesc2, 1u);
                        tc_mma_bf16(d_tmem, a_desc + 4, b_desc + 4, idesc2, 1u);
                        tc_mma_bf16(d_tmem, a_desc + 6, b_desc + 6, idesc2, 1u);
                    }
                    tc_commit(empty0 + 8 * rp.s);
                    rp.advance(NS, S);
                }
                if (ok) tc_commit(accf0 + 8 * b);
            }
            if (stash) tma_store_wait_read<0>();
        }
    } else if (warp < 10) {
        // ------------------------------------------------------------------ epilogue warps
        // Eight warps: warp w may touch the TMEM lanes of quadrant w % 4, so two warps share each
        // 32-row quadrant and split the columns (64 of every 128) between them.
        const int q = warp & 3;
        const int hcol = (warp - 2) >> 2;            // 0 or 1: which 64-column half of a tile
        const int row = q * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(q * 32) << 16);
        bool ok = mbar_wait_warp(smem_u32(&ctl->t_full), 0, abort_flag, p.status);
        tc_fence_after();
        const uint32_t sw = static_cast<uint32_t>(lane & 7);      // == row & 7
        if (ok) {
            for (int c = hcol; c < p.r_pad / 32; c += 2) {
                uint32_t v[32];
                tmem_ld32(lane_base + c * 32, v);
                tmem_ld_wait();
                const uint32_t panel = t_smem + (c >> 1) * kTileBytes + row * 128;
                const uint32_t cb = (c & 1) * 4;
#pragma unroll
                for (int t = 0; t < 4; ++t) st_shared_v4(panel + (((cb + t) ^ sw) << 4), pack8(v + 8 * t));
            }
            tc_fence_before();
            fence_proxy_async_smem();
        }
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(smem_u32(&ctl->t_ready));

        // Store staging: one 4 KB panel (32 rows x 64 columns) per warp, either in a dedicated
        // region or (large r) in the B1 part of ring stages, which is idle during phase 2.
        const int ew = warp - 2;                      // 0..7
        uint32_t stg;
        if (p.staging_off) {
            stg = smem_u32(smem + p.staging_off) + ew * 4096;
        } else {
            const int per_stage = p.r_pad / 32;       // 4 KB pieces in the B1 part of one stage
            stg = ring + (ew / per_stage) * S + kTileBytes + (ew % per_stage) * 4096;
        }
        bool stored = false;
        const int r0 = m0 + q * 32;
        const uint32_t prow = stg + lane * 128;
        for (int j = 0; j < ntile && ok; ++j) {
            const uint32_t b = static_cast<uint32_t>(j) & (kAccBufs - 1);
            ok = mbar_wait_warp(smem_u32(&ctl->acc_full[b]), (static_cast<uint32_t>(j) / kAccBufs) & 1u, abort_flag,
                                p.status);
            tc_fence_after();
            if (!ok) break;
            // drain this warp's 64 columns and hand the TMEM buffer back before converting
            uint32_t v[2][32];
            tmem_ld32(lane_base + b * 128 + hcol * 64, v[0]);
            tmem_ld32(lane_base + b * 128 + hcol * 64 + 32, v[1]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                tma_store_wait_read<0>();             // the previous store has finished reading the panel
            }
            __syncwarp();
#pragma unroll
            for (int t = 0; t < 8; ++t)
                st_shared_v4(prow + ((static_cast<uint32_t>(t) ^ sw) << 4), pack8(v[t >> 2] + 8 * (t & 3)));
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                const int n0 = (t_beg + j) * 128 + hcol * 64;
                if (r0 < p.M && q * 32 < p.rows_tile && n0 < p.N2) {
                    if (p.conv_cblks > 0) tma_store_3d(&tmOut, stg, n0, q * 32, blockIdx.x);
                    else tma_store_2d(&tmOut, stg, n0, r0);
                    tma_store_commit();
                    stored = true;
                }
            }
        }
        if (lane == 0 && stored) tma_store_wait_read<0>();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace

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

// out may be null (phase 1 only: T is written and nothing else).  All pointers must satisfy tma_ok.
int chain(const void* A, int64_t lda, int64_t M, int64_t K1, const void* B1, int64_t ldb1, int64_t r,
          const void* B2, int64_t ldb2, int64_t N2, void* out, int64_t ldo, void* T, int64_t ldt,
          cudaStream_t stream, const ChainConv* conv, int max_split) {
    ChainPlan plan;
    const int box_h = conv ? conv_box_h(conv->H, conv->W, 128) : 1;
    const int rows_tile = conv ? box_h * conv->W : 128;
    if (!chain_plan(M, K1, N2, r, out != nullptr, &plan, rows_tile, max_split)) return PF_ERR_UNSUPPORTED;
    CUtensorMap ta, tb1, tb2, to, tt;
    bool ok = conv ? cached_map_nhwc(&ta, A, conv->N, conv->H, conv->W, conv->C, conv->W, box_h)
                   : cached_map_2d(&ta, A, M, K1, lda, 128);
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
        p.conv_box_h = box_h; p.conv_tiles_per_img = conv->H / box_h;
    }
    p.rows_tile = rows_tile;
    p.status = device_status_ptr();
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    dim3 grid(static_cast<unsigned>(plan.row_tiles), static_cast<unsigned>(plan.nsplit), 1);
    if (launch_overlapped(tc_chain_kernel, grid, dim3(kChainThreads), plan.smem, stream, ta, tb1, tb2, to, tt, p) !=
        cudaSuccess)
        return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

}  // namespace tc
}  // namespace pf
