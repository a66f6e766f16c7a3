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
// When there are more row tiles than SMs (and r <= 128) the kernel is persistent: a CTA walks over row
// tiles blockIdx.x, blockIdx.x + gridDim.x, ...; the producers run ahead into the next tile's phase 1
// while the epilogue warps still convert and store the outputs of the current one, and the phase-2
// accumulators then live beside T's in tensor memory (128 + 3 x 128 columns) instead of on top of it.
// Shared memory: control block | T (r_pad x 256 B) | ring of stages (16 KB A or B2 tile + r_pad x
// 128 B B1 tile).  In phase 2 the B1 part of every stage is idle and serves as store staging.
// This header holds the kernel (a template, instantiated once per translation unit: the single-tile
// form in pf_tc_chain.cu, the persistent form in pf_tc_chain_multi.cu, so that each lives in a module
// of its own) and the parameter block the host fills.
#ifndef PF_TC_CHAIN_KERNEL_CUH_
#define PF_TC_CHAIN_KERNEL_CUH_

#include <cuda.h>

#include "pf_tc_prims.cuh"

namespace pf {
namespace tc {

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
    int rows_tile;          // rows of A in one tile: 128, or box_h * W pixels (<= 128) for the convolution
    int row_tiles;          // tiles along M; a CTA takes tiles blockIdx.x, blockIdx.x + gridDim.x, ...
    int acc_base, acc_bufs; // TMEM column of the first phase-2 accumulator and their number (4 on top of T's
                            // columns, or 3 behind them when tiles overlap)
    // Output epilogue of the kEpi form: out = act(acc + bias), bias [N2] in bf16 (null = none),
    // act 0 = identity, 1 = max(0, .); applied in fp32 before the single rounding to bf16.
    const void* bias;
    int act;
    unsigned int* status;
};

namespace {

constexpr int kMaxStages = 8;
constexpr int kChainThreads = 352;          // A producer, MMA warp, 8 epilogue warps, B producer
constexpr uint32_t kTileBytes = 16384;      // 128 rows x 64 bf16
constexpr int kAccBufs = 4;                 // at most 4 x 128 TMEM columns of phase-2 accumulators
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


__device__ __forceinline__ uint4 pack8(const uint32_t* v) {
    uint4 o;
    o.x = pack_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
    o.y = pack_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
    o.z = pack_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
    o.w = pack_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
    return o;
}

__device__ __forceinline__ uint32_t relu_bf16x2(uint32_t w) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(w), "r"(0u));
    return r;
}

// Position in the cycle of phase-2 accumulators: buffer index and its phase bit.
struct AccPos {
    uint32_t b = 0, ph = 0;
    __device__ __forceinline__ void advance(uint32_t nb) {
        if (++b == nb) { b = 0; ph ^= 1u; }
    }
};

// Ring position: stage index, its byte offset and the phase bit, advanced without divisions.
struct RingPos {
    uint32_t s = 0, off = 0, ph = 0;
    __device__ __forceinline__ void advance(uint32_t ns, uint32_t stage_bytes) {
        if (++s == ns) { s = 0; off = 0; ph ^= 1u; } else { off += stage_bytes; }
    }
};

// kMulti: a CTA may own several row tiles (persistent grid); otherwise exactly the tile blockIdx.x, and
// the loops over tiles below fold away at compile time.
// kEpi: the output epilogue adds a bias row and applies the activation (see ChainParams).
template <bool kMulti, bool kEpi = false>
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
    const int tile0 = blockIdx.x, tile_step = gridDim.x;
    const int nt_total = (p.N2 + 127) / 128;
    const int t_beg = blockIdx.y * p.tiles_per_split;
    const int ntile = max(0, min(nt_total, t_beg + p.tiles_per_split) - t_beg);
    const int nkb1 = (p.K1 + 63) / 64;
    const int nkb2 = p.r_pad / 64;
    const uint32_t NS = static_cast<uint32_t>(p.num_stages);
    const uint32_t S = static_cast<uint32_t>(p.stage_bytes);
    const int bps = p.boxes_per_stage;
    const uint32_t NB = kMulti ? static_cast<uint32_t>(p.acc_bufs) : static_cast<uint32_t>(kAccBufs);
    const uint32_t acc_col0 = kMulti ? static_cast<uint32_t>(p.acc_base) : 0u;

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
            for (int kb = 0; kb < kEarlyTiles && kb < nkb1; ++kb) tma_prefetch_l2_2d(&tmA, kb * 64, tile0 * p.rows_tile);
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
            const int skip = ntile * ((nkb2 + bps - 1) / bps);      // stages of a tile's phase 2 (B2 only)
            bool ok = true;
            int tile = tile0;
            do {
                const int m0 = tile * p.rows_tile;
                // convolution: (tap row, tap column, channel block) advance as counters; integer divisions
                // in the loop over k-blocks would sit on the producer's critical path
                const int cv_img = p.conv_cblks > 0 ? tile / p.conv_tiles_per_img : 0;
                const int cv_h0 = (tile - cv_img * p.conv_tiles_per_img) * p.conv_box_h - p.conv_pad;
                int cv_cb = 0, cv_ta = 0, cv_tb = 0;
                for (int kb = 0; kb < nkb1; ++kb) {
                    ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
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
                // the B producer fills the tile's phase-2 stages alone; this thread still takes each of
                // them in turn (waits, loads nothing), so that it never runs more than one lap ahead
                if constexpr (!kMulti) {
                    break;
                } else {
                    for (int i = 0; i < skip && ok; ++i) {
                        ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                        rp.advance(NS, S);
                    }
                    tile += tile_step;
                }
            } while (ok && tile < p.row_tiles);
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
            int tile = tile0;
            do {
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
                if (!kMulti) break;
                tile += tile_step;
            } while (ok && tile < p.row_tiles);
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
            const uint32_t idesc2 = make_idesc_bf16(128, 128, 0, 0);
            const uint64_t t_desc = make_smem_desc(t_smem, 16, 1024);
            const uint32_t accf0 = smem_u32(&ctl->acc_full[0]), acce0 = smem_u32(&ctl->acc_empty[0]);
            const uint32_t acc_tmem = tmem + acc_col0;
            AccPos ap;
            uint32_t it = 0;              // tiles done by this CTA: parity of t_full / t_ready
            bool stash_pending = false;
            int tile = tile0;
            do {
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
                if (!ok) break;
                // the epilogue warps overwrite T in shared memory once t_full fires: the previous tile's
                // stash store must have read it (its phase-2 MMAs are complete by then, being older)
                if (kMulti && stash_pending) { tma_store_wait_read<0>(); stash_pending = false; }
                tc_commit(smem_u32(&ctl->t_full));
                ok = mbar_wait(smem_u32(&ctl->t_ready), it & 1u, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                if (p.store_T && blockIdx.y == 0) {
                    for (int q = 0; q < nkb2; ++q) {
                        if (p.conv_cblks > 0) tma_store_3d(&tmT, t_smem + q * kTileBytes, q * 64, 0, tile);
                        else tma_store_2d(&tmT, t_smem + q * kTileBytes, q * 64, tile * p.rows_tile);
                    }
                    tma_store_commit();
                    stash_pending = true;
                }
                for (int j = 0; j < ntile && ok; ++j) {
                    ok = mbar_wait(acce0 + 8 * ap.b, ap.ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = acc_tmem + ap.b * 128;
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
                    if (ok) tc_commit(accf0 + 8 * ap.b);
                    ap.advance(NB);
                }
                if (!kMulti) break;
                tile += tile_step;
                ++it;
            } while (ok && tile < p.row_tiles);
            if (stash_pending) tma_store_wait_read<0>();
        }
    } else if (warp < 10) {
        // ------------------------------------------------------------------ epilogue warps
        // Eight warps: warp w may touch the TMEM lanes of quadrant w % 4, so two warps share each
        // 32-row quadrant and split the columns (64 of every 128) between them.
        const int q = warp & 3;
        const int hcol = (warp - 2) >> 2;            // 0 or 1: which 64-column half of a tile
        const int row = q * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(q * 32) << 16);
        const uint32_t acc_base = lane_base + acc_col0;
        const uint32_t sw = static_cast<uint32_t>(lane & 7);      // == row & 7
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
        const uint32_t prow = stg + lane * 128;
        bool stored = false, ok = true;
        AccPos ap;
        uint32_t it = 0;
        int tile = tile0;
        do {
            ok = mbar_wait_warp(smem_u32(&ctl->t_full), it & 1u, abort_flag, p.status);
            tc_fence_after();
            if (!ok) break;
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
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->t_ready));

            const int r0 = tile * p.rows_tile + q * 32;
            for (int j = 0; j < ntile; ++j) {
                // kEpi: the bias of this warp's 64 columns, as 32 bf16 pairs per thread (every lane loads the
                // same addresses: one broadcast transaction per load), fetched before the accumulator arrives
                uint32_t bw[kEpi ? 32 : 1];
                if constexpr (kEpi) {
                    const int cb = (t_beg + j) * 128 + hcol * 64;
                    const unsigned short* bp = reinterpret_cast<const unsigned short*>(p.bias);
                    if (bp && cb + 64 <= p.N2 && (reinterpret_cast<uintptr_t>(bp) & 15) == 0) {
                        const uint4* b4 = reinterpret_cast<const uint4*>(bp + cb);
#pragma unroll
                        for (int t = 0; t < 8; ++t) {
                            const uint4 w = __ldg(b4 + t);
                            bw[4 * t] = w.x; bw[4 * t + 1] = w.y; bw[4 * t + 2] = w.z; bw[4 * t + 3] = w.w;
                        }
                    } else {
#pragma unroll
                        for (int t = 0; t < 32; ++t) {
                            const int c = cb + 2 * t;
                            const uint32_t lo = (bp && c < p.N2) ? bp[c] : 0u, hi = (bp && c + 1 < p.N2) ? bp[c + 1] : 0u;
                            bw[t] = lo | (hi << 16);
                        }
                    }
                }
                ok = mbar_wait_warp(smem_u32(&ctl->acc_full[ap.b]), ap.ph, abort_flag, p.status);
                tc_fence_after();
                if (!ok) break;
                // drain this warp's 64 columns and hand the TMEM buffer back before converting
                uint32_t v[2][32];
                tmem_ld32(acc_base + ap.b * 128 + hcol * 64, v[0]);
                tmem_ld32(acc_base + ap.b * 128 + hcol * 64 + 32, v[1]);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&ctl->acc_empty[ap.b]));
                    tma_store_wait_read<0>();             // the previous store has finished reading the panel
                }
                __syncwarp();
                ap.advance(NB);
                if constexpr (kEpi) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) {
                        const float b = __uint_as_float((c & 1) ? (bw[c >> 1] & 0xffff0000u) : (bw[c >> 1] << 16));
                        v[c >> 5][c & 31] = __float_as_uint(__uint_as_float(v[c >> 5][c & 31]) + b);
                    }
                }
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    uint4 o = pack8(v[t >> 2] + 8 * (t & 3));
                    if constexpr (kEpi) {
                        // max(0, .) commutes with the (monotonic) rounding, so it is taken on the rounded pairs
                        if (p.act == 1) { o.x = relu_bf16x2(o.x); o.y = relu_bf16x2(o.y); o.z = relu_bf16x2(o.z); o.w = relu_bf16x2(o.w); }
                    }
                    st_shared_v4(prow + ((static_cast<uint32_t>(t) ^ sw) << 4), o);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int n0 = (t_beg + j) * 128 + hcol * 64;
                    if (r0 < p.M && q * 32 < p.rows_tile && n0 < p.N2) {
                        if (p.conv_cblks > 0) tma_store_3d(&tmOut, stg, n0, q * 32, tile);
                        else tma_store_2d(&tmOut, stg, n0, r0);
                        tma_store_commit();
                        stored = true;
                    }
                }
            }
            if (!kMulti) break;
            tile += tile_step;
            ++it;
        } while (ok && tile < p.row_tiles);
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

// Launch of the forms with the bias / activation epilogue (pf_tc_chain_act.cu).
int chain_launch_act(bool persistent, dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta,
                     const CUtensorMap& tb1, const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt,
                     const ChainParams& p);
// Launch of the software-pipelined persistent form (pf_tc_chain_pipe.cuh, compiled in pf_tc_chain_multi.cu).
int chain_launch_pipe(dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta, const CUtensorMap& tb1,
                      const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt, const ChainParams& p);
// Launch of the persistent form (pf_tc_chain_multi.cu); same arguments as the kernel.
int chain_launch_multi(dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta, const CUtensorMap& tb1,
                       const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt, const ChainParams& p);

}  // namespace tc
}  // namespace pf
#endif
