// The persistent fused chain with its two products software-pipelined across row tiles (r <= 128).
//
// A CTA walks over row tiles t = 0, 1, ... (tile index blockIdx.x + t * gridDim.x).  In the plain
// persistent form the MMA thread waits, between the first product of tile t and the first product of
// tile t + 1, until the epilogue warps have moved T(t) from tensor memory to shared memory; the ring is
// full meanwhile and the SM's load path idles.  Here the order of issue is
//     P1(0) | P1(1) P2(0) | P1(2) P2(1) | ... | P2(last)
// (P1 = first product, into one of TWO T accumulators; P2 = second product of the tile before, reading
// one of TWO T buffers in shared memory), so the first products follow each other without a gap and the
// conversion of T(t) has the whole of P1(t+1) to finish.  The ring carries the stages in that order.
// Tensor memory: 2 x r_pad columns of T accumulators, then the output accumulators (3 x 128 columns for
// r_pad = 64, 2 x 128 for r_pad = 128).  Shared memory: control | T buffer 0 | T buffer 1 | ring | staging.
// Barriers as in pf_tc_chain_kernel.cuh, with t_full / t_ready per T buffer.  Every wait is bounded.
#ifndef PF_TC_CHAIN_PIPE_CUH_
#define PF_TC_CHAIN_PIPE_CUH_

#include "pf_tc_chain_kernel.cuh"

namespace pf {
namespace tc {
namespace {

struct PipeCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t t_full[2];
    uint64_t t_ready[2];
    uint64_t acc_full[kAccBufs];
    uint64_t acc_empty[kAccBufs];
    uint32_t tmem_base;
    uint32_t abort;
};

__global__ void __launch_bounds__(kChainThreads, 1)
tc_chain_pipe_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB1,
                     const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmOut,
                     const __grid_constant__ CUtensorMap tmT, const ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    PipeCtl* ctl = reinterpret_cast<PipeCtl*>(smem);
    const uint32_t t_bytes = static_cast<uint32_t>(p.r_pad) * 256u;
    const uint32_t t_smem0 = smem_u32(smem + 1024);
    const uint32_t ring = t_smem0 + 2u * t_bytes;
    volatile uint32_t* abort_flag = &ctl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile0 = blockIdx.x, tile_step = gridDim.x;
    const int nt = tile0 < p.row_tiles ? (p.row_tiles - tile0 + tile_step - 1) / tile_step : 0;   // tiles of this CTA
    const int ntile = min((p.N2 + 127) / 128, p.tiles_per_split);      // output column tiles (one split only)
    const int nkb1 = (p.K1 + 63) / 64;
    const int nkb2 = p.r_pad / 64;
    const uint32_t NS = static_cast<uint32_t>(p.num_stages);
    const uint32_t S = static_cast<uint32_t>(p.stage_bytes);
    const uint32_t NB = static_cast<uint32_t>(p.acc_bufs);
    const uint32_t acc_col0 = static_cast<uint32_t>(p.acc_base);

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->t_full[b]), 1);
            mbar_init(smem_u32(&ctl->t_ready[b]), 8);
        }
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
    pdl_wait();
    pdl_launch_dependents();
    const uint32_t tmem = ctl->tmem_base;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);

    if (warp == 0) {
        if (elect_one()) {
            // ---------------------------------------------------------- producer of A
            RingPos rp;
            const uint32_t txa = static_cast<uint32_t>(p.rows_tile) * 128u;
            bool ok = true;
            // ring order: P1(0), then per t: P1(t+1) (if any), P2(t).  The P2 stages are taken without loading.
            for (int t = 0; t <= nt && ok; ++t) {
                if (t < nt) {
                    const int tile = tile0 + t * tile_step;
                    const int m0 = tile * p.rows_tile;
                    const int cv_img = p.conv_cblks > 0 ? tile / p.conv_tiles_per_img : 0;
                    const int cv_h0 = (tile - cv_img * p.conv_tiles_per_img) * p.conv_box_h - p.conv_pad;
                    int cv_cb = 0, cv_ta = 0, cv_tb = 0;
                    for (int kb = 0; kb < nkb1; ++kb) {
                        ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t full = full0 + 8 * rp.s;
                        mbar_expect_tx(full, txa);
                        if (p.conv_cblks > 0) {
                            tma_load_4d(ring + rp.off, &tmA, full, cv_cb * 64, cv_tb - p.conv_pad, cv_h0 + cv_ta, cv_img);
                            if (++cv_cb == p.conv_cblks) {
                                cv_cb = 0;
                                if (++cv_tb == p.conv_kw) { cv_tb = 0; ++cv_ta; }
                            }
                        } else {
                            tma_load_2d(ring + rp.off, &tmA, full, kb * 64, m0);
                        }
                        rp.advance(NS, S);
                    }
                }
                if (t >= 1) {
                    for (int j = 0; j < ntile && ok; ++j) {
                        ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                        rp.advance(NS, S);
                    }
                }
            }
        }
    } else if (warp == 10) {
        if (elect_one()) {
            // ---------------------------------------------------------- producer of B1 and B2
            RingPos rp;
            bool ok = true;
            const uint32_t txb = static_cast<uint32_t>(p.r_pad) * 128u;
            for (int t = 0; t <= nt && ok; ++t) {
                if (t < nt) {
                    for (int kb = 0; kb < nkb1; ++kb) {
                        ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t full = full0 + 8 * rp.s;
                        const uint32_t dst = ring + rp.off + kTileBytes;
                        mbar_expect_tx(full, txb);
                        for (int q = 0; q < nkb2; ++q) tma_load_2d(dst + q * 8192, &tmB1, full, q * 64, kb * 64);
                        rp.advance(NS, S);
                    }
                }
                if (t >= 1) {
                    for (int j = 0; j < ntile && ok; ++j) {
                        ok = mbar_wait(empty0 + 8 * rp.s, rp.ph ^ 1u, abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t full = full0 + 8 * rp.s;
                        mbar_arrive(full);                      // stands in for the A producer
                        mbar_expect_tx(full, kTileBytes * nkb2);
                        for (int q = 0; q < nkb2; ++q)
                            tma_load_2d(ring + rp.off + q * kTileBytes, &tmB2, full, q * 64, j * 128);
                        rp.advance(NS, S);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            // ---------------------------------------------------------- MMA issuer
            RingPos rp;
            AccPos ap;
            bool ok = true;
            const uint32_t idesc1 = make_idesc_bf16(128, p.r_pad, 0, 1);
            const uint32_t idesc2 = make_idesc_bf16(128, 128, 0, 0);
            const uint64_t a_ring = make_smem_desc(ring, 16, 1024);
            const uint64_t b1_ring = make_smem_desc(ring + kTileBytes, 8192, 1024);
            const uint32_t accf0 = smem_u32(&ctl->acc_full[0]), acce0 = smem_u32(&ctl->acc_empty[0]);
            bool stash_pending = false;
            for (int t = 0; t <= nt && ok; ++t) {
                if (t < nt) {
                    // P1(t) into T accumulator t & 1 (drained of tile t - 2: this thread waited for t_ready(t - 2))
                    const uint32_t d_t = tmem + static_cast<uint32_t>(t & 1) * static_cast<uint32_t>(p.r_pad);
                    for (int kb = 0; kb < nkb1; ++kb) {
                        ok = mbar_wait(full0 + 8 * rp.s, rp.ph, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t a_desc = a_ring + (rp.off >> 4), b_desc = b1_ring + (rp.off >> 4);
                        tc_mma_bf16(d_t, a_desc, b_desc, idesc1, kb > 0 ? 1u : 0u);
                        tc_mma_bf16(d_t, a_desc + 2, b_desc + 128, idesc1, 1u);
                        tc_mma_bf16(d_t, a_desc + 4, b_desc + 256, idesc1, 1u);
                        tc_mma_bf16(d_t, a_desc + 6, b_desc + 384, idesc1, 1u);
                        tc_commit(empty0 + 8 * rp.s);
                        rp.advance(NS, S);
                    }
                    if (!ok) break;
                    // T buffer t & 1 in shared memory is rewritten once t_full fires: the stash store of tile
                    // t - 2 must have read it (the second product of t - 2 is complete by then, being older)
                    if (stash_pending) { tma_store_wait_read<0>(); stash_pending = false; }
                    tc_commit(smem_u32(&ctl->t_full[t & 1]));
                }
                if (t >= 1) {
                    const int u = t - 1;                                   // P2(u)
                    ok = mbar_wait(smem_u32(&ctl->t_ready[u & 1]), static_cast<uint32_t>(u >> 1) & 1u, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t t_smem = t_smem0 + static_cast<uint32_t>(u & 1) * t_bytes;
                    const int tile = tile0 + u * tile_step;
                    if (p.store_T) {
                        for (int q = 0; q < nkb2; ++q) {
                            if (p.conv_cblks > 0) tma_store_3d(&tmT, t_smem + q * kTileBytes, q * 64, 0, tile);
                            else tma_store_2d(&tmT, t_smem + q * kTileBytes, q * 64, tile * p.rows_tile);
                        }
                        tma_store_commit();
                        stash_pending = true;
                    }
                    const uint64_t t_desc = make_smem_desc(t_smem, 16, 1024);
                    for (int j = 0; j < ntile && ok; ++j) {
                        ok = mbar_wait(acce0 + 8 * ap.b, ap.ph ^ 1u, abort_flag, p.status);
                        if (!ok) break;
                        ok = mbar_wait(full0 + 8 * rp.s, rp.ph, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t d_tmem = tmem + acc_col0 + ap.b * 128;
                        for (int q = 0; q < nkb2; ++q) {
                            const uint64_t a_desc = t_desc + static_cast<uint32_t>(q * (kTileBytes >> 4));
                            const uint64_t b_desc = a_ring + ((rp.off + q * kTileBytes) >> 4);
                            tc_mma_bf16(d_tmem, a_desc, b_desc, idesc2, q > 0 ? 1u : 0u);
                            tc_mma_bf16(d_tmem, a_desc + 2, b_desc + 2, idesc2, 1u);
                            tc_mma_bf16(d_tmem, a_desc + 4, b_desc + 4, idesc2, 1u);
                            tc_mma_bf16(d_tmem, a_desc + 6, b_desc + 6, idesc2, 1u);
                        }
                        tc_commit(empty0 + 8 * rp.s);
                        tc_commit(accf0 + 8 * ap.b);
                        rp.advance(NS, S);
                        ap.advance(NB);
                    }
                }
            }
            if (stash_pending) tma_store_wait_read<0>();
        }
    } else if (warp < 10) {
        // -------------------------------------------------------------- epilogue warps
        const int q = warp & 3;
        const int hcol = (warp - 2) >> 2;
        const int row = q * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(q * 32) << 16);
        const uint32_t acc_base = lane_base + acc_col0;
        const uint32_t sw = static_cast<uint32_t>(lane & 7);
        const uint32_t stg = smem_u32(smem + p.staging_off) + static_cast<uint32_t>(warp - 2) * 4096u;
        const uint32_t prow = stg + lane * 128;
        bool stored = false, ok = true;
        AccPos ap;
        // per step t: move T(t) to shared memory, then convert and store the outputs of tile t - 1
        for (int t = 0; t <= nt && ok; ++t) {
            if (t < nt) {
                ok = mbar_wait_warp(smem_u32(&ctl->t_full[t & 1]), static_cast<uint32_t>(t >> 1) & 1u, abort_flag, p.status);
                tc_fence_after();
                if (!ok) break;
                const uint32_t t_smem = t_smem0 + static_cast<uint32_t>(t & 1) * t_bytes;
                const uint32_t t_acc = lane_base + static_cast<uint32_t>(t & 1) * static_cast<uint32_t>(p.r_pad);
                for (int c = hcol; c < p.r_pad / 32; c += 2) {
                    uint32_t v[32];
                    tmem_ld32(t_acc + c * 32, v);
                    tmem_ld_wait();
                    const uint32_t panel = t_smem + (c >> 1) * kTileBytes + row * 128;
                    const uint32_t cb = (c & 1) * 4;
#pragma unroll
                    for (int i = 0; i < 4; ++i) st_shared_v4(panel + (((cb + i) ^ sw) << 4), pack8(v + 8 * i));
                }
                tc_fence_before();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->t_ready[t & 1]));
            }
            if (t >= 1) {
                const int tile = tile0 + (t - 1) * tile_step;
                const int r0 = tile * p.rows_tile + q * 32;
                for (int j = 0; j < ntile; ++j) {
                    ok = mbar_wait_warp(smem_u32(&ctl->acc_full[ap.b]), ap.ph, abort_flag, p.status);
                    tc_fence_after();
                    if (!ok) break;
                    uint32_t v[2][32];
                    tmem_ld32(acc_base + ap.b * 128 + hcol * 64, v[0]);
                    tmem_ld32(acc_base + ap.b * 128 + hcol * 64 + 32, v[1]);
                    tmem_ld_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&ctl->acc_empty[ap.b]));
                        tma_store_wait_read<0>();
                    }
                    __syncwarp();
                    ap.advance(NB);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        st_shared_v4(prow + ((static_cast<uint32_t>(i) ^ sw) << 4), pack8(v[i >> 2] + 8 * (i & 3)));
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int n0 = j * 128 + hcol * 64;
                        if (r0 < p.M && q * 32 < p.rows_tile && n0 < p.N2) {
                            if (p.conv_cblks > 0) tma_store_3d(&tmOut, stg, n0, q * 32, tile);
                            else tma_store_2d(&tmOut, stg, n0, r0);
                            tma_store_commit();
                            stored = true;
                        }
                    }
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
}  // namespace tc
}  // namespace pf
#endif
