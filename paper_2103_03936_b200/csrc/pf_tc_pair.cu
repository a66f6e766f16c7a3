// Plain GEMM C[M,N] = A * B on CTA pairs (tcgen05 cta_group::2) for the tensor-bound products of
// the factorized layers (large ranks, where the layer runs as unfused products).
//
// Two CTAs of a cluster compute one 256 x 256 output tile with MMAs of shape 256 x 256 x 16 that
// span both SMs: CTA `rank` holds rows [128 rank, 128 rank + 128) of the A tile and columns
// [128 rank, 128 rank + 128) of the B tile in its shared memory and receives rows
// [128 rank, +128) x all 256 columns of the accumulator in its tensor memory.  Per k-block each
// CTA therefore loads 16 KB of A and 16 KB of B for 128 x 256 outputs: 64 bytes per clock of
// tensor time instead of the 96 a single CTA needs for the same tile, which is more than the
// load path of one SM delivers.
//
// Protocol (rank 0 = leader, issues every MMA):
//   full[s]      leader's barrier; the leader's two producer threads arrive with the byte count of
//                BOTH CTAs' loads of their operand; every TMA load of either CTA completes on it
//   empty[s]     one per CTA; the leader's tcgen05.commit arrives on both (multicast), releasing the
//                stage to the producers of both CTAs
//   acc_full[b]  one per CTA and accumulator buffer, same multicast: buffer b of both CTAs is complete
//   acc_empty[b] leader's barrier; the eight epilogue warps of BOTH CTAs arrive on it once they have
//                read buffer b out of tensor memory
// The kernel is persistent: a pair walks over output tiles (pair index, pair index + number of
// pairs, ...) with two accumulator buffers of 256 columns, so the epilogue of one tile (and the
// pipeline fill of the next) overlaps the MMAs of the other buffer; the products it serves have a
// short contraction (K = r), where a tile's epilogue and start-up cost as much as its main loop.
// Every wait is bounded; the two CTAs meet at a cluster barrier after set-up (the partner's
// barriers and tensor memory exist before anything refers to them) and before they leave.
#include <cuda.h>

#include <algorithm>

#include "pf_tc.h"
#include "pf_tc_host.h"
#include "pf_tc_prims.cuh"

namespace pf {
namespace tc {
namespace {

constexpr int kPairThreads = 352;   // A producer, MMA issue, 8 epilogue warps, B producer
constexpr int kPairStages = 6;
constexpr uint32_t kHalfBytes = 16384;          // 128 rows x 64 bf16
constexpr uint32_t kPairStageBytes = 2 * kHalfBytes;
constexpr uint32_t kPairCols = 256;             // fp32 accumulator columns per CTA and buffer
constexpr uint32_t kPairStaging = 32768;        // 8 epilogue warps x 4 KB store panels

struct PairCtl {
    uint64_t full[kPairStages];
    uint64_t empty[kPairStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort;
};

struct PairParams {
    int M, N, K;
    int a_mn, b_mn;          // 1 = operand stored with the M/N index contiguous
    void* C;                 // bf16 [M, ldc], 16-byte aligned, ldc a multiple of 8
    long long ldc;
    int tiles_m, tiles;      // 256-row tile rows, and all 256 x 256 tiles (tile t = (t % tiles_m, t / tiles_m))
    unsigned int* status;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t cluster_addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}
// Arrive on an mbarrier that may live in the partner CTA (cluster-scope release).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Bounded wait (see mbar_wait) on a barrier that threads of the partner CTA arrive on.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        " selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  unsigned int* status) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
#pragma unroll 1
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycleLimit) break;
        }
    }
    *abort_flag = 1u;
    if (status) atomicExch(status, kStatusTimeout);
    return false;
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t ncols) {  // whole warp, both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {  // whole warp, both CTAs
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Tile load whose completion is counted on a barrier that may live in the partner CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c0,
                                                 int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1)
        : "memory");
}
// D[tmem of both CTAs] (+)= A * B over the CTA pair.
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs once the MMAs issued so far are done.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(static_cast<uint16_t>(3))
        : "memory");
}

__global__ void __launch_bounds__(kPairThreads, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const PairParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem);
    uint8_t* staging = smem + 1024;
    uint8_t* tiles = smem + 1024 + kPairStaging;
    volatile uint32_t* abort_flag = &ctl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = static_cast<int>(blockIdx.x) >> 1, npairs = static_cast<int>(gridDim.x) >> 1;
    const int nkb = (p.K + 63) / 64;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2);     // the leader's two producer threads
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), 16);  // eight epilogue warps of each CTA
        }
        ctl->abort = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&ctl->tmem_base), 2 * kPairCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    cluster_sync_all();
    pdl_wait();
    pdl_launch_dependents();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0 || warp == 10) {
        if (elect_one()) {
            // ------------------------------------------------------------ producers (A: warp 0, B: warp 10)
            const bool do_a = warp == 0;
            const uint32_t full_leader0 = map_to_cta(smem_u32(&ctl->full[0]), 0);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int t = pair; t < p.tiles && ok; t += npairs) {
                const int tn = t / p.tiles_m, tm = t - tn * p.tiles_m;
                const int m0 = tm * 256 + static_cast<int>(rank) * 128;      // this CTA's rows of A
                const int nb0 = tn * 256 + static_cast<int>(rank) * 128;     // this CTA's part of B
                for (int i = 0; i < nkb; ++i) {
                    ok = mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    if (rank == 0) mbar_expect_tx(smem_u32(&ctl->full[s]), 2 * kHalfBytes);   // both CTAs' tiles of this operand
                    const uint32_t bar = full_leader0 + 8 * s;
                    const uint32_t a_dst = smem_u32(tiles + s * kPairStageBytes);
                    const uint32_t b_dst = a_dst + kHalfBytes;
                    const int k0 = i * 64;
                    if (do_a) {
                        if (p.a_mn) {
                            tma_load_2d_pair(a_dst, &tmA, bar, m0, k0);
                            tma_load_2d_pair(a_dst + 8192, &tmA, bar, m0 + 64, k0);
                        } else {
                            tma_load_2d_pair(a_dst, &tmA, bar, k0, m0);
                        }
                    } else if (p.b_mn) {
                        tma_load_2d_pair(b_dst, &tmB, bar, nb0, k0);
                        tma_load_2d_pair(b_dst + 8192, &tmB, bar, nb0 + 64, k0);
                    } else {
                        tma_load_2d_pair(b_dst, &tmB, bar, k0, nb0);
                    }
                    if (++s == kPairStages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && elect_one()) {
            // ------------------------------------------------------------ MMA issue (leader only)
            bool ok = true;
            // both CTAs must have been given the same tensor-memory columns
            if (ld_cluster_u32(map_to_cta(smem_u32(&ctl->tmem_base), 1)) != tmem_base) {
                *abort_flag = 1u;
                if (p.status) atomicExch(p.status, kStatusTimeout);
                ok = false;
            }
            const uint32_t idesc = make_idesc_bf16(256, 256, p.a_mn, p.b_mn);
            const uint32_t a_step = p.a_mn ? 128u : 2u, b_step = p.b_mn ? 128u : 2u;   // in 16-byte units
            uint32_t s = 0, ph = 0;
            uint32_t j = 0;
            for (int t = pair; t < p.tiles && ok; t += npairs, ++j) {
                const uint32_t buf = j & 1u;
                ok = mbar_wait_cluster(smem_u32(&ctl->acc_empty[buf]), ((j >> 1) & 1u) ^ 1u, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kPairCols;
                for (int i = 0; i < nkb; ++i) {
                    ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(tiles + s * kPairStageBytes);
                    const uint32_t b_addr = a_addr + kHalfBytes;
                    const uint64_t a_desc = p.a_mn ? make_smem_desc(a_addr, 8192, 1024) : make_smem_desc(a_addr, 16, 1024);
                    const uint64_t b_desc = p.b_mn ? make_smem_desc(b_addr, 8192, 1024) : make_smem_desc(b_addr, 16, 1024);
                    tc_mma_bf16_pair(d_tmem, a_desc, b_desc, idesc, i > 0 ? 1u : 0u);
                    tc_mma_bf16_pair(d_tmem, a_desc + a_step, b_desc + b_step, idesc, 1u);
                    tc_mma_bf16_pair(d_tmem, a_desc + 2 * a_step, b_desc + 2 * b_step, idesc, 1u);
                    tc_mma_bf16_pair(d_tmem, a_desc + 3 * a_step, b_desc + 3 * b_step, idesc, 1u);
                    tc_commit_pair(smem_u32(&ctl->empty[s]));
                    if (++s == kPairStages) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit_pair(smem_u32(&ctl->acc_full[buf]));
            }
        }
    } else if (warp < 10) {
        // ---------------------------------------------------------------- epilogue (both CTAs, own rows)
        // eight warps: two per TMEM lane quadrant, each draining two of the four 64-column chunks (with
        // a short contraction the epilogue of a tile takes as long as its MMAs)
        const int q = warp & 3;
        const int c_beg = ((warp - 2) >> 2) * 2;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        __nv_bfloat16* Cb = reinterpret_cast<__nv_bfloat16*>(p.C);
        // 32 rows x 64 columns staged per warp (128 bytes per row, 16-byte pieces XOR-swizzled by
        // the row), then four whole 128-byte row segments per store instruction
        const uint32_t panel = smem_u32(staging) + static_cast<uint32_t>(warp - 2) * 4096u;
        const uint32_t own = panel + static_cast<uint32_t>(lane) * 128u, sw = static_cast<uint32_t>(lane & 7);
        const int sub = lane >> 3, piece = lane & 7;
        const size_t row_step = static_cast<size_t>(4) * p.ldc;
        const uint32_t acc_empty_leader0 = map_to_cta(smem_u32(&ctl->acc_empty[0]), 0);
        uint32_t j = 0;
        for (int t = pair; t < p.tiles; t += npairs, ++j) {
            const uint32_t buf = j & 1u;
            const int tn = t / p.tiles_m, tm = t - tn * p.tiles_m;
            const int m0 = tm * 256 + static_cast<int>(rank) * 128, n0 = tn * 256;
            if (!mbar_wait_warp(smem_u32(&ctl->acc_full[buf]), (j >> 1) & 1u, abort_flag, p.status)) break;
            tc_fence_after();
#pragma unroll 1
            for (int c = c_beg; c < c_beg + 2; ++c) {
                uint32_t v0[32], v1[32];
                tmem_ld32(lane_base + buf * kPairCols + c * 64, v0);
                tmem_ld32(lane_base + buf * kPairCols + c * 64 + 32, v1);
                tmem_ld_wait();
                if (c == c_beg + 1) {
                    // this warp has read its part of the buffer: hand it back to the leader's MMA thread
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_leader0 + 8 * buf);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    uint4 o;
                    o.x = pack_bf16x2(__uint_as_float(v0[8 * u + 0]), __uint_as_float(v0[8 * u + 1]));
                    o.y = pack_bf16x2(__uint_as_float(v0[8 * u + 2]), __uint_as_float(v0[8 * u + 3]));
                    o.z = pack_bf16x2(__uint_as_float(v0[8 * u + 4]), __uint_as_float(v0[8 * u + 5]));
                    o.w = pack_bf16x2(__uint_as_float(v0[8 * u + 6]), __uint_as_float(v0[8 * u + 7]));
                    st_shared_v4(own + ((static_cast<uint32_t>(u) ^ sw) << 4), o);
                    o.x = pack_bf16x2(__uint_as_float(v1[8 * u + 0]), __uint_as_float(v1[8 * u + 1]));
                    o.y = pack_bf16x2(__uint_as_float(v1[8 * u + 2]), __uint_as_float(v1[8 * u + 3]));
                    o.z = pack_bf16x2(__uint_as_float(v1[8 * u + 4]), __uint_as_float(v1[8 * u + 5]));
                    o.w = pack_bf16x2(__uint_as_float(v1[8 * u + 6]), __uint_as_float(v1[8 * u + 7]));
                    st_shared_v4(own + ((static_cast<uint32_t>(4 + u) ^ sw) << 4), o);
                }
                __syncwarp();
                const int col = n0 + c * 64 + piece * 8;
                const int rin0 = q * 32 + sub;
                __nv_bfloat16* dst = Cb + static_cast<size_t>(m0 + rin0) * p.ldc + col;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + sub;
                    const uint4 w = ld_shared_v4(panel + static_cast<uint32_t>(rr) * 128u +
                                                 ((static_cast<uint32_t>(piece) ^ static_cast<uint32_t>(rr & 7)) << 4));
                    if (m0 + rin0 + i * 4 < p.M) {
                        if (col + 8 <= p.N) {
                            *reinterpret_cast<uint4*>(dst) = w;
                        } else {
                            const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (col + e < p.N)
                                    dst[e] = __ushort_as_bfloat16(static_cast<unsigned short>((ws[e >> 1] >> ((e & 1) * 16)) & 0xffffu));
                        }
                    }
                    dst += row_step;
                }
                __syncwarp();
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // neither CTA leaves (or frees tensor memory) while the other may still signal it
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc_pair(tmem_base, 2 * kPairCols);
    }
}

}  // namespace

// C[M,N] (bf16, 16-byte aligned, ldc % 8 == 0) = A * B on CTA pairs.  Returns PF_ERR_UNSUPPORTED when
// the operands do not fit (the caller then uses the single-CTA kernel).
int gemm_pair_2sm(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb, bool b_mn, int64_t M, int64_t N,
                  int64_t K, void* C, int64_t ldc, cudaStream_t stream) {
    if (M < 1 || N < 1 || K < 1 || M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return PF_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(C) & 15) != 0 || ldc % 8 != 0) return PF_ERR_UNSUPPORTED;
    const int64_t tiles_m = ceil_div(M, 256), tiles_n = ceil_div(N, 256);
    if (tiles_m * tiles_n > 0x7fffffff) return PF_ERR_UNSUPPORTED;
    const int64_t pairs = std::min<int64_t>(tiles_m * tiles_n, num_sms() / 2);   // persistent: one CTA per SM
    CUtensorMap ta, tb;
    const bool oka = a_mn ? cached_map_2d(&ta, A, K, M, lda, 64) : cached_map_2d(&ta, A, M, K, lda, 128);
    const bool okb = b_mn ? cached_map_2d(&tb, B, K, N, ldb, 64) : cached_map_2d(&tb, B, N, K, ldb, 128);
    if (!oka || !okb) return PF_ERR_CUDA;
    PairParams p;
    p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
    p.a_mn = a_mn; p.b_mn = b_mn; p.C = C; p.ldc = ldc; p.status = device_status_ptr();
    p.tiles_m = static_cast<int>(tiles_m); p.tiles = static_cast<int>(tiles_m * tiles_n);
    const size_t smem = 1024 + 1024 + kPairStaging + static_cast<size_t>(kPairStages) * kPairStageBytes;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
            cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(pairs * 2), 1, 1);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, tc_gemm_pair_kernel, ta, tb, p) != cudaSuccess) return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

}  // namespace tc
}  // namespace pf
