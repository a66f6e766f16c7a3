// Tensor-core path (bf16 storage) for sm_100a: tcgen05 MMAs with accumulators in tensor memory,
// operands staged in shared memory by TMA through an mbarrier pipeline.
//
// Kernel in this file:
//   tc_gemm_kernel<BN>  C[M,N] = A * B for every operand orientation the factorized layers need
//                       (row-major operands read either along or across the contraction index,
//                       i.e. K-major or MN-major shared-memory descriptors), with an optional
//                       reduction split whose fp32 partials are summed in a fixed order.
// Warp roles: warp 0 = TMA producer of operand A, warp 1 = TMEM allocation + MMA issue, warps 2..5 =
// epilogue (each owns the 32 TMEM lanes of its warp-id quadrant), warp 6 = TMA producer of operand B.
#include "pf_tc.h"

#include <cuda.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "pf_tc_host.h"
#include "pf_tc_prims.cuh"

namespace pf {
namespace tc {
namespace {

constexpr int kBM = 128;       // rows of the output tile = TMEM lanes
constexpr int kBK = 64;        // contraction elements per pipeline stage (128 bytes of bf16)
constexpr int kMaxStages = 6;
constexpr int kGemmThreads = 224;   // A producer, MMA issue, 4 epilogue warps, B producer
constexpr int kFixSlots = 32;  // counter sets handed out round-robin to launches that split a contraction
constexpr int kFixTiles = 160; // output tiles of one split product (tiles * slices never exceeds the SM count)

// Arrival / departure counters of the in-kernel slice sum, two per output tile.  They are zero
// between launches: the last CTA to leave a tile clears its pair.
__device__ unsigned int g_fix_counters[kFixSlots][kFixTiles * 2];

struct GemmCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint64_t fix_full;       // the slices this CTA sums have been copied into shared memory
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t fix_ok;
};

struct GemmParams {
    int M, N, K;
    int a_mn, b_mn;          // 1 = operand stored with the M/N index contiguous
    int kb_per_split;        // k-blocks handled by one z-slice
    int splits;
    int num_stages;
    int bn;                  // columns of an output tile (the kernel's template value; 64 or 128 in a shared launch)
    int tiles_x;             // row tiles of this product (tile id = column tile * tiles_x + row tile)
    void* C;                 // bf16 [M, ldc]
    long long ldc;
    void* C2;                // optional second copy of the result at another pitch (split contractions only)
    long long ldc2;
    float* partial;          // splits > 1: fp32 slices, one 128 x BN block per (tile, slice)
    unsigned int* counters;  // splits > 1: two counters per tile
    unsigned int* status;
    // Implicit-GEMM convolution operand A (tmA is then a 4-D NHWC map):
    //   conv_mode 1 (dX): A K-major; row tile = cv_box_h full-width image rows of dT; k-block =
    //                     (tap, 64-rank block), tap offsets flipped; B rows are offset by tap * cv_C.
    //   conv_mode 2 (dU): A MN-major; row tile = (tap, 128-channel block) of the unrolled factor;
    //                     k-block = 64 pixels (cv_box_h full-width rows) of the image x.
    int conv_mode, cv_blks, cv_kw, cv_pad, cv_C, cv_box_h, cv_tpi;
    int rows_tile;           // output rows per CTA: 128, or cv_box_h * W pixels for conv_mode 1
    int kpix;                // conv_mode 2: pixels per k-block (cv_box_h * W <= 64), else 64
    int nkb_total;           // k-blocks of the whole contraction
    int independent;         // 1: reads nothing the preceding kernel of the stream writes (see gemm_tile)
    // Grouped products (several problems of one shape in a launch): tmA / tmB are 3-D maps whose outermost
    // coordinate is the group (a shared operand has one group only), outputs of group g start g * c_gstride
    // elements after C.  kb_per_group > 0 instead makes the group part of the CONTRACTION: k-block kb reads
    // group kb / kb_per_group, 64-element block kb % kb_per_group of both operands (the sum over groups of
    // A_g B_g^T, i.e. dX of several factor pairs that share one input).
    int groups, a_shared, b_shared, kb_per_group, tiles_y;
    long long c_gstride;
};

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// One output tile (128 rows x BN columns) of C = A * B, or one slice of its contraction.
//
// Epilogue.  Unsplit: each epilogue warp turns its 32 accumulator rows into bf16, transposes them
// through a padded shared-memory panel and writes whole 128-byte row segments (any pitch, any
// alignment, clipped at the matrix edge).  Split: the fp32 slice goes to the workspace in the
// order [32-column chunk][4-column group][row][4], which makes every store instruction of a warp
// one contiguous 512-byte run; then the CTAs of a tile meet at a counter and each sums, in slice
// order, its share of the rows over all slices and writes bf16 (bit-reproducible, no second launch).
template <int BN>
__device__ __forceinline__ void gemm_tile(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p,
                                          const int bx, const int by, const int bz, const int bg) {
    constexpr uint32_t kABytes = kBM * kBK * 2;          // 16 KB
    constexpr uint32_t kBBytes = BN * kBK * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    GemmCtl* ctl = reinterpret_cast<GemmCtl*>(smem);
    uint8_t* tiles = smem + 1024;
    volatile uint32_t* abort_flag = &ctl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = bx * p.rows_tile, n0 = by * BN;
    const int nkb_total = p.nkb_total;
    const int kb_beg = bz * p.kb_per_split;
    const int kb_end = min(nkb_total, kb_beg + p.kb_per_split);
    const int nkb = kb_end - kb_beg;
    const uint32_t NS = static_cast<uint32_t>(p.num_stages);
    const int tile = (bg * p.tiles_y + by) * p.tiles_x + bx;
    const bool grouped = p.groups > 1 || p.kb_per_group > 0;

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2);     // one expect_tx arrival per producer thread
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->tmem_full), 1);
        mbar_init(smem_u32(&ctl->fix_full), 1);
        ctl->abort = 0;
        ctl->fix_ok = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (p.conv_mode == 2 && p.kpix < 64) {
        // k-blocks hold fewer than 64 pixels: the unused contraction rows of every A stage must be
        // zero (TMA never writes them), so that they add nothing to the sum
        for (int i = threadIdx.x; i < static_cast<int>(NS) * static_cast<int>(kABytes / 16); i += blockDim.x) {
            const int st = i / static_cast<int>(kABytes / 16), off = i - st * static_cast<int>(kABytes / 16);
            *reinterpret_cast<uint4*>(tiles + st * kStageBytes + off * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // A product marked independent reads nothing that the kernel launched just before it writes, so
    // it does not wait for that kernel: its blocks run beside it on SMs that kernel leaves free.  (Every
    // kernel of this library lets its successor start only after its own wait has returned, i.e. once
    // everything older in the stream is complete, so older results are safe to read.)
    if (!p.independent) pdl_wait();     // everything above overlapped the previous kernel's tail
    pdl_launch_dependents();
    const uint32_t tmem_base = ctl->tmem_base;

    // Producers and MMA issuer are each one thread chosen with elect.sync that runs its whole role
    // (a thread singled out by a lane-id test issues TMA / tcgen05 instructions several times slower).
    // Two producers, one per operand: a producer thread needs about 130 ns per stage for its loop,
    // barrier wait and expect_tx plus 40 ns per TMA instruction, which with four tile loads per
    // stage paced the whole pipeline when one thread issued both operands.
    if (warp == 0 || warp == 6) {
        if (elect_one()) {
            const bool do_a = warp == 0;
            const uint32_t my_bytes = !do_a ? kBBytes
                                      : p.conv_mode == 1 ? static_cast<uint32_t>(p.rows_tile) * 128u
                                      : p.conv_mode == 2 ? static_cast<uint32_t>(p.kpix) * 256u
                                                         : kABytes;
            uint32_t s = 0, ph = 0;
            // convolution operands: tap / block / image positions advance as counters (an integer
            // division per k-block would sit on the producer's critical path)
            int c1_rb = 0, c1_ta = 0, c1_tb = 0, c1_img = 0, c1_h0 = 0;     // conv_mode 1
            int c2_c0 = 0, c2_x = 0, c2_y = 0, c2_img = 0, c2_t = 0;          // conv_mode 2
            if (p.conv_mode == 1) {
                const int tap = kb_beg / p.cv_blks;
                c1_rb = kb_beg - tap * p.cv_blks;
                c1_ta = tap / p.cv_kw;
                c1_tb = tap - c1_ta * p.cv_kw;
                c1_img = bx / p.cv_tpi;
                c1_h0 = (bx - c1_img * p.cv_tpi) * p.cv_box_h + p.cv_pad;
            } else if (p.conv_mode == 2) {
                const int tap = m0 / p.cv_C;
                c2_c0 = m0 - tap * p.cv_C;
                const int ta = tap / p.cv_kw;
                c2_x = tap - ta * p.cv_kw - p.cv_pad;
                c2_y = ta - p.cv_pad;
                c2_img = kb_beg / p.cv_tpi;
                c2_t = kb_beg - c2_img * p.cv_tpi;
            }
            for (int i = 0; i < nkb; ++i) {
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag, p.status)) break;
                const uint32_t full = smem_u32(&ctl->full[s]);
                const uint32_t a_dst = smem_u32(tiles + s * kStageBytes);
                const uint32_t b_dst = a_dst + kABytes;
                mbar_expect_tx(full, my_bytes);
                const int k0 = (kb_beg + i) * kBK;
                if (p.conv_mode == 1) {
                    if (do_a) tma_load_4d(a_dst, &tmA, full, c1_rb * 64, p.cv_pad - c1_tb, c1_h0 - c1_ta, c1_img);
                    else tma_load_2d(b_dst, &tmB, full, c1_rb * 64, (c1_ta * p.cv_kw + c1_tb) * p.cv_C + n0);
                    if (++c1_rb == p.cv_blks) {
                        c1_rb = 0;
                        if (++c1_tb == p.cv_kw) { c1_tb = 0; ++c1_ta; }
                    }
                    if (++s == NS) { s = 0; ph ^= 1u; }
                    continue;
                }
                if (p.conv_mode == 2) {
                    const int hy = c2_t * p.cv_box_h + c2_y;
                    if (do_a) {
                        tma_load_4d(a_dst, &tmA, full, c2_c0, c2_x, hy, c2_img);
                        tma_load_4d(a_dst + 8192, &tmA, full, c2_c0 + 64, c2_x, hy, c2_img);
                    } else {
#pragma unroll
                        for (int h = 0; h < BN / 64; ++h)
                            tma_load_2d(b_dst + h * 8192, &tmB, full, n0 + 64 * h, (kb_beg + i) * p.kpix);
                    }
                    if (++c2_t == p.cv_tpi) { c2_t = 0; ++c2_img; }
                    if (++s == NS) { s = 0; ph ^= 1u; }
                    continue;
                } else if (grouped) {
                    int g = bg, kk0 = k0;
                    if (p.kb_per_group > 0) {
                        g = (kb_beg + i) / p.kb_per_group;
                        kk0 = ((kb_beg + i) - g * p.kb_per_group) * kBK;
                    }
                    if (do_a) {
                        const int ga = p.a_shared ? 0 : g;
                        if (p.a_mn) {
                            tma_load_3d(a_dst, &tmA, full, m0, kk0, ga);
                            tma_load_3d(a_dst + 8192, &tmA, full, m0 + 64, kk0, ga);
                        } else {
                            tma_load_3d(a_dst, &tmA, full, kk0, m0, ga);
                        }
                    } else {
                        const int gb = p.b_shared ? 0 : g;
                        if (p.b_mn) {
#pragma unroll
                            for (int h = 0; h < BN / 64; ++h) tma_load_3d(b_dst + h * 8192, &tmB, full, n0 + 64 * h, kk0, gb);
                        } else {
                            tma_load_3d(b_dst, &tmB, full, kk0, n0, gb);
                        }
                    }
                } else if (do_a) {
                    if (p.a_mn) {
                        tma_load_2d(a_dst, &tmA, full, m0, k0);
                        tma_load_2d(a_dst + 8192, &tmA, full, m0 + 64, k0);
                    } else {
                        tma_load_2d(a_dst, &tmA, full, k0, m0);
                    }
                } else if (p.b_mn) {
#pragma unroll
                    for (int h = 0; h < BN / 64; ++h) tma_load_2d(b_dst + h * 8192, &tmB, full, n0 + 64 * h, k0);
                } else {
                    tma_load_2d(b_dst, &tmB, full, k0, n0);
                }
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            const uint32_t idesc = make_idesc_bf16(kBM, BN, p.a_mn, p.b_mn);
            // K-major: 8-row groups 1024 B apart, 16 contraction elements = 32 B along the row.
            // MN-major: 64-element M/N panels 8192 B apart (LBO), 8 contraction rows per
            // 1024 B group (SBO), 16 contraction rows = 2048 B.
            const uint32_t a_step = p.a_mn ? 128u : 2u, b_step = p.b_mn ? 128u : 2u;   // in 16-byte units
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int i = 0; i < nkb; ++i) {
                ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(tiles + s * kStageBytes);
                const uint32_t b_addr = a_addr + kABytes;
                const uint64_t a_desc = p.a_mn ? make_smem_desc(a_addr, 8192, 1024) : make_smem_desc(a_addr, 16, 1024);
                const uint64_t b_desc = p.b_mn ? make_smem_desc(b_addr, 8192, 1024) : make_smem_desc(b_addr, 16, 1024);
                tc_mma_bf16(tmem_base, a_desc, b_desc, idesc, i > 0 ? 1u : 0u);
                tc_mma_bf16(tmem_base, a_desc + a_step, b_desc + b_step, idesc, 1u);
                tc_mma_bf16(tmem_base, a_desc + 2 * a_step, b_desc + 2 * b_step, idesc, 1u);
                tc_mma_bf16(tmem_base, a_desc + 3 * a_step, b_desc + 3 * b_step, idesc, 1u);
                tc_commit(smem_u32(&ctl->empty[s]));   // frees the stage once these MMAs have read it
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
            if (ok) tc_commit(smem_u32(&ctl->tmem_full));
        }
    } else if (warp < 6) {
        const int q = warp & 3;                          // TMEM lane quadrant this warp may access
        const bool ok = mbar_wait_warp(smem_u32(&ctl->tmem_full), 0, abort_flag, p.status);
        tc_fence_after();
        if (ok) {
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
            if (p.splits > 1) {
                // fp32 slice: this warp's 32 rows go to shared memory as rows of BN floats (the 16-byte
                // pieces of a row XOR-permuted by the row, which keeps the writes and the later reads
                // free of bank conflicts), leave as ONE bulk copy of 32 x BN x 4 bytes to the
                // workspace (the workspace keeps the permuted order; only the sum below reads it),
                // and the warp reports its arrival once the copy has completed
                constexpr uint32_t kRowBytes = BN * 4, kPieces = BN / 4;
                const uint32_t wbase = smem_u32(tiles) + static_cast<uint32_t>(q * 32) * kRowBytes;
                const uint32_t rbase = wbase + static_cast<uint32_t>(lane) * kRowBytes;
                const uint32_t rsw = static_cast<uint32_t>(q * 32 + lane) & (kPieces - 1);
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(lane_base + c * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        st_shared_v4(rbase + (((static_cast<uint32_t>(c * 8 + g)) ^ rsw) << 4),
                                     make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]));
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    uint8_t* dst = reinterpret_cast<uint8_t*>(p.partial) +
                                   (static_cast<size_t>(tile) * p.splits + bz) * (static_cast<size_t>(kBM) * kRowBytes) +
                                   static_cast<size_t>(q * 32) * kRowBytes;
                    bulk_store(dst, wbase, 32u * kRowBytes);
                    tma_store_commit();
                    tma_store_wait_all();          // the rows are in the workspace
                    fence_proxy_async_all();
                    __threadfence();
                    atomicAdd(p.counters + 2 * tile, 1u);
                }
            } else {
                // every MMA has completed, so the pipeline stages are free: 32 x 33-word panel per warp
                uint32_t* stg = reinterpret_cast<uint32_t*>(tiles) + (warp - 2) * (32 * 33);
                __nv_bfloat16* Cb = reinterpret_cast<__nv_bfloat16*>(p.C) + static_cast<long long>(bg) * p.c_gstride;
                const bool pair_ok = (p.ldc % 2) == 0 && (reinterpret_cast<uintptr_t>(Cb) & 3) == 0;
                const bool vec_ok = (p.ldc % 8) == 0 && (reinterpret_cast<uintptr_t>(Cb) & 15) == 0;
                if (vec_ok) {
                    // 16-byte aligned rows: stage 32 rows x 64 columns (128 bytes per row, 16-byte pieces
                    // XOR-swizzled by the row so that both passes are free of bank conflicts), then
                    // store four whole 128-byte row segments per instruction
                    const uint32_t panel = smem_u32(tiles) + static_cast<uint32_t>(warp - 2) * 4096u;
                    const uint32_t own = panel + static_cast<uint32_t>(lane) * 128u, sw = static_cast<uint32_t>(lane & 7);
                    const int sub = lane >> 3, piece = lane & 7;
                    const size_t row_step = static_cast<size_t>(4) * p.ldc;
#pragma unroll 1
                    for (int c = 0; c < BN / 64; ++c) {
                        uint32_t v0[32], v1[32];
                        tmem_ld32(lane_base + c * 64, v0);
                        tmem_ld32(lane_base + c * 64 + 32, v1);
                        tmem_ld_wait();
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(v0[8 * t + 0]), __uint_as_float(v0[8 * t + 1]));
                            o.y = pack_bf16x2(__uint_as_float(v0[8 * t + 2]), __uint_as_float(v0[8 * t + 3]));
                            o.z = pack_bf16x2(__uint_as_float(v0[8 * t + 4]), __uint_as_float(v0[8 * t + 5]));
                            o.w = pack_bf16x2(__uint_as_float(v0[8 * t + 6]), __uint_as_float(v0[8 * t + 7]));
                            st_shared_v4(own + ((static_cast<uint32_t>(t) ^ sw) << 4), o);
                            o.x = pack_bf16x2(__uint_as_float(v1[8 * t + 0]), __uint_as_float(v1[8 * t + 1]));
                            o.y = pack_bf16x2(__uint_as_float(v1[8 * t + 2]), __uint_as_float(v1[8 * t + 3]));
                            o.z = pack_bf16x2(__uint_as_float(v1[8 * t + 4]), __uint_as_float(v1[8 * t + 5]));
                            o.w = pack_bf16x2(__uint_as_float(v1[8 * t + 6]), __uint_as_float(v1[8 * t + 7]));
                            st_shared_v4(own + ((static_cast<uint32_t>(4 + t) ^ sw) << 4), o);
                        }
                        __syncwarp();
                        const int col = n0 + c * 64 + piece * 8;
                        const int rin0 = q * 32 + sub;
                        __nv_bfloat16* dst = Cb + static_cast<size_t>(m0 + rin0) * p.ldc + col;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = i * 4 + sub, rin_i = rin0 + i * 4;
                            const uint4 w = ld_shared_v4(panel + static_cast<uint32_t>(rr) * 128u +
                                                         ((static_cast<uint32_t>(piece) ^ static_cast<uint32_t>(rr & 7)) << 4));
                            if (m0 + rin_i < p.M && rin_i < p.rows_tile) {
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
                } else
#pragma unroll 1
                for (int c = 0; c < BN / 64; ++c) {
                    uint32_t v0[32], v1[32];
                    tmem_ld32(lane_base + c * 64, v0);
                    tmem_ld32(lane_base + c * 64 + 32, v1);
                    tmem_ld_wait();
#pragma unroll
                    for (int w = 0; w < 16; ++w) {
                        stg[lane * 33 + w] = pack_bf16x2(__uint_as_float(v0[2 * w]), __uint_as_float(v0[2 * w + 1]));
                        stg[lane * 33 + 16 + w] = pack_bf16x2(__uint_as_float(v1[2 * w]), __uint_as_float(v1[2 * w + 1]));
                    }
                    __syncwarp();
                    const int col = n0 + c * 64 + 2 * lane;
#pragma unroll 4
                    for (int j = 0; j < 32; ++j) {
                        const int rj = q * 32 + j, rowj = m0 + rj;
                        if (rowj < p.M && rj < p.rows_tile) {
                            const uint32_t w = stg[j * 33 + lane];
                            __nv_bfloat16* dst = Cb + static_cast<size_t>(rowj) * p.ldc + col;
                            if (pair_ok && col + 1 < p.N) {
                                *reinterpret_cast<uint32_t*>(dst) = w;
                            } else {
                                if (col < p.N) dst[0] = __ushort_as_bfloat16(static_cast<unsigned short>(w & 0xffffu));
                                if (col + 1 < p.N) dst[1] = __ushort_as_bfloat16(static_cast<unsigned short>(w >> 16));
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, BN);
    if (p.splits <= 1) return;

    // ---- slice sum: wait until every slice of this tile is in the workspace (four warps of every slice
    // report), then sum a share of it.  A share is a run of whole rows, contiguous in every slice, so
    // one bulk copy per slice brings it into the idle pipeline stages: a single trip to L2 for the
    // whole sum.  The slices are added in slice order (bit-reproducible) and each summed row leaves as
    // whole 8-byte pieces, a warp writing 256 contiguous bytes per instruction.
    unsigned int* cnt = p.counters + 2 * tile;
    const int S = p.splits;
    constexpr uint32_t kRowBytes = BN * 4, kPieces = BN / 4;
    const int rper = (kBM + S - 1) / S;
    const int r_beg = bz * rper;
    const int nr = max(0, min(kBM, r_beg + rper) - r_beg);
    const uint32_t share = static_cast<uint32_t>(nr) * kRowBytes;
    if (threadIdx.x == 0) {
        uint32_t good = (*abort_flag == 0u) ? 1u : 0u;
        if (good) {
            const unsigned int want = 4u * static_cast<unsigned int>(S);
            const long long t0 = clock64();
            while (ld_acquire_gpu(cnt) < want) {
                if (clock64() - t0 > kWaitCycleLimit) {
                    good = 0u;
                    if (p.status) atomicExch(p.status, kStatusTimeout);
                    break;
                }
            }
            __threadfence();
            fence_proxy_async_all();
            if (good && nr > 0) {
                const uint32_t bar = smem_u32(&ctl->fix_full);
                const uint8_t* src = reinterpret_cast<const uint8_t*>(p.partial) +
                                     (static_cast<size_t>(tile) * S) * (static_cast<size_t>(kBM) * kRowBytes) +
                                     static_cast<size_t>(r_beg) * kRowBytes;
                mbar_expect_tx(bar, share * static_cast<uint32_t>(S));
                for (int s = 0; s < S; ++s)
                    bulk_load(smem_u32(tiles) + static_cast<uint32_t>(s) * share,
                              src + static_cast<size_t>(s) * (static_cast<size_t>(kBM) * kRowBytes), share, bar);
                good = mbar_wait(bar, 0, abort_flag, p.status) ? 1u : 0u;
            }
        }
        ctl->fix_ok = good;
    }
    __syncthreads();
    if (ctl->fix_ok) {
        __nv_bfloat16* Cb = reinterpret_cast<__nv_bfloat16*>(p.C) + static_cast<long long>(bg) * p.c_gstride;
        __nv_bfloat16* C2b = reinterpret_cast<__nv_bfloat16*>(p.C2);
        const uint32_t base = smem_u32(tiles);
        const bool vec8 = (p.ldc % 4) == 0 && (reinterpret_cast<uintptr_t>(Cb) & 7) == 0;
        // consecutive threads take consecutive 16-byte pieces of one row
        for (int id = threadIdx.x; id < nr * static_cast<int>(kPieces); id += kGemmThreads) {
            const int rl = id / static_cast<int>(kPieces), pc = id % static_cast<int>(kPieces);
            const int rr = r_beg + rl;
            const uint32_t off = static_cast<uint32_t>(rl) * kRowBytes +
                                 ((static_cast<uint32_t>(pc) ^ (static_cast<uint32_t>(rr) & (kPieces - 1))) << 4);
            uint4 w = ld_shared_v4(base + off);
            float4 acc = make_float4(__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w));
#pragma unroll 4
            for (int s = 1; s < S; ++s) {
                w = ld_shared_v4(base + static_cast<uint32_t>(s) * share + off);
                acc.x += __uint_as_float(w.x); acc.y += __uint_as_float(w.y);
                acc.z += __uint_as_float(w.z); acc.w += __uint_as_float(w.w);
            }
            const int row = m0 + rr, col = n0 + pc * 4;
            if (row < p.M) {
                __nv_bfloat16* dst = Cb + static_cast<size_t>(row) * p.ldc + col;
                if (vec8 && col + 3 < p.N) {
                    *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16x2(acc.x, acc.y), pack_bf16x2(acc.z, acc.w));
                } else {
                    if (col < p.N) dst[0] = __float2bfloat16_rn(acc.x);
                    if (col + 1 < p.N) dst[1] = __float2bfloat16_rn(acc.y);
                    if (col + 2 < p.N) dst[2] = __float2bfloat16_rn(acc.z);
                    if (col + 3 < p.N) dst[3] = __float2bfloat16_rn(acc.w);
                }
                if (C2b) {   // the same sums once more, for a destination whose pitch the first cannot have
                    __nv_bfloat16* d2 = C2b + static_cast<size_t>(row) * p.ldc2 + col;
                    if (col < p.N) d2[0] = __float2bfloat16_rn(acc.x);
                    if (col + 1 < p.N) d2[1] = __float2bfloat16_rn(acc.y);
                    if (col + 2 < p.N) d2[2] = __float2bfloat16_rn(acc.z);
                    if (col + 3 < p.N) d2[3] = __float2bfloat16_rn(acc.w);
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && ctl->fix_ok) {
        const unsigned int left = atomicAdd(cnt + 1, 1u);
        if (left + 1u == static_cast<unsigned int>(S)) {   // every slice has read what it needs
            cnt[0] = 0u;
            cnt[1] = 0u;
            __threadfence();
        }
    }
}

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, BN <= 128 ? 2 : 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const GemmParams p) {
    const int sl = p.splits < 1 ? 1 : p.splits;
    gemm_tile<BN>(tmA, tmB, p, blockIdx.x, blockIdx.y, static_cast<int>(blockIdx.z) % sl, static_cast<int>(blockIdx.z) / sl);
}

// Up to three independent products in one launch (dU = x^T G, dV = dY^T T and, where it is a plain
// product, dX of one layer): CTAs [0, end0) work on product 0, [end0, end1) on product 1, the rest on
// product 2; each decodes (row tile, column tile, slice) from its linear index.  One launch pays the
// start-up latency once and packs the short CTAs of one product beside the long ones of another.
// Tiles may be 64 or 128 columns wide per product.
__device__ __forceinline__ void gemm_any(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p, int idx,
                                         const int2 t) {
    const int sl = p.splits < 1 ? 1 : p.splits;
    const int bx = idx % t.x, by = (idx / t.x) % t.y, zz = idx / (t.x * t.y);
    if (p.bn == 64) gemm_tile<64>(tmA, tmB, p, bx, by, zz % sl, zz / sl);
    else gemm_tile<128>(tmA, tmB, p, bx, by, zz % sl, zz / sl);
}
__global__ void __launch_bounds__(kGemmThreads, 2)
tc_gemm3_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
                const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
                const GemmParams p0, const GemmParams p1, const GemmParams p2, const int end0, const int end1,
                const int2 tiles0, const int2 tiles1, const int2 tiles2) {
    const int idx = blockIdx.x;
    if (idx < end0) gemm_any(tmA0, tmB0, p0, idx, tiles0);
    else if (idx < end1) gemm_any(tmA1, tmB1, p1, idx - end0, tiles1);
    else gemm_any(tmA2, tmB2, p2, idx - end1, tiles2);
}

// ------------------------------------------------------------------------------ host side
// One operand of C = A * B.  `mn_major == false`: stored [MN, K] row-major (contraction index
// contiguous).  `mn_major == true`: stored [K, MN] row-major (M or N index contiguous).
struct Operand {
    const void* p;
    int64_t ld;
    bool mn_major;
    int64_t gs = 0;     // grouped products: elements between the matrices of consecutive groups (0 = one matrix shared by all)
};

// Several problems of one shape in one product.  sum_groups: the groups are summed into ONE output (the
// group index is part of the contraction; both operands K-major), otherwise every group has its own
// output, c_gs elements apart.
struct Grouping {
    int groups = 1;
    int64_t c_gs = 0;
    bool sum_groups = false;
};

// 3-D bf16 tensor map over `groups` row-major [rows, cols] matrices gs elements apart (boxes of 64 columns x
// box_rows rows of one group; out-of-range elements read as zero).  Cached like the 2-D maps.
bool cached_map_3d(CUtensorMap* map, const void* p, int64_t groups, int64_t rows, int64_t cols, int64_t ld, int64_t gs,
                   int box_rows) {
    constexpr int kSlots = 128;
    struct Key { const void* p; int64_t groups, rows, cols, ld, gs; int box_rows; };
    struct Slot { Key key; CUtensorMap map; bool used; };
    static Slot slots[kSlots];
    static std::mutex mu;
    if (groups < 1) return false;
    if (groups == 1) gs = rows * ld;                       // a single group: any valid stride
    if ((gs * 2) % 16 != 0 || gs * 2 >= (1LL << 40)) return false;
    uint64_t h = reinterpret_cast<uintptr_t>(p) * 0x9E3779B97F4A7C15ull;
    h ^= static_cast<uint64_t>(rows) * 0xC2B2AE3D27D4EB4Full + static_cast<uint64_t>(cols) * 0x165667B19E3779F9ull +
         static_cast<uint64_t>(ld) * 31 + static_cast<uint64_t>(box_rows) + static_cast<uint64_t>(gs) * 131 + static_cast<uint64_t>(groups) * 7;
    Slot& sl = slots[(h >> 20) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    const Key& k = sl.key;
    if (sl.used && k.p == p && k.groups == groups && k.rows == rows && k.cols == cols && k.ld == ld && k.gs == gs &&
        k.box_rows == box_rows) {
        *map = sl.map;
        return true;
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(groups)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * 2, static_cast<cuuint64_t>(gs) * 2};
    const cuuint32_t box[3] = {64u, static_cast<cuuint32_t>(box_rows), 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(p), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    sl.key = Key{p, groups, rows, cols, ld, gs, box_rows};
    sl.map = *map;
    sl.used = true;
    return true;
}

size_t gemm_smem(int bn, int stages) {
    return 1024 + 1024 + static_cast<size_t>(stages) * (kBM * kBK * 2 + bn * kBK * 2);
}
// Pipeline depth: a grid that fits one wave gets every stage shared memory has room for; a
// larger grid gets stages small enough for two CTAs per SM, so that the prologue and epilogue of
// one CTA overlap the main loop of the other.
int pick_stages(int bn, int64_t ctas) {
    const size_t stage = static_cast<size_t>(kBM * kBK * 2 + bn * kBK * 2);
    const size_t room = (ctas > num_sms() && bn <= 128) ? (113 * 1024 - 2048) : (200 * 1024 - 2048);
    int ns = static_cast<int>(room / stage);
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns < 2) ns = 2;
    return ns;
}

template <int BN>
cudaError_t launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, dim3 grid,
                        cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(std::min(gemm_smem(BN, kMaxStages), static_cast<size_t>(227 * 1024))));
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaError_t e = launch_overlapped(tc_gemm_kernel<BN>, grid, dim3(kGemmThreads), gemm_smem(BN, p.num_stages), stream,
                                      ta, tb, p);
    if (e == cudaSuccess) count_launch();
    return e;
}

// Device address of the counter set a launch may use (sets rotate, so that launches in flight on
// different streams do not share counters unless more than kFixSlots of them overlap).
unsigned int* next_fix_counters() {
    static unsigned int* base[64] = {};
    static std::atomic<unsigned int> next{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!base[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_fix_counters) != cudaSuccess) return nullptr;
        base[dev] = static_cast<unsigned int*>(ptr);
    }
    return base[dev] + static_cast<size_t>(next.fetch_add(1) % kFixSlots) * (kFixTiles * 2);
}

// Workspace floats of a split product: one 128 x bn block per (tile, slice).
size_t partial_bytes(int64_t M, int64_t N, int splits) {
    if (splits <= 1) return 0;
    const int bn = N <= 64 ? 64 : 128;
    return static_cast<size_t>(ceil_div(M, kBM) * ceil_div(N, bn)) * splits * kBM * bn * 4;
}

int pick_splits(int64_t M, int64_t N, int bn, int64_t K) {
    const int64_t tiles = ceil_div(M, kBM) * ceil_div(N, bn);
    const int64_t nkb = ceil_div(K, kBK);
    if (tiles < 1 || nkb < 1) return 1;
    int64_t s = num_sms() / tiles;
    if (s > nkb / 4) s = nkb / 4;     // at least 4 k-blocks per slice
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}
int pick_bn(int64_t N) { return N <= 64 ? 64 : 128; }

// CTA pairs (256 x 256 tiles, persistent) pay off for wide outputs once every pair gets at least two
// tiles, or fewer tiles with a long contraction each; short products with few tiles are better
// off as many small single-CTA tiles.
bool pair_worthwhile(int64_t M, int64_t N, int64_t K) {
    const int64_t tiles = ceil_div(M, 256) * ceil_div(N, 256);
    return N >= 256 && (tiles >= num_sms() || (tiles >= 48 && K >= 2048));
}

// Slice counts for two products that share one launch (dU: Mu x N, dV: Mv x N, both contracting
// over K): all CTAs should fit one wave and finish together, so the longest CTA (in k-blocks) is
// minimised subject to tiles_u * su + tiles_v * sv <= SM count.
void pick_pair_splits(int64_t Mu, int64_t Mv, int64_t N, int64_t K, int kblock, int* su, int* sv) {
    const int bn = pick_bn(N);
    const int64_t tu = ceil_div(Mu, kBM) * ceil_div(N, bn), tv = ceil_div(Mv, kBM) * ceil_div(N, bn);
    const int64_t nkb = ceil_div(K, kblock);
    *su = 1; *sv = 1;
    if (tu < 1 || tv < 1 || nkb < 1 || tu + tv > num_sms()) return;
    int64_t best = nkb + 1;
    for (int64_t a = 1; a <= 64 && a <= nkb && tu * a + tv <= num_sms(); ++a) {
        int64_t b = (num_sms() - tu * a) / tv;
        if (b > 64) b = 64;
        if (b > nkb) b = nkb;
        if (b < 1) continue;
        const int64_t longest = std::max(ceil_div(nkb, a), ceil_div(nkb, b));
        if (longest < best) { best = longest; *su = static_cast<int>(a); *sv = static_cast<int>(b); }
    }
}

// Slices of dU (k x r) and dV (n x r) in the backward of the linear layer, and whether dV runs BESIDE
// the fused dX kernel instead of after it.  dV = dY^T T needs nothing that kernel writes.  When the
// contraction of the fused kernel's first product is long against its output (n >= 2k), that kernel is
// left unsplit (one block per 128-row tile, no block repeats another's first product), which leaves
// SMs free; the dV blocks are sized to exactly those SMs, come first in their launch and do not wait
// for the fused kernel, and the dU blocks (which need G) follow on the other SMs once that kernel's
// blocks retire.  (Measured on the Transformer-FFN shapes: doing the same for n < 2k, where only the
// 20 SMs the split fused kernel leaves idle are free, loses more through the long dV blocks than the
// overlap gains.)
void bwd_split_plan(int64_t m, int64_t k, int64_t n, int64_t r, bool fused_dx, int* su, int* sv, bool* beside) {
    pick_pair_splits(k, n, r, m, kBK, su, sv);
    *beside = false;
    if (!fused_dx || n < 2 * k) return;
    const int bn = pick_bn(r);
    const int64_t row_tiles = ceil_div(m, kBM), nkb = ceil_div(m, kBK);
    const int64_t tu = ceil_div(k, kBM) * ceil_div(r, bn), tv = ceil_div(n, kBM) * ceil_div(r, bn);
    const int64_t free_sms = num_sms() - row_tiles;
    const int64_t smax = std::max<int64_t>(1, std::min<int64_t>(64, nkb / 4));
    if (free_sms < tv || tu > kFixTiles || tv > kFixTiles) return;
    const int64_t b = std::min(free_sms / tv, smax);
    // dU gets the SMs that dV does not hold: dV may still be running when the fused kernel retires
    const int64_t a = std::min((num_sms() - tv * b) / tu, smax);
    if (a < 1 || b < 1) return;
    *su = static_cast<int>(a);
    *sv = static_cast<int>(b);
    *beside = true;
}

// C[M,N] (bf16, ldc) = A * B.  `partial` must hold splits*M*N floats when splits > 1.
struct ConvA {
    int mode;                   // 1: dX (A = dT image), 2: dU (A = x image)
    int N, H, W, Cimg;          // the NHWC tensor A is read from (Cimg channels)
    int kw, pad, Cw;            // kernel width, padding, channels of the layer input (rows per tap of U)
};

struct GemmLaunch {
    CUtensorMap ta, tb;
    GemmParams p;
    dim3 grid;
    int bn;
};

// Encodes the tensor maps and launch geometry of C[M,N] = A * B without launching.
int gemm_prepare(const Operand& A, const Operand& B, int64_t M, int64_t N, int64_t K, void* C, int64_t ldc,
                 int splits, float* partial, const ConvA* cv, GemmLaunch* out, const Grouping* gr = nullptr) {
    if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return PF_ERR_UNSUPPORTED;
    const int groups = gr ? gr->groups : 1;
    const bool sum_groups = gr && gr->sum_groups;
    if (gr && (cv || groups < 1 || groups > 1024 || (sum_groups && (A.mn_major || B.mn_major)))) return PF_ERR_UNSUPPORTED;
    // wide outputs that would need more than one wave of 128-column tiles (two CTAs per SM) take
    // 256-column tiles
    const int bn = (splits <= 1 && N >= 512 && ceil_div(M, kBM) * ceil_div(N, 128) > 2 * num_sms()) ? 256 : pick_bn(N);
    CUtensorMap& ta = out->ta;
    CUtensorMap& tb = out->tb;
    bool oka, okb;
    if (cv && cv->mode == 1) {          // B = U as a (taps * Cw) x R matrix, K-major
        oka = cached_map_nhwc(&ta, A.p, cv->N, cv->H, cv->W, cv->Cimg, cv->W, conv_box_h(cv->H, cv->W, 128));
        okb = cached_map_2d(&tb, B.p, static_cast<int64_t>(K / cv->Cimg) * cv->Cw, cv->Cimg, B.ld, bn);
    } else if (cv && cv->mode == 2) {
        oka = cached_map_nhwc(&ta, A.p, cv->N, cv->H, cv->W, cv->Cimg, cv->W, conv_box_h(cv->H, cv->W, 64));
        okb = cached_map_2d(&tb, B.p, K, N, B.ld, 64);
    } else if (gr) {
        const int64_t ga = A.gs == 0 ? 1 : groups, gb = B.gs == 0 ? 1 : groups;
        oka = A.mn_major ? cached_map_3d(&ta, A.p, ga, K, M, A.ld, A.gs, 64) : cached_map_3d(&ta, A.p, ga, M, K, A.ld, A.gs, kBM);
        okb = B.mn_major ? cached_map_3d(&tb, B.p, gb, K, N, B.ld, B.gs, 64) : cached_map_3d(&tb, B.p, gb, N, K, B.ld, B.gs, bn);
    } else {
        oka = A.mn_major ? cached_map_2d(&ta, A.p, K, M, A.ld, 64) : cached_map_2d(&ta, A.p, M, K, A.ld, kBM);
        okb = B.mn_major ? cached_map_2d(&tb, B.p, K, N, B.ld, 64) : cached_map_2d(&tb, B.p, N, K, B.ld, bn);
    }
    if (!oka || !okb) return PF_ERR_CUDA;
    GemmParams& p = out->p;
    p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
    p.a_mn = A.mn_major; p.b_mn = B.mn_major;
    p.C = C; p.ldc = ldc; p.partial = partial;
    p.C2 = nullptr; p.ldc2 = 0;
    p.conv_mode = 0; p.cv_blks = 1; p.cv_kw = 1; p.cv_pad = 0; p.cv_C = 1; p.cv_box_h = 1; p.cv_tpi = 1;
    if (cv) {
        p.conv_mode = cv->mode; p.cv_kw = cv->kw; p.cv_pad = cv->pad; p.cv_C = cv->Cw;
        p.cv_blks = cv->Cimg / 64;
        p.cv_box_h = conv_box_h(cv->H, cv->W, cv->mode == 1 ? 128 : 64);
        p.cv_tpi = cv->H / p.cv_box_h;
    }
    p.rows_tile = (cv && cv->mode == 1) ? p.cv_box_h * cv->W : kBM;
    p.kpix = (cv && cv->mode == 2) ? p.cv_box_h * cv->W : kBK;
    p.groups = gr ? groups : 1;
    p.a_shared = gr && A.gs == 0; p.b_shared = gr && B.gs == 0;
    p.c_gstride = gr ? gr->c_gs : 0;
    p.kb_per_group = 0;
    int64_t nkb = ceil_div(K, p.kpix);
    if (sum_groups) {                       // the groups are part of the contraction: one output
        p.kb_per_group = static_cast<int>(nkb);
        nkb *= groups;
        p.groups = 1;
    }
    const int out_groups = sum_groups ? 1 : groups;
    p.nkb_total = static_cast<int>(nkb);
    p.kb_per_split = static_cast<int>(ceil_div(nkb, splits < 1 ? 1 : splits));
    p.splits = static_cast<int>(ceil_div(nkb, p.kb_per_split));   // every slice gets >= 1 k-block
    p.status = device_status_ptr();
    dim3 grid(static_cast<unsigned>(ceil_div(M, p.rows_tile)), static_cast<unsigned>(ceil_div(N, bn)),
              static_cast<unsigned>(p.splits * out_groups));
    if (grid.y > 65535 || grid.z > 65535) return PF_ERR_UNSUPPORTED;
    p.tiles_x = static_cast<int>(grid.x);
    p.tiles_y = static_cast<int>(grid.y);
    p.bn = bn;
    p.num_stages = pick_stages(bn, static_cast<int64_t>(grid.x) * grid.y * grid.z);
    p.counters = nullptr;
    p.independent = 0;
    if (p.splits > 1) {
        // the CTAs of a tile wait for one another, so all of them must be resident at once
        if (static_cast<int64_t>(grid.x) * grid.y * out_groups > kFixTiles || static_cast<int64_t>(grid.x) * grid.y * grid.z > num_sms() ||
            bn == 256 || partial == nullptr)
            return PF_ERR_UNSUPPORTED;
        // the slices of a CTA's share are gathered in the pipeline stages
        const int64_t rper = ceil_div(kBM, p.splits);
        const int64_t room = static_cast<int64_t>(p.num_stages) * (kBM * kBK * 2 + bn * kBK * 2);
        if (rper * p.splits * (bn * 4) > room || static_cast<int64_t>(kBM) * bn * 4 > room) return PF_ERR_UNSUPPORTED;
        p.counters = next_fix_counters();
        if (!p.counters) return PF_ERR_CUDA;
    }
    out->grid = grid;
    out->bn = bn;
    return PF_OK;
}

// Launches one prepared product on its own.
int launch_prepared(const GemmLaunch& g, cudaStream_t stream) {
    const cudaError_t e = g.bn == 64    ? launch_gemm<64>(g.ta, g.tb, g.p, g.grid, stream)
                          : g.bn == 128 ? launch_gemm<128>(g.ta, g.tb, g.p, g.grid, stream)
                                        : launch_gemm<256>(g.ta, g.tb, g.p, g.grid, stream);
    return e == cudaSuccess ? PF_OK : PF_ERR_CUDA;
}

// `copy2` (optional): asks for a second copy of C at pitch ldc2; *copy2_done tells whether the launch
// wrote it (only a split contraction can), else the caller copies C itself.
int gemm(const Operand& A, const Operand& B, int64_t M, int64_t N, int64_t K, void* C, int64_t ldc,
         int splits, float* partial, cudaStream_t stream, const ConvA* cv = nullptr, void* copy2 = nullptr,
         int64_t ldc2 = 0, bool* copy2_done = nullptr) {
    // wide, many-tile (tensor-bound) products run on CTA pairs, which halve the operand traffic per SM
    if (!cv && splits <= 1 && pair_worthwhile(M, N, K)) {
        const int st2 = gemm_pair_2sm(A.p, A.ld, A.mn_major, B.p, B.ld, B.mn_major, M, N, K, C, ldc, stream);
        if (st2 != PF_ERR_UNSUPPORTED) {
            if (copy2_done) *copy2_done = false;
            return st2;
        }
    }
    GemmLaunch g;
    int st = gemm_prepare(A, B, M, N, K, C, ldc, splits, partial, cv, &g);
    if (st == PF_ERR_UNSUPPORTED && splits > 1) st = gemm_prepare(A, B, M, N, K, C, ldc, 1, nullptr, cv, &g);
    if (st != PF_OK) return st;
    if (copy2_done) *copy2_done = false;
    if (copy2 && g.p.splits > 1) {
        g.p.C2 = copy2; g.p.ldc2 = ldc2;
        if (copy2_done) *copy2_done = true;
    }
    const GemmParams& p = g.p;
    cudaError_t e = g.bn == 64    ? launch_gemm<64>(g.ta, g.tb, p, g.grid, stream)
                    : g.bn == 128 ? launch_gemm<128>(g.ta, g.tb, p, g.grid, stream)
                                  : launch_gemm<256>(g.ta, g.tb, p, g.grid, stream);
    return e == cudaSuccess ? PF_OK : PF_ERR_CUDA;
}

// One launch for up to three prepared products.  Products whose contraction is split must come
// first and fit the machine together (their CTAs wait for one another); tiles are 64 or 128 wide.
int gemm_multi(const GemmLaunch* const* g, int count, cudaStream_t stream) {
    if (count < 1 || count > 3) return PF_ERR_UNSUPPORTED;
    int ctas[3] = {0, 0, 0};
    int total = 0, split_ctas = 0;
    bool seen_plain = false;
    for (int i = 0; i < count; ++i) {
        if (g[i]->bn != 64 && g[i]->bn != 128) return PF_ERR_UNSUPPORTED;
        ctas[i] = static_cast<int>(g[i]->grid.x * g[i]->grid.y * g[i]->grid.z);
        total += ctas[i];
        if (g[i]->p.splits > 1) {
            if (seen_plain) return PF_ERR_UNSUPPORTED;
            split_ctas += ctas[i];
        } else {
            seen_plain = true;
        }
    }
    // The blocks of a split product wait for one another and must be resident together.  A first
    // product marked independent never waits for anything later in the launch and is dispatched
    // first, so it only has to fit by itself, and the products behind it by themselves.
    const bool lead = count > 1 && g[0]->p.independent && g[0]->p.splits > 1;
    const int resident = lead ? std::max(ctas[0], split_ctas - ctas[0]) : split_ctas;
    if (resident > num_sms()) return PF_ERR_UNSUPPORTED;
    const int wave = lead ? std::max(ctas[0], total - ctas[0]) : total;
    GemmParams prm[3];
    size_t smem = 0;
    for (int i = 0; i < 3; ++i) {
        const GemmLaunch* src = g[i < count ? i : 0];
        prm[i] = src->p;
        const int stages = pick_stages(src->bn, wave);
        prm[i].num_stages = stages;
        if (i < count) {
            smem = std::max(smem, gemm_smem(src->bn, stages));
            const int64_t rper = ceil_div(kBM, prm[i].splits);
            const int64_t room = static_cast<int64_t>(stages) * (kBM * kBK * 2 + src->bn * kBK * 2);
            if (prm[i].splits > 1 && (rper * prm[i].splits * (src->bn * 4) > room || static_cast<int64_t>(kBM) * src->bn * 4 > room))
                return PF_ERR_UNSUPPORTED;
        }
    }
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_gemm3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(gemm_smem(128, kMaxStages))) != cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    const GemmLaunch* a = g[0];
    const GemmLaunch* b = g[count > 1 ? 1 : 0];
    const GemmLaunch* c = g[count > 2 ? 2 : 0];
    const int end0 = ctas[0], end1 = ctas[0] + ctas[1];
    const cudaError_t e = launch_overlapped(
        tc_gemm3_kernel, dim3(static_cast<unsigned>(total)), dim3(kGemmThreads), smem, stream, a->ta, a->tb, b->ta, b->tb,
        c->ta, c->tb, prm[0], prm[1], prm[2], end0, end1, make_int2(a->grid.x, a->grid.y), make_int2(b->grid.x, b->grid.y),
        make_int2(c->grid.x, c->grid.y));
    if (e != cudaSuccess) return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

// A row-major bf16 matrix that TMA must read: used as is when 16-byte aligned with a pitch that is
// a multiple of 8 elements, otherwise copied to `scratch` with the pitch rounded up.
struct Staged {
    const void* p;
    int64_t ld;
};
int64_t pad8(int64_t v) { return (v + 7) / 8 * 8; }

// The re-pitch copies of one call are collected and issued as one launch.
struct RepackList {
    RepackJob jobs[6];
    int count = 0;
    int flush(cudaStream_t stream) {
        const cudaError_t e = count > 0 ? repack_rows_bf16_multi(jobs, count, stream) : cudaSuccess;
        count = 0;
        return e == cudaSuccess ? PF_OK : PF_ERR_CUDA;
    }
};

// returns 0 = usable, 1 = needs repack but no room reserved (decline), <0 never
int stage_operand(const void* p, int64_t ld, int64_t rows, int64_t cols, char*& scratch, Staged* out, RepackList* list) {
    if (tma_ok(p, ld)) { out->p = p; out->ld = ld; return 0; }
    if (cols % 8 == 0) return 1;   // the workspace query reserves repack room only for ragged widths
    const int64_t ldp = pad8(cols);
    list->jobs[list->count++] = RepackJob{p, ld, scratch, ldp, rows, cols, ldp};
    out->p = scratch; out->ld = ldp;
    scratch += align_up(static_cast<size_t>(rows) * ldp * 2, 256);
    return 0;
}
// The fused chain pays off once there are enough 128-row tiles to fill the machine, and while the
// rank is small enough for the layer to be bound by memory traffic: from r = 256 up the two
// products are tensor-bound and run faster unfused on CTA pairs (the intermediate is only m x r).
bool use_chain(int64_t m, int64_t r) { return m >= 2048 && r <= 192; }

size_t repack_room(int64_t rows, int64_t cols) {
    return cols % 8 == 0 ? 0 : align_up(static_cast<size_t>(rows) * pad8(cols) * 2, 256);
}

// Room for the fp32 slices of dU and dV under either backward structure (which one a call takes
// depends on pointers the workspace query does not see): no block count exceeds one per SM per product.
void bwd_partial_bytes(int64_t m, int64_t k, int64_t n, int64_t r, size_t* bytes_u, size_t* bytes_v) {
    int su, sv, su2, sv2;
    bool beside;
    bwd_split_plan(m, k, n, r, false, &su, &sv, &beside);
    bwd_split_plan(m, k, n, r, true, &su2, &sv2, &beside);
    *bytes_u = align_up(std::max(partial_bytes(k, r, su), partial_bytes(k, r, su2)), 256);
    *bytes_v = align_up(std::max(partial_bytes(n, r, sv), partial_bytes(n, r, sv2)), 256);
}

}  // namespace

// Extra workspace of the tensor-core linear path: repack buffers for operands whose width is not a
// multiple of 8 elements (TMA needs 16-byte row pitches), the two m x r intermediates at a padded
// pitch, and split partials of dU / dV.
size_t linear_extra_workspace(int64_t m, int64_t k, int64_t n, int64_t r, bool bwd) {
    size_t b = 0;
    b += repack_room(m, k) + repack_room(k, r) + repack_room(n, r);        // x, U, V
    b += align_up(static_cast<size_t>(m) * pad8(r) * 2, 256);               // T at padded pitch
    if (bwd) {
        b += repack_room(m, n);                                             // dY
        b += align_up(static_cast<size_t>(m) * pad8(r) * 2, 256);           // G at padded pitch
        // slices for either backward structure (the choice depends on pointers the query does not see)
        size_t bu, bv;
        bwd_partial_bytes(m, k, n, r, &bu, &bv);
        b += bu + bv;
    }
    // skinny batches: the m x r products (x U, dY V) are split over their contraction to fill the SMs
    const int s1 = std::max(pick_splits(m, r, pick_bn(r), k), bwd ? pick_splits(m, r, pick_bn(r), n) : 1);
    b += align_up(partial_bytes(m, r, s1), 256);
    return b;
}

// Bytes of `a.ws` that linear_fwd(a) will really touch for these pointers and sizes (it takes the
// same decisions in the same order), and whether it will handle the call at all.  The public
// workspace query cannot see pointers and pitches and therefore reserves for every path.
size_t linear_fwd_need(const LinearArgs& a, bool* handles) {
    *handles = false;
    if (encode_fn() == nullptr) return 0;
    if (a.k > (1 << 22) || a.n > (1 << 22) || a.r > (1 << 22)) return 0;
    size_t room = 0;
    const struct { const void* p; int64_t ld, rows, cols; } ops[3] = {
        {a.x, a.ldx, a.m, a.k}, {a.U, a.ldu, a.k, a.r}, {a.V, a.ldv, a.n, a.r}};
    for (const auto& o : ops) {
        if (tma_ok(o.p, o.ld)) continue;
        if (o.cols % 8 == 0) return 0;               // declined: FMA kernels
        room += repack_room(o.rows, o.cols);
    }
    *handles = true;
    const size_t t_bytes = align_up(static_cast<size_t>(a.m) * pad8(a.r) * 2, 256);
    const bool stash_direct = a.T && tma_ok(a.T, a.ldt);
    ChainPlan plan;
    if (use_chain(a.m, a.r) && tma_ok(a.y, a.ldy) && chain_plan(a.m, a.k, a.n, a.r, true, &plan))
        return room + ((a.T && !stash_direct) ? t_bytes : 0);
    return room + t_bytes + align_up(partial_bytes(a.m, a.r, pick_splits(a.m, a.r, pick_bn(a.r), a.k)), 256);
}

int linear_fwd(const LinearArgs& a, int* handled) {
    *handled = 0;
    if (encode_fn() == nullptr) return PF_OK;
    // the grids below index column tiles with 16 bits: absurdly wide layers take the FMA kernels
    if (a.k > (1 << 22) || a.n > (1 << 22) || a.r > (1 << 22)) return PF_OK;
    int st = PF_OK;
    char* scratch = a.ws;
    Staged x, U, V;
    RepackList repacks;
    if (stage_operand(a.x, a.ldx, a.m, a.k, scratch, &x, &repacks)) return PF_OK;
    if (stage_operand(a.U, a.ldu, a.k, a.r, scratch, &U, &repacks)) return PF_OK;
    if (stage_operand(a.V, a.ldv, a.n, a.r, scratch, &V, &repacks)) return PF_OK;
    st = repacks.flush(a.stream);
    if (st != PF_OK) return st;
    *handled = 1;
    // T: written straight into the stash when TMA can read it back, else into padded scratch
    void* T = scratch;
    int64_t ldT = pad8(a.r);
    const bool stash_direct = a.T && tma_ok(a.T, a.ldt);
    if (stash_direct) { T = a.T; ldT = a.ldt; }
    ChainPlan plan;
    bool stash_written = false;   // the stash at its own (TMA-unreadable) pitch came out of the first product
    if (use_chain(a.m, a.r) && tma_ok(a.y, a.ldy) && chain_plan(a.m, a.k, a.n, a.r, true, &plan)) {
        // one fused kernel; the intermediate leaves the chip only if a stash was asked for
        st = chain(x.p, x.ld, a.m, a.k, U.p, U.ld, a.r, V.p, V.ld, a.n, a.y, a.ldy, a.T ? T : nullptr, ldT,
                   a.stream, nullptr, 0, a.bias, a.act);
    } else {
        float* p1 = reinterpret_cast<float*>(scratch + align_up(static_cast<size_t>(a.m) * pad8(a.r) * 2, 256));
        st = gemm({x.p, x.ld, false}, {U.p, U.ld, true}, a.m, a.r, a.k, T, ldT,
                  pick_splits(a.m, a.r, pick_bn(a.r), a.k), p1, a.stream, nullptr,
                  (a.T && !stash_direct) ? a.T : nullptr, a.ldt, &stash_written);
        if (st != PF_OK) return st;
        st = gemm({T, ldT, false}, {V.p, V.ld, false}, a.m, a.n, a.r, a.y, a.ldy, 1, nullptr, a.stream);
        // unfused products: bias and activation in a pass of their own over y
        if (st == PF_OK && (a.bias || a.act) &&
            bias_act_inplace(a.y, a.ldy, a.m, a.n, a.bias, a.act, PF_BF16, a.stream) != cudaSuccess)
            return PF_ERR_CUDA;
    }
    if (st != PF_OK) return st;
    if (a.T && !stash_direct && !stash_written &&
        repack_rows_bf16(T, ldT, a.T, a.ldt, a.m, a.r, a.r, a.stream) != cudaSuccess)
        return PF_ERR_CUDA;
    return PF_OK;
}

int linear_bwd(const LinearArgs& a, int* handled) {
    *handled = 0;
    if (encode_fn() == nullptr) return PF_OK;
    // the grids below index column tiles with 16 bits: absurdly wide layers take the FMA kernels
    if (a.k > (1 << 22) || a.n > (1 << 22) || a.r > (1 << 22)) return PF_OK;
    int st = PF_OK;
    char* scratch = a.ws;
    Staged x, U, V, dY, T;
    RepackList repacks;
    if (stage_operand(a.x, a.ldx, a.m, a.k, scratch, &x, &repacks)) return PF_OK;
    if (stage_operand(a.U, a.ldu, a.k, a.r, scratch, &U, &repacks)) return PF_OK;
    if (stage_operand(a.V, a.ldv, a.n, a.r, scratch, &V, &repacks)) return PF_OK;
    if (stage_operand(a.dY, a.lddy, a.m, a.n, scratch, &dY, &repacks)) return PF_OK;
    char* Tbuf = scratch;
    scratch += align_up(static_cast<size_t>(a.m) * pad8(a.r) * 2, 256);
    if (a.T) {
        if (tma_ok(a.T, a.ldt)) { T.p = a.T; T.ld = a.ldt; }
        else if (a.r % 8 == 0) return PF_OK;   // odd pitch on an even width: FMA path
        else {
            repacks.jobs[repacks.count++] = RepackJob{a.T, a.ldt, Tbuf, pad8(a.r), a.m, a.r, pad8(a.r)};
            T.p = Tbuf; T.ld = pad8(a.r);
        }
    }
    st = repacks.flush(a.stream);
    if (st != PF_OK) return st;
    *handled = 1;
    bool need_T = false;
    if (!a.T) {
        need_T = true;
        T.p = Tbuf; T.ld = pad8(a.r);
    }
    char* G = scratch;
    const int64_t ldG = pad8(a.r);
    scratch += align_up(static_cast<size_t>(a.m) * ldG * 2, 256);
    size_t pu_bytes = 0, pv_bytes = 0;
    ChainPlan plan;
    const bool fused_dx = use_chain(a.m, a.r) && (!a.dX || tma_ok(a.dX, a.lddx)) &&
                          chain_plan(a.m, a.n, a.k, a.r, a.dX != nullptr, &plan);
    int su, sv;
    bool dv_beside;
    bwd_split_plan(a.m, a.k, a.n, a.r, fused_dx, &su, &sv, &dv_beside);
    bwd_partial_bytes(a.m, a.k, a.n, a.r, &pu_bytes, &pv_bytes);
    float* pu = reinterpret_cast<float*>(scratch);
    scratch += pu_bytes;
    float* pv = reinterpret_cast<float*>(scratch);
    scratch += pv_bytes;
    float* p1 = reinterpret_cast<float*>(scratch);
    // the slices of the reductions as they will be launched (the last prepared product is the launched one)
    auto note = [](LinearArgs::Slices* out, const GemmLaunch* g) {
        if (!out) return;
        *out = LinearArgs::Slices();
        if (g && g->p.splits > 1) {
            out->partial = g->p.partial; out->splits = g->p.splits; out->bn = g->bn;
            out->tiles_x = static_cast<int>(g->grid.x); out->tiles_y = static_cast<int>(g->grid.y);
        }
    };
    // G = dY V ; dX = G U^T ; dU = x^T G ; dV = dY^T T
    if (need_T) {   // no stash: recompute T = x U
        st = gemm({x.p, x.ld, false}, {U.p, U.ld, true}, a.m, a.r, a.k, Tbuf, pad8(a.r),
                  pick_splits(a.m, a.r, pick_bn(a.r), a.k), p1, a.stream);
        if (st != PF_OK) return st;
    }
    bool dx_pending = false;     // dX still to be computed as a plain product G U^T
    if (fused_dx) {
        st = chain(dY.p, dY.ld, a.m, a.n, V.p, V.ld, a.r, U.p, U.ld, a.k, a.dX, a.lddx, G, ldG, a.stream, nullptr,
                   dv_beside ? 1 : 0);
        if (st != PF_OK) return st;
    } else {
        // Few rows: G = dY V is a contraction split across blocks, and dV = dY^T T, which needs nothing
        // of it, shares its launch (the second block slot of every SM); dU and dX follow in a second one.
        const int sg = pick_splits(a.m, a.r, pick_bn(a.r), a.n);
        GemmLaunch gg, gv, gu, gx;
        bool ok = !pair_worthwhile(a.m, a.r, a.n) && !pair_worthwhile(a.n, a.r, a.m) &&
                  gemm_prepare({dY.p, dY.ld, false}, {V.p, V.ld, true}, a.m, a.r, a.n, G, ldG, sg, p1, nullptr, &gg) == PF_OK &&
                  gemm_prepare({dY.p, dY.ld, true}, {T.p, T.ld, true}, a.n, a.r, a.m, a.dV, a.lddv, sv, pv, nullptr, &gv) == PF_OK &&
                  gemm_prepare({x.p, x.ld, true}, {G, ldG, true}, a.k, a.r, a.m, a.dU, a.lddu, su, pu, nullptr, &gu) == PF_OK;
        if (ok && a.dX)
            ok = gemm_prepare({G, ldG, false}, {U.p, U.ld, false}, a.m, a.k, a.r, a.dX, a.lddx, 1, nullptr, nullptr, &gx) == PF_OK;
        ok = ok && (gg.p.splits > 1 || gv.p.splits <= 1) && (gu.p.splits > 1 || !a.dX || gx.p.splits <= 1);
        if (ok) {
            note(a.du_slices, &gu);
            note(a.dv_slices, &gv);
            const GemmLaunch* first[2] = {&gg, &gv};
            st = gemm_multi(first, 2, a.stream);
            if (st == PF_OK) {
                const GemmLaunch* second[2] = {&gu, &gx};
                st = gemm_multi(second, a.dX ? 2 : 1, a.stream);
                if (st != PF_ERR_UNSUPPORTED) return st;
                // tile widths that cannot share a launch: one launch each
                st = launch_prepared(gu, a.stream);
                if (st == PF_OK && a.dX) st = launch_prepared(gx, a.stream);
                return st;
            }
            if (st != PF_ERR_UNSUPPORTED) return st;
        }
        st = gemm({dY.p, dY.ld, false}, {V.p, V.ld, true}, a.m, a.r, a.n, G, ldG, sg, p1, a.stream);
        if (st != PF_OK) return st;
        dx_pending = a.dX != nullptr;
    }
    {   // dU = x^T G, dV = dY^T T (and dX = G U^T when it is still due): one launch when their tiles allow
        GemmLaunch gu, gv, gx;
        bool ok = gemm_prepare({x.p, x.ld, true}, {G, ldG, true}, a.k, a.r, a.m, a.dU, a.lddu, su, pu, nullptr, &gu) == PF_OK &&
                  gemm_prepare({dY.p, dY.ld, true}, {T.p, T.ld, true}, a.n, a.r, a.m, a.dV, a.lddv, sv, pv, nullptr, &gv) == PF_OK;
        if (ok && dx_pending)
            ok = gemm_prepare({G, ldG, false}, {U.p, U.ld, false}, a.m, a.k, a.r, a.dX, a.lddx, 1, nullptr, nullptr, &gx) == PF_OK;
        if (ok) {
            note(a.du_slices, &gu);
            note(a.dv_slices, &gv);
            const GemmLaunch* list[3] = {&gu, &gv, &gx};
            // a split product has to come before the plain ones
            if (gu.p.splits <= 1 && gv.p.splits > 1) { list[0] = &gv; list[1] = &gu; }
            if (dv_beside && !dx_pending) {
                // dV first (its blocks are dispatched first, onto the SMs the fused kernel left free) and
                // without waiting for the fused kernel; dU follows as that kernel's blocks retire
                gv.p.independent = 1;
                list[0] = &gv; list[1] = &gu;
            }
            st = gemm_multi(list, dx_pending ? 3 : 2, a.stream);
            if (st != PF_ERR_UNSUPPORTED) return st;
            if (dx_pending) {
                // dX has wide tiles of its own (CTA pairs): launch it alone, dU and dV still together
                st = gemm({G, ldG, false}, {U.p, U.ld, false}, a.m, a.k, a.r, a.dX, a.lddx, 1, nullptr, a.stream);
                if (st != PF_OK) return st;
                dx_pending = false;
                if (!(pair_worthwhile(a.k, a.r, a.m) && pair_worthwhile(a.n, a.r, a.m))) {
                    st = gemm_multi(list, 2, a.stream);
                    if (st != PF_ERR_UNSUPPORTED) return st;
                }
            }
        }
    }
    if (dx_pending) {
        st = gemm({G, ldG, false}, {U.p, U.ld, false}, a.m, a.k, a.r, a.dX, a.lddx, 1, nullptr, a.stream);
        if (st != PF_OK) return st;
    }
    note(a.du_slices, nullptr);      // launched by gemm(), which may choose other kernels and slice counts
    note(a.dv_slices, nullptr);
    st = gemm({x.p, x.ld, true}, {G, ldG, true}, a.k, a.r, a.m, a.dU, a.lddu, su, pu, a.stream);
    if (st != PF_OK) return st;
    return gemm({dY.p, dY.ld, true}, {T.p, T.ld, true}, a.n, a.r, a.m, a.dV, a.lddv, sv, pv, a.stream);
}

// ------------------------------------------------------------------------------ grouped linear layer
namespace {
int grouped_splits(int64_t tiles, int64_t nkb) {
    int64_t s = num_sms() / std::max<int64_t>(tiles, 1);
    s = std::min<int64_t>(s, std::min<int64_t>(64, nkb / 4));
    return static_cast<int>(std::max<int64_t>(s, 1));
}
struct GroupedPlan {
    int bn;                       // tile width of the m x r and (k|n) x r products
    int s1, sg, su, sv;           // slices of x U, dY V, dU, dV
    size_t t_bytes, p1_bytes, pu_bytes, pv_bytes;
};
GroupedPlan grouped_plan(int groups, int64_t m, int64_t k, int64_t n, int64_t r) {
    GroupedPlan g;
    g.bn = pick_bn(r);
    const int64_t tr = ceil_div(r, g.bn);
    const int64_t tm = ceil_div(m, kBM) * tr * groups, tk = ceil_div(k, kBM) * tr * groups, tn = ceil_div(n, kBM) * tr * groups;
    g.s1 = grouped_splits(tm, ceil_div(k, kBK));
    g.sg = grouped_splits(tm, ceil_div(n, kBK));
    g.su = grouped_splits(tk, ceil_div(m, kBK));
    g.sv = grouped_splits(tn, ceil_div(m, kBK));
    if (tm > kFixTiles) g.s1 = g.sg = 1;
    if (tk > kFixTiles) g.su = 1;
    if (tn > kFixTiles) g.sv = 1;
    g.t_bytes = align_up(static_cast<size_t>(groups) * m * pad8(r) * 2, 256);
    g.p1_bytes = align_up(static_cast<size_t>(groups) * std::max(partial_bytes(m, r, g.s1), partial_bytes(m, r, g.sg)), 256);
    g.pu_bytes = align_up(static_cast<size_t>(groups) * partial_bytes(k, r, g.su), 256);
    g.pv_bytes = align_up(static_cast<size_t>(groups) * partial_bytes(n, r, g.sv), 256);
    return g;
}
bool grouped_ok(const void* p, int64_t ld, int64_t gs) { return tma_ok(p, ld) && gs % 8 == 0; }
}  // namespace

size_t grouped_workspace(int groups, int64_t m, int64_t k, int64_t n, int64_t r, bool bwd) {
    const GroupedPlan g = grouped_plan(groups, m, k, n, r);
    return g.t_bytes + g.p1_bytes + (bwd ? g.t_bytes + g.pu_bytes + g.pv_bytes : 0);
}

int linear_grouped_fwd(const GroupedArgs& a, int* handled) {
    *handled = 0;
    if (encode_fn() == nullptr || a.groups > 1024 || a.k > (1 << 22) || a.n > (1 << 22) || a.r > (1 << 22)) return PF_OK;
    if (!grouped_ok(a.x, a.ldx, a.sx) || !grouped_ok(a.U, a.ldu, a.su) || !grouped_ok(a.V, a.ldv, a.sv)) return PF_OK;
    const GroupedPlan gp = grouped_plan(a.groups, a.m, a.k, a.n, a.r);
    // T: the stash itself when TMA can read it back, else scratch at a padded pitch (copied out afterwards)
    const bool stash_direct = a.T && grouped_ok(a.T, a.ldt, a.st);
    if (a.T && !stash_direct) return PF_OK;
    void* T = stash_direct ? a.T : static_cast<void*>(a.ws);
    const int64_t ldT = stash_direct ? a.ldt : pad8(a.r), sT = stash_direct ? a.st : a.m * pad8(a.r);
    float* p1 = reinterpret_cast<float*>(a.ws + gp.t_bytes);
    GemmLaunch g1, g2;
    const Grouping gt{a.groups, sT, false}, gy{a.groups, a.sy, false};
    int st = gemm_prepare({a.x, a.ldx, false, a.sx}, {a.U, a.ldu, true, a.su}, a.m, a.r, a.k, T, ldT, gp.s1, p1, nullptr, &g1, &gt);
    if (st == PF_OK)
        st = gemm_prepare({T, ldT, false, sT}, {a.V, a.ldv, false, a.sv}, a.m, a.n, a.r, a.y, a.ldy, 1, nullptr, nullptr, &g2, &gy);
    if (st == PF_ERR_UNSUPPORTED) return PF_OK;
    if (st != PF_OK) return st;
    *handled = 1;
    st = launch_prepared(g1, a.stream);
    if (st != PF_OK) return st;
    return launch_prepared(g2, a.stream);
}

int linear_grouped_bwd(const GroupedArgs& a, int* handled) {
    *handled = 0;
    if (encode_fn() == nullptr || a.groups > 1024 || a.k > (1 << 22) || a.n > (1 << 22) || a.r > (1 << 22)) return PF_OK;
    if (!grouped_ok(a.x, a.ldx, a.sx) || !grouped_ok(a.U, a.ldu, a.su) || !grouped_ok(a.V, a.ldv, a.sv) ||
        !grouped_ok(a.dY, a.lddy, a.sdy) || (a.T && !grouped_ok(a.T, a.ldt, a.st)))
        return PF_OK;
    const GroupedPlan gp = grouped_plan(a.groups, a.m, a.k, a.n, a.r);
    char* ws = a.ws;
    void* Tbuf = ws; ws += gp.t_bytes;
    float* p1 = reinterpret_cast<float*>(ws); ws += gp.p1_bytes;
    void* Gbuf = ws; ws += gp.t_bytes;
    float* pu = reinterpret_cast<float*>(ws); ws += gp.pu_bytes;
    float* pv = reinterpret_cast<float*>(ws);
    const int64_t ldW = pad8(a.r), sW = a.m * pad8(a.r);
    const void* T = a.T ? a.T : Tbuf;
    const int64_t ldT = a.T ? a.ldt : ldW, sT = a.T ? a.st : sW;
    const bool shared_x = a.sx == 0 && a.groups > 1;
    GemmLaunch gT, gG, gV, gU, gX;
    const Grouping gw{a.groups, sW, false}, gdv{a.groups, a.sdv, false}, gdu{a.groups, a.sdu, false};
    const Grouping gdx{a.groups, shared_x ? 0 : a.sdx, shared_x};
    int st = PF_OK;
    if (!a.T) st = gemm_prepare({a.x, a.ldx, false, a.sx}, {a.U, a.ldu, true, a.su}, a.m, a.r, a.k, Tbuf, ldW, gp.s1, p1, nullptr, &gT, &gw);
    // the recomputed T and G share the slice buffer p1: they are separate launches, one after the other
    if (st == PF_OK) st = gemm_prepare({a.dY, a.lddy, false, a.sdy}, {a.V, a.ldv, true, a.sv}, a.m, a.r, a.n, Gbuf, ldW, gp.sg, p1, nullptr, &gG, &gw);
    if (st == PF_OK) st = gemm_prepare({a.dY, a.lddy, true, a.sdy}, {T, ldT, true, sT}, a.n, a.r, a.m, a.dV, a.lddv, gp.sv, pv, nullptr, &gV, &gdv);
    if (st == PF_OK) st = gemm_prepare({a.x, a.ldx, true, a.sx}, {Gbuf, ldW, true, sW}, a.k, a.r, a.m, a.dU, a.lddu, gp.su, pu, nullptr, &gU, &gdu);
    if (st == PF_OK && a.dX)
        st = gemm_prepare({Gbuf, ldW, false, sW}, {a.U, a.ldu, false, a.su}, a.m, a.k, a.r, a.dX, a.lddx, 1, nullptr, nullptr, &gX, &gdx);
    if (st == PF_ERR_UNSUPPORTED) return PF_OK;
    if (st != PF_OK) return st;
    *handled = 1;
    if (!a.T) {
        st = launch_prepared(gT, a.stream);
        if (st != PF_OK) return st;
    }
    // launch A: G = dY V and dV = dY^T T (independent of each other); launch B: dU = x^T G and dX = G U^T
    auto pair = [&](const GemmLaunch& p0, const GemmLaunch& q0, bool has_q) {
        const GemmLaunch* list[2] = {&p0, &q0};
        if (has_q && p0.p.splits <= 1 && q0.p.splits > 1) { list[0] = &q0; list[1] = &p0; }   // split products first
        int r2 = gemm_multi(list, has_q ? 2 : 1, a.stream);
        if (r2 != PF_ERR_UNSUPPORTED) return r2;
        r2 = launch_prepared(p0, a.stream);
        if (r2 == PF_OK && has_q) r2 = launch_prepared(q0, a.stream);
        return r2;
    };
    st = pair(gG, gV, true);
    if (st != PF_OK) return st;
    return pair(gU, gX, a.dX != nullptr);
}

// After a bounded wait has expired some CTAs may have left their tile counters non-zero.
void reset_fix_counters() {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_fix_counters) == cudaSuccess) cudaMemset(ptr, 0, sizeof(unsigned int) * kFixSlots * kFixTiles * 2);
}

// Tensor-core envelope of the factorized convolution: stride 1, "same" padding, channel counts
// that tile evenly, image rows that pack into 128-pixel (forward, dX) and 64-pixel (dU) tiles.
// (The forward also takes stride 2: its image tiles are fetched with a step of two pixels, and only the
// output row has to fit a tile.  The backward of a strided convolution runs on the FMA kernels.)
static bool conv_tc_ok(const ConvArgs& a, bool fwd = false) {
    if ((a.stride != 1 && !(fwd && a.stride == 2)) || a.kh != a.kw || 2 * a.pad != a.kh - 1) return false;
    if (a.C % 128 != 0 || a.R % 64 != 0 || a.O % 8 != 0 || a.R > 384) return false;
    if (fwd ? a.Wo > 128 : a.W > 64) return false;    // backward: one image row must fit a 64-pixel k-block of dU
    if (static_cast<int64_t>(a.N) * a.H * a.W > 0x7fffffff) return false;
    return encode_fn() != nullptr;
}
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

size_t conv_extra_workspace(int N, int H, int W, int C, int R, int O, int kh, int kw, int stride, int pad,
                            bool bwd) {
    if (!bwd) return 0;
    // split partials of dU ((kh*kw*C) x R) and dV (O x R)
    const int64_t P = static_cast<int64_t>(N) * H * W, Keff = static_cast<int64_t>(kh) * kw * C;
    int su, sv;
    pick_pair_splits(Keff, O, R, P, conv_box_h(H, W, 64) * W, &su, &sv);
    (void)stride; (void)pad;
    return align_up(partial_bytes(Keff, R, su), 256) + align_up(partial_bytes(O, R, sv), 256);
}

int conv_fwd(const ConvArgs& a, int* handled) {
    *handled = 0;
    if (!conv_tc_ok(a, true) || !aligned16(a.x) || !aligned16(a.U) || !aligned16(a.V) || !aligned16(a.y) ||
        (a.T && !aligned16(a.T)))
        return PF_OK;
    const int64_t M = static_cast<int64_t>(a.N) * a.Ho * a.Wo, Keff = static_cast<int64_t>(a.kh) * a.kw * a.C;
    if (M < 1 || a.stride * a.Wo > 256) return PF_OK;
    ChainPlan plan;
    if (!chain_plan(M, Keff, a.O, a.R, true, &plan, conv_box_h(a.Ho, a.Wo, 128) * a.Wo)) return PF_OK;
    *handled = 1;
    const ChainConv cv{a.N, a.H, a.W, a.C, a.kh, a.kw, a.pad, a.stride};
    return chain(a.x, a.C, M, Keff, a.U, a.R, a.R, a.V, a.R, a.O, a.y, a.O, a.T, a.R, a.stream, &cv);
}

int conv_bwd(const ConvArgs& a, int* handled) {
    *handled = 0;
    if (!conv_tc_ok(a) || !aligned16(a.x) || !aligned16(a.U) || !aligned16(a.V) || !aligned16(a.dY) ||
        (a.T && !aligned16(a.T)) || (a.dX && !aligned16(a.dX)))
        return PF_OK;
    const int64_t M = static_cast<int64_t>(a.N) * a.H * a.W, Keff = static_cast<int64_t>(a.kh) * a.kw * a.C;
    ChainPlan plan;
    if (!a.T && !chain_plan(M, Keff, a.O, a.R, false, &plan)) return PF_OK;
    int st;
    const void* T = a.T ? a.T : a.ws_T;
    void* dT = a.ws_G;
    int su, sv;
    pick_pair_splits(Keff, a.O, a.R, M, conv_box_h(a.H, a.W, 64) * a.W, &su, &sv);
    float* pu = reinterpret_cast<float*>(a.ws);
    float* pv = reinterpret_cast<float*>(a.ws + align_up(partial_bytes(Keff, a.R, su), 256));
    // Every product is prepared (tensor maps, geometry; nothing launched) before the call is
    // accepted, so a shape that one of them cannot take still reaches the FMA kernels.
    // dU[tap] = shifted x^T dT ; dV = dY^T T   (reductions over all pixels, split across CTAs)
    // dX = sum over taps of shifted dT times U[tap]^T  (implicit GEMM, contraction kh*kw*R)
    const ConvA cu{2, a.N, a.H, a.W, a.C, a.kw, a.pad, a.C};
    const ConvA cx{1, a.N, a.H, a.W, a.R, a.kw, a.pad, a.C};
    GemmLaunch gt, gu, gv, gx;
    auto prepare = [](const Operand& A, const Operand& B, int64_t Mm, int64_t Nn, int64_t Kk, void* C, int64_t ldc,
                      int splits, float* partial, const ConvA* cv, GemmLaunch* out) {
        int r = gemm_prepare(A, B, Mm, Nn, Kk, C, ldc, splits, partial, cv, out);
        if (r == PF_ERR_UNSUPPORTED && splits > 1) r = gemm_prepare(A, B, Mm, Nn, Kk, C, ldc, 1, nullptr, cv, out);
        return r;
    };
    st = prepare({a.dY, a.O, false}, {a.V, a.R, true}, M, a.R, a.O, dT, a.R, 1, nullptr, nullptr, &gt);
    if (st == PF_OK) st = prepare({a.x, a.C, true}, {dT, a.R, true}, Keff, a.R, M, a.dU, a.R, su, pu, &cu, &gu);
    if (st == PF_OK) st = prepare({a.dY, a.O, true}, {T, a.R, true}, a.O, a.R, M, a.dV, a.R, sv, pv, nullptr, &gv);
    if (st == PF_OK && a.dX)
        st = prepare({dT, a.R, false}, {a.U, a.R, false}, M, a.C, static_cast<int64_t>(a.kh) * a.kw * a.R, a.dX, a.C, 1,
                     nullptr, &cx, &gx);
    if (st == PF_ERR_UNSUPPORTED) return PF_OK;      // declined: nothing has been launched
    if (st != PF_OK) return st;
    *handled = 1;
    {   // both reductions are launched exactly as prepared (together or one by one)
        const GemmLaunch* gs[2] = {&gu, &gv};
        LinearArgs::Slices* outs[2] = {a.du_slices, a.dv_slices};
        for (int i = 0; i < 2; ++i) {
            if (!outs[i]) continue;
            *outs[i] = LinearArgs::Slices();
            if (gs[i]->p.splits > 1) {
                outs[i]->partial = gs[i]->p.partial; outs[i]->splits = gs[i]->p.splits; outs[i]->bn = gs[i]->bn;
                outs[i]->tiles_x = static_cast<int>(gs[i]->grid.x); outs[i]->tiles_y = static_cast<int>(gs[i]->grid.y);
            }
        }
    }
    if (!a.T) {   // recompute the thin convolution (phase 1 of the forward only)
        const ChainConv cv{a.N, a.H, a.W, a.C, a.kh, a.kw, a.pad};
        st = chain(a.x, a.C, M, Keff, a.U, a.R, a.R, a.V, a.R, a.O, nullptr, a.O, a.ws_T, a.R, a.stream, &cv);
        if (st != PF_OK) return st;
    }
    // dT = dY V  (per pixel)
    st = launch_prepared(gt, a.stream);
    if (st != PF_OK) return st;
    // dU, dV and dX depend on dT only and share one launch: the few long CTAs of the split reductions
    // start first and the many short dX tiles fill the second CTA slot of every SM beside them.
    const GemmLaunch* list[3] = {&gu, &gv, &gx};
    if (gu.p.splits <= 1 && gv.p.splits > 1) { list[0] = &gv; list[1] = &gu; }
    st = gemm_multi(list, a.dX ? 3 : 2, a.stream);
    if (st != PF_ERR_UNSUPPORTED) return st;
    // separate launches (tile widths that cannot share one)
    if (a.dX) {
        st = launch_prepared(gx, a.stream);
        if (st != PF_OK) return st;
    }
    st = launch_prepared(gu, a.stream);
    if (st != PF_OK) return st;
    return launch_prepared(gv, a.stream);
}

}  // namespace tc
}  // namespace pf
