/*
 * pf.h -- C ABI of the low-rank pre-factorized layer library for NVIDIA B200 (sm_100a).
 *
 * The library computes the forward and backward passes of layers whose dense weight
 * W (k x n) has been replaced by two factors U (k x r) and V (n x r), W ~ U V^T
 * (Pufferfish, Section 2), plus the flat gradient buffer that is communicated once per
 * iteration (Section 4.1).
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *   - The caller owns every buffer.  The library never allocates, frees or
 *     synchronises; all work is enqueued on `cuda_stream` (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and returns immediately.
 *   - Inputs are never modified.  Outputs are overwritten (never accumulated into).
 *     No output may alias an input or another output.
 *   - All tensors of one call share `dtype`; products are accumulated in fp32 and
 *     rounded once (round-to-nearest-even) to `dtype` at the final store.  With
 *     PF_BF16 the on-chip intermediate x U (and dY V) is rounded to bf16 before the
 *     second product.
 *   - Matrices are row-major.  A leading dimension `ld*` is the distance in ELEMENTS
 *     between consecutive rows and must be >= the row length.
 *   - `workspace` is caller-provided scratch of at least the matching
 *     pf_*_workspace() query, 256-byte aligned; its contents are undefined afterwards.
 *     Two calls that may overlap on the GPU must not share a workspace.
 *   - Besides the workspace the library keeps a few fixed device arrays of its own (a
 *     status word and 40 KB of counters at which the thread blocks of a split reduction
 *     meet).  A reduction over the batch (dU, dV, and x U / dY V when the batch is small) is
 *     cut into slices whose thread blocks wait for one another inside one launch, so all
 *     of them must be resident at once: the library sizes such a launch to at most one block
 *     per SM of the device, which guarantees that on an otherwise idle GPU.  Kernels of
 *     other streams (or processes) that occupy SMs at the same time can delay a sibling
 *     block; the wait is bounded (about two seconds), after which the launch gives up, leaves
 *     its outputs unwritten and pf_last_device_status() reports PF_ERR_TIMEOUT.  Calls of this
 *     library on different streams of equal priority may be in flight together (each launch
 *     takes the next of 32 counter sets: keep at most 32 such calls unfinished per device);
 *     do not mix stream priorities, and do not run backward calls beside long-running
 *     kernels that pin most SMs.
 *   - Gradients that are sums over the batch (dU, dV) are added in a fixed order:
 *     repeating a call on the same inputs gives bit-identical results.
 *   - Every entry returns a pf_status.  Errors detected on the host (bad pointer,
 *     bad dimension, workspace too small, ...) are returned BEFORE anything is
 *     launched.  Nothing is printed, nothing aborts.
 *   - Problems with no rows / no tensors (m = 0, N = 0, count = 0) are PF_OK no-ops.
 */
#ifndef PF_H_
#define PF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PF_OK = 0,
    PF_ERR_INVALID_ARG = 1, /* null required pointer, dimension < 1, ld too small, bad dtype,
                               misaligned pointer, negative count */
    PF_ERR_UNSUPPORTED = 2, /* valid mathematics outside the implemented envelope */
    PF_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small; pack capacity too small */
    PF_ERR_CUDA = 4,        /* a CUDA runtime / driver call or a launch failed */
    PF_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (see pf_last_device_status) */
} pf_status;

typedef enum {
    PF_F32 = 0, /* fp32 storage, fp32 FMA arithmetic */
    PF_BF16 = 1 /* bf16 storage, tensor-core products with fp32 accumulation */
} pf_dtype;

/* Static, human-readable name of a status code. */
const char* pf_status_string(int status);

/* Library version, major*10000 + minor*100 + patch. */
int pf_version(void);

/* Number of kernels this library has launched in this process so far (monotonic, all
 * devices and streams).  Lets a caller verify that work ran in this library's kernels. */
long long pf_launch_count(void);

/* Device-side status of the current device: PF_OK, or PF_ERR_TIMEOUT if a kernel of
 * this library gave up on a bounded wait since the last query.  Synchronises the
 * device (blocking) and clears the flag.  Never needed on the normal path. */
int pf_last_device_status(void);

/* ---------------------------------------------------------------------------------
 * Factorized fully-connected layer   y = (x U) V^T
 * (Section 2.1 "Low-rank factorization for FC layers"; Appendix B "FC layer", whose
 *  row convention (xU)V^T is used: U is the input-side factor, V the output-side one.)
 *
 *   x [m, k] (ldx)   U [k, r] (ldu)   V [n, r] (ldv)   y [m, n] (ldy)
 *   T_stash [m, r] (ldt): optional output, the intermediate T = x U rounded to `dtype`,
 *                         for reuse by the backward pass; NULL = not written.
 * m >= 0; k, n, r >= 1 (r need not divide anything; r > min(k, n) is legal).
 * ------------------------------------------------------------------------------- */
size_t pf_lowrank_linear_workspace(int64_t m, int64_t k, int64_t n, int64_t r,
                                   int dtype, int is_bwd);

int pf_lowrank_linear_fwd(const void* x, int64_t ldx, const void* U, int64_t ldu,
                          const void* V, int64_t ldv, void* y, int64_t ldy,
                          void* T_stash, int64_t ldt,
                          int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The forward with the bias and activation that follow the layer in a network:
 *   y = act((x U) V^T + bias)
 * the first half of the factorized feed-forward block FFN(x) = max(0, x W1 + b1) W2 + b2 with
 * W1 = U1 V1^T (Section 2.4; biases are not factorized, Section 2.1), or, with PF_ACT_NONE, any
 * factorized layer followed by its bias (the second half of the FFN, the LSTM gate pre-activations
 * of Section 2.3).
 *   bias [n] in `dtype`, contiguous; NULL = no bias.     act: PF_ACT_NONE or PF_ACT_RELU.
 * bias and activation are applied to the fp32 result before the single rounding to `dtype` in the
 * fused kernel (m >= 2048 rows at r <= 192, PF_BF16).  On the other paths y is first stored in
 * `dtype` and a second pass adds the bias and applies the activation in place (two roundings for
 * PF_BF16; one extra launch).  T_stash is x U as in pf_lowrank_linear_fwd (bias does not enter it).
 * Same workspace, pitches and error behaviour as pf_lowrank_linear_fwd; an act outside the enum is
 * PF_ERR_INVALID_ARG.  The backward of the activation (dY masked by y > 0) and the bias gradient
 * (column sums of dY) are the caller's: pf_lowrank_linear_bwd takes the gradient of (x U) V^T. */
typedef enum {
    PF_ACT_NONE = 0,
    PF_ACT_RELU = 1 /* max(0, .) */
} pf_act;
int pf_lowrank_linear_fwd_act(const void* x, int64_t ldx, const void* U, int64_t ldu,
                              const void* V, int64_t ldv, const void* bias, int act,
                              void* y, int64_t ldy, void* T_stash, int64_t ldt,
                              int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The step of the backward pass that undoes pf_lowrank_linear_fwd_act's epilogue, before
 * pf_lowrank_linear_bwd is called with the result: for y = act(z + bias) and an upstream dY [m, n],
 *   dZ   = dY where y > 0, 0 elsewhere (PF_ACT_RELU);  dZ = dY (PF_ACT_NONE)     written OVER dY
 *   dbias[j] = sum over the m rows of dZ[:, j]  (plain sum, fp32 accumulation in a fixed order,
 *              rounded once to `dtype`)                    [n], NULL = not wanted
 * (Section 2.4: the feed-forward block max(0, x W1 + b1) W2 + b2; biases are trained unfactorized,
 * Section 2.1.)  y (ldy) is the forward's output and is read only for PF_ACT_RELU.  The workspace of
 * pf_bias_act_bwd_workspace(m, n) bytes is needed only when dbias is given.  Two launches with
 * dbias, one without; m = 0 zeroes dbias. */
size_t pf_bias_act_bwd_workspace(int64_t m, int64_t n);
int pf_bias_act_bwd(const void* y, int64_t ldy, void* dY, int64_t lddy, void* dbias,
                    int64_t m, int64_t n, int act, int dtype,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same forward for callers that cannot allocate device memory and therefore have no
 * workspace to pass: latency-critical host paths where cudaMalloc is forbidden because it
 * synchronises the device, plug-ins that are handed tensors but no allocator, and processes
 * whose device memory is already fully committed to a pool they do not control.
 * (The paper has no counterpart; this is a deployment variant.)
 *
 * Identical to pf_lowrank_linear_fwd except that the scratch is a fixed array inside the
 * library image (PF_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the
 * process exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The bound is the scratch this call will really use, which depends on the path its
 *     sizes, pointers and pitches select (it can be far below the public workspace query, which
 *     reserves for every path): many rows at a small rank (m >= 2048, r <= 192, 16-byte aligned
 *     rows) take the fused kernel, which keeps x U on chip and needs nothing when the stash
 *     is written directly; otherwise one m x r copy of x U, the fp32 slices of a split first
 *     product, and re-pitched copies of operands whose row pitch is not a multiple of 16 bytes.
 *     A call that needs more than PF_STATIC_SCRATCH_BYTES is rejected with PF_ERR_WORKSPACE
 *     before anything is launched.  Of the benchmark shapes both Transformer-FFN layers fit,
 *     the LSTM gate layer (700 x 1500 -> 6000, r = 375) fits with 16-byte row pitches and is
 *     refused with its tight 3000 / 750-byte pitches.
 *   - The first call on each device is the set-up call: it looks up the array's device address
 *     with that device current, and (the driver loads modules lazily) it is also when the array
 *     itself is materialised, so free device memory drops once, by the array's size; no later
 *     call changes it.  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the previous call
 *     left in it: two calls that may overlap on the GPU (different streams) race and must be
 *     ordered by the caller.  Nothing in the array has to be cleared between calls.
 * pf_static_scratch_bytes() returns PF_STATIC_SCRATCH_BYTES as compiled. */
#define PF_STATIC_SCRATCH_BYTES (8u << 20)
int pf_lowrank_linear_fwd_static(const void* x, int64_t ldx, const void* U, int64_t ldu,
                                 const void* V, int64_t ldv, void* y, int64_t ldy,
                                 void* T_stash, int64_t ldt,
                                 int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                                 void* cuda_stream);
size_t pf_static_scratch_bytes(void);

/* Gradients of the layer above for an upstream gradient dY [m, n] (chain rule on
 * y = (xU)V^T; plain sums over the m rows, no averaging):
 *   G  = dY V           [m, r]  (kept on chip / in workspace)
 *   dX = G U^T          [m, k]  (lddx)   NULL = not wanted (first layer)
 *   dU = x^T G          [k, r]  (lddu)
 *   dV = dY^T (x U)     [n, r]  (lddv)
 * T_stash [m, r] (ldt): the forward's stashed x U, or NULL to have it recomputed. */
int pf_lowrank_linear_bwd(const void* x, int64_t ldx, const void* U, int64_t ldu,
                          const void* V, int64_t ldv, const void* dY, int64_t lddy,
                          const void* T_stash, int64_t ldt,
                          void* dX, int64_t lddx, void* dU, int64_t lddu, void* dV, int64_t lddv,
                          int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same backward with two options for the factor gradients, as gradient accumulation over
 * micro-batches and fp32 master gradients need them (the paper trains with mixed precision and
 * all-reduces the factor gradients, Sections 4.1 and 3; it does not spell these variants out):
 *   PF_GRAD_ACCUMULATE  dU and dV are ADDED to what the matrices hold: dU <- dU + x^T G, dV <- dV + dY^T (xU)
 *                       (the caller zeroes them before the first micro-batch);
 *   PF_GRAD_F32         dU [k, r] and dV [n, r] are fp32 matrices (lddu, lddv in floats) whatever
 *                       `dtype` is: with PF_BF16 the fp32 sums are stored unrounded.
 * dX is never accumulated and stays in `dtype`.  flags = 0 is pf_lowrank_linear_bwd.  The call runs
 * the same kernels as the plain backward, with the plain gradients directed into the workspace, and
 * one more small launch writes the caller's matrices: where a reduction over the batch was split across
 * thread blocks (every benchmark shape) from the fp32 slices that reduction left in the workspace,
 * summed again in the same order, so that the values are the unrounded fp32 sums (rounded once when
 * added into a PF_BF16 matrix); on the remaining paths from the plain gradient (PF_BF16: the
 * micro-batch's gradient has then been rounded to bf16 before it is widened or added).
 * Same workspace query, pitches and errors as pf_lowrank_linear_bwd; unknown flag bits are
 * PF_ERR_INVALID_ARG.  With m = 0 and PF_GRAD_ACCUMULATE nothing is written. */
#define PF_GRAD_ACCUMULATE 1u
#define PF_GRAD_F32 2u
int pf_lowrank_linear_bwd_ex(const void* x, int64_t ldx, const void* U, int64_t ldu,
                             const void* V, int64_t ldv, const void* dY, int64_t lddy,
                             const void* T_stash, int64_t ldt,
                             void* dX, int64_t lddx, void* dU, int64_t lddu, void* dV, int64_t lddv,
                             int64_t m, int64_t k, int64_t n, int64_t r, int dtype, unsigned flags,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Grouped factorized fully-connected layers: `groups` layers of ONE shape (m, k, n, r), each with its
 * own factor pair (U_g, V_g), in one call -- the per-gate factorization of an LSTM layer
 * (Section 2.3, eq. "lr-lstm-rule": every gate matrix W_i*, W_h* is replaced by its own U V^T; the
 * LSTM table of the appendix lists the 1500 x 375 / 375 x 1500 factors per gate) and the four
 * projections W^Q, W^K, W^V, W^O of a factorized attention block (Section 2.4).
 *     y_g = (x_g U_g) V_g^T ,   g = 0 .. groups-1
 * Every tensor of group g starts s* ELEMENTS after that of group g-1 (sx for x, su for U, ...); the
 * matrices themselves are as in the ungrouped calls.  sx = 0 means ONE input x shared by all groups
 * (the gates of an LSTM all read the same x_t); factors and outputs are always per group.
 * With bf16 and 16-byte aligned pointers, pitches and strides the whole call is two launches
 * (all x_g U_g, then all T_g V_g^T), whatever `groups`; other layouts, and fp32, run group by group
 * through the ungrouped kernels (same results, more launches).
 *
 * Backward, for dY_g [m, n] (stride sdy):
 *   dU_g = x_g^T (dY_g V_g),  dV_g = dY_g^T (x_g U_g)                       (strides sdu, sdv)
 *   dX_g = (dY_g V_g) U_g^T   (stride sdx)            when every group has its own x (sx != 0);
 *   dX   = sum over g of (dY_g V_g) U_g^T, ONE m x k matrix (sdx ignored)   when x is shared (sx = 0),
 *          since a shared input collects the gradient of every group that reads it.
 *   NULL dX = not wanted.  T_stash (stride st): the forward's stash, or NULL to recompute.
 * Two launches (three when T is recomputed) on the fast path.
 * ------------------------------------------------------------------------------- */
size_t pf_lowrank_linear_grouped_workspace(int groups, int64_t m, int64_t k, int64_t n, int64_t r,
                                           int dtype, int is_bwd);

int pf_lowrank_linear_grouped_fwd(int groups,
                                  const void* x, int64_t ldx, int64_t sx,
                                  const void* U, int64_t ldu, int64_t su,
                                  const void* V, int64_t ldv, int64_t sv,
                                  void* y, int64_t ldy, int64_t sy,
                                  void* T_stash, int64_t ldt, int64_t st,
                                  int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

int pf_lowrank_linear_grouped_bwd(int groups,
                                  const void* x, int64_t ldx, int64_t sx,
                                  const void* U, int64_t ldu, int64_t su,
                                  const void* V, int64_t ldv, int64_t sv,
                                  const void* dY, int64_t lddy, int64_t sdy,
                                  const void* T_stash, int64_t ldt, int64_t st,
                                  void* dX, int64_t lddx, int64_t sdx,
                                  void* dU, int64_t lddu, int64_t sdu,
                                  void* dV, int64_t lddv, int64_t sdv,
                                  int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Factorized convolution: a kh x kw convolution into R channels (factor U) followed by a
 * 1 x 1 convolution to O channels (factor V), nothing in between
 * (Section 2.2 "Factorizing a convolution layer"; Appendix B "Convolution layer").
 * Cross-correlation (no kernel flip), zero padding `pad`, stride `stride` on the
 * kh x kw convolution only; no dilation, no groups.
 *
 *   x [N, H, W, C] NHWC, contiguous
 *   U [kh, kw, C, R]  = the unrolled (kh*kw*C) x R matrix of Section 2.2, rows tap-major
 *   V [O, R]
 *   y [N, Ho, Wo, O] NHWC,  Ho = (H + 2 pad - kh) / stride + 1 (floor), Wo likewise
 *   T_stash [N, Ho, Wo, R]: optional output of the thin convolution; NULL = not written.
 * Returns PF_ERR_UNSUPPORTED for kh != kw or stride < 1.
 * ------------------------------------------------------------------------------- */
size_t pf_lowrank_conv_workspace(int N, int H, int W, int C, int R, int O,
                                 int kh, int kw, int stride, int pad, int dtype, int is_bwd);

int pf_lowrank_conv_fwd(const void* x, const void* U, const void* V, void* y, void* T_stash,
                        int N, int H, int W, int C, int R, int O,
                        int kh, int kw, int stride, int pad, int dtype,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Gradients of the factorized convolution for dY [N, Ho, Wo, O]:
 *   dT = dY V (per pixel), dV [O, R] = dY^T T, dU [kh, kw, C, R] = im2col(x)^T dT,
 *   dX [N, H, W, C] = transposed convolution of dT with U (NULL = not wanted).
 * T_stash: the forward's stash or NULL to recompute. */
int pf_lowrank_conv_bwd(const void* x, const void* U, const void* V, const void* dY,
                        const void* T_stash, void* dX, void* dU, void* dV,
                        int N, int H, int W, int C, int R, int O,
                        int kh, int kw, int stride, int pad, int dtype,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* pf_lowrank_conv_bwd with the gradient options of pf_lowrank_linear_bwd_ex (PF_GRAD_ACCUMULATE,
 * PF_GRAD_F32) for dU [kh, kw, C, R] and dV [O, R]; same mechanism, same workspace query. */
int pf_lowrank_conv_bwd_ex(const void* x, const void* U, const void* V, const void* dY,
                           const void* T_stash, void* dX, void* dU, void* dV,
                           int N, int H, int W, int C, int R, int O, int kh, int kw, int stride,
                           int pad, int dtype, unsigned flags, void* workspace, size_t workspace_bytes,
                           void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Flat gradient buffer (Section 4.1 "Implementation details and optimizations": all
 * gradient tensors are packed into one flat buffer so that one all-reduce per iteration
 * suffices).  Copies tensor i (numels[i] elements of `dtype`) bit for bit to
 * flat[offsets_out[i] ...], in list order, tightly (no padding, no conversion, no scaling):
 *   offsets_out[0] = 0, offsets_out[i+1] = offsets_out[i] + numels[i].
 *
 *   grads        host array of `count` device pointers (element-aligned)
 *   numels       host array of `count` element counts (>= 0)
 *   flat         device buffer of `flat_capacity_elems` elements
 *   offsets_out  host array of count+1 entries, written before return (element units)
 * No workspace is needed (workspace arguments are accepted and ignored).
 * PF_ERR_WORKSPACE if the tensors do not fit in flat_capacity_elems.
 * ------------------------------------------------------------------------------- */
int pf_pack_factor_grads(const void* const* grads, const int64_t* numels, int count, int dtype,
                         void* flat, int64_t flat_capacity_elems, int64_t* offsets_out,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The inverse of pf_pack_factor_grads, for the step after the all-reduce of the flat buffer
 * (Section 4.1: one buffer is communicated per iteration; every factor then needs its own averaged
 * gradient back): tensor i receives flat[offsets_out[i] .. offsets_out[i] + numels[i]) bit for bit,
 * with the same tight offsets (prefix sums of numels, written to offsets_out before return).
 *   flat   device buffer of `flat_elems` elements (read only)
 *   grads  host array of `count` device pointers (element-aligned), the destinations
 * PF_ERR_WORKSPACE if the list is longer than flat_elems.  No workspace is needed. */
int pf_unpack_factor_grads(const void* flat, int64_t flat_elems, void* const* grads, const int64_t* numels,
                           int count, int dtype, int64_t* offsets_out,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PF_H_ */
