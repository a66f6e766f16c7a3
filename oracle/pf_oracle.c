/*
 * fp64 CPU oracle for low-rank pre-factorized layers.  TEST INFRASTRUCTURE ONLY:
 * it exists so that tests, the smoke check and the benchmark's CPU-baseline leg can
 * verify the CUDA library; no product code path may call it, and it shares no code
 * with the CUDA library.
 *
 * Every function is the plain definition written out as loops, in double precision,
 * with no blocking, fusion or reordering beyond the definition itself:
 *
 *   - factorized FC layer  y = (x U) V^T  (paper Section 2.1 and Appendix B "FC layer";
 *     row convention of Appendix B: U is the input-side k x r factor, V the output-side
 *     factor stored n x r),
 *   - its gradients by the chain rule on that formula (plain sums over rows, no 1/m),
 *   - factorized convolution: a k x k convolution into r channels followed by a 1 x 1
 *     convolution to c_out channels (Section 2.2 "Factorizing a convolution layer",
 *     Appendix B "Convolution layer"), read as cross-correlation with zero padding and
 *     nothing between the two convolutions,
 *   - flat gradient buffer: all gradient tensors copied back to back into one buffer
 *     (Section 4.1 "Implementation details and optimizations").
 *
 * Layouts: all matrices row-major and contiguous.  Conv tensors are NHWC; the thin
 * conv factor is U[kh][kw][C][R] (an (kh*kw*C) x R row-major matrix: the unrolled
 * matrix of Section 2.2 with rows ordered tap-major), V is [O][R].
 *
 * OpenMP only splits independent output rows across threads; each output element is
 * still one sequential sum in index order.
 */
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int pf_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* T[i,j] = sum_c x[i,c] U[c,j];   y[i,o] = sum_j T[i,j] V[o,j].   (Appendix B, FC layer) */
void pf_oracle_linear_fwd(const double* x, const double* U, const double* V,
                          long m, long k, long n, long r, double* T, double* y) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < m; ++i) {
        double* Ti = T + i * r;
        for (long j = 0; j < r; ++j) Ti[j] = 0.0;
        for (long c = 0; c < k; ++c) {
            const double xc = x[i * k + c];
            const double* Uc = U + c * r;
            for (long j = 0; j < r; ++j) Ti[j] += xc * Uc[j];
        }
        for (long o = 0; o < n; ++o) {
            const double* Vo = V + o * r;
            double acc = 0.0;
            for (long j = 0; j < r; ++j) acc += Ti[j] * Vo[j];
            y[i * n + o] = acc;
        }
    }
}

/* Chain rule on y = (xU)V^T with upstream gradient dY:
 *   G[i,j]  = sum_o dY[i,o] V[o,j]
 *   dX[i,c] = sum_j G[i,j] U[c,j]
 *   dU[c,j] = sum_i x[i,c] G[i,j]
 *   dV[o,j] = sum_i dY[i,o] T[i,j],  T = xU.
 * T must hold x U (as produced by pf_oracle_linear_fwd). */
void pf_oracle_linear_bwd(const double* x, const double* U, const double* V, const double* dY,
                          const double* T, long m, long k, long n, long r,
                          double* G, double* dX, double* dU, double* dV) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < m; ++i) {
        double* Gi = G + i * r;
        for (long j = 0; j < r; ++j) Gi[j] = 0.0;
        for (long o = 0; o < n; ++o) {
            const double d = dY[i * n + o];
            const double* Vo = V + o * r;
            for (long j = 0; j < r; ++j) Gi[j] += d * Vo[j];
        }
        for (long c = 0; c < k; ++c) {
            const double* Uc = U + c * r;
            double acc = 0.0;
            for (long j = 0; j < r; ++j) acc += Gi[j] * Uc[j];
            dX[i * k + c] = acc;
        }
    }
#pragma omp parallel for schedule(static)
    for (long c = 0; c < k; ++c) {
        double* dUc = dU + c * r;
        for (long j = 0; j < r; ++j) dUc[j] = 0.0;
        for (long i = 0; i < m; ++i) {
            const double xv = x[i * k + c];
            const double* Gi = G + i * r;
            for (long j = 0; j < r; ++j) dUc[j] += xv * Gi[j];
        }
    }
#pragma omp parallel for schedule(static)
    for (long o = 0; o < n; ++o) {
        double* dVo = dV + o * r;
        for (long j = 0; j < r; ++j) dVo[j] = 0.0;
        for (long i = 0; i < m; ++i) {
            const double d = dY[i * n + o];
            const double* Ti = T + i * r;
            for (long j = 0; j < r; ++j) dVo[j] += d * Ti[j];
        }
    }
}

/* T[n,ho,wo,j] = sum_{a,b,c} x[n, ho*st-pad+a, wo*st-pad+b, c] U[a,b,c,j]  (x = 0 outside),
 * y[n,ho,wo,o] = sum_j T[n,ho,wo,j] V[o,j].          (Section 2.2, Appendix B conv layer) */
void pf_oracle_conv_fwd(const double* x, const double* U, const double* V,
                        long N, long H, long W, long C, long R, long O,
                        long kh, long kw, long st, long pad, double* T, double* y) {
    const long Ho = (H + 2 * pad - kh) / st + 1;
    const long Wo = (W + 2 * pad - kw) / st + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (long nn = 0; nn < N; ++nn) {
        for (long ho = 0; ho < Ho; ++ho) {
            for (long wo = 0; wo < Wo; ++wo) {
                double* Tp = T + ((nn * Ho + ho) * Wo + wo) * R;
                for (long j = 0; j < R; ++j) Tp[j] = 0.0;
                for (long a = 0; a < kh; ++a) {
                    const long h = ho * st - pad + a;
                    if (h < 0 || h >= H) continue;
                    for (long b = 0; b < kw; ++b) {
                        const long w = wo * st - pad + b;
                        if (w < 0 || w >= W) continue;
                        const double* xp = x + ((nn * H + h) * W + w) * C;
                        for (long c = 0; c < C; ++c) {
                            const double xv = xp[c];
                            const double* Uc = U + ((a * kw + b) * C + c) * R;
                            for (long j = 0; j < R; ++j) Tp[j] += xv * Uc[j];
                        }
                    }
                }
                double* yp = y + ((nn * Ho + ho) * Wo + wo) * O;
                for (long o = 0; o < O; ++o) {
                    const double* Vo = V + o * R;
                    double acc = 0.0;
                    for (long j = 0; j < R; ++j) acc += Tp[j] * Vo[j];
                    yp[o] = acc;
                }
            }
        }
    }
}

/* Gradients of the factorized convolution (chain rule on pf_oracle_conv_fwd):
 *   dT[p,j]      = sum_o dY[p,o] V[o,j]                       (p = output pixel)
 *   dV[o,j]      = sum_p dY[p,o] T[p,j]
 *   dU[a,b,c,j]  = sum_{n,ho,wo} x[n,ho*st-pad+a,wo*st-pad+b,c] dT[n,ho,wo,j]
 *   dX[n,h,w,c]  = sum over (a,b,j) with ho=(h+pad-a)/st, wo=(w+pad-b)/st integral and in
 *                  range of dT[n,ho,wo,j] U[a,b,c,j].
 * T must hold the forward intermediate. */
void pf_oracle_conv_bwd(const double* x, const double* U, const double* V, const double* dY,
                        const double* T, long N, long H, long W, long C, long R, long O,
                        long kh, long kw, long st, long pad,
                        double* dT, double* dX, double* dU, double* dV) {
    const long Ho = (H + 2 * pad - kh) / st + 1;
    const long Wo = (W + 2 * pad - kw) / st + 1;
    const long P = N * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < P; ++p) {
        double* dTp = dT + p * R;
        for (long j = 0; j < R; ++j) dTp[j] = 0.0;
        for (long o = 0; o < O; ++o) {
            const double d = dY[p * O + o];
            const double* Vo = V + o * R;
            for (long j = 0; j < R; ++j) dTp[j] += d * Vo[j];
        }
    }
#pragma omp parallel for schedule(static)
    for (long o = 0; o < O; ++o) {
        double* dVo = dV + o * R;
        for (long j = 0; j < R; ++j) dVo[j] = 0.0;
        for (long p = 0; p < P; ++p) {
            const double d = dY[p * O + o];
            const double* Tp = T + p * R;
            for (long j = 0; j < R; ++j) dVo[j] += d * Tp[j];
        }
    }
#pragma omp parallel for schedule(static)
    for (long q = 0; q < kh * kw * C; ++q) {
        const long c = q % C;
        const long b = (q / C) % kw;
        const long a = q / (C * kw);
        double* dUq = dU + q * R;
        for (long j = 0; j < R; ++j) dUq[j] = 0.0;
        for (long nn = 0; nn < N; ++nn) {
            for (long ho = 0; ho < Ho; ++ho) {
                const long h = ho * st - pad + a;
                if (h < 0 || h >= H) continue;
                for (long wo = 0; wo < Wo; ++wo) {
                    const long w = wo * st - pad + b;
                    if (w < 0 || w >= W) continue;
                    const double xv = x[((nn * H + h) * W + w) * C + c];
                    const double* dTp = dT + ((nn * Ho + ho) * Wo + wo) * R;
                    for (long j = 0; j < R; ++j) dUq[j] += xv * dTp[j];
                }
            }
        }
    }
#pragma omp parallel for schedule(static) collapse(2)
    for (long nn = 0; nn < N; ++nn) {
        for (long h = 0; h < H; ++h) {
            for (long w = 0; w < W; ++w) {
                double* dXp = dX + ((nn * H + h) * W + w) * C;
                for (long c = 0; c < C; ++c) dXp[c] = 0.0;
                for (long a = 0; a < kh; ++a) {
                    const long hn = h + pad - a;
                    if (hn < 0 || hn % st != 0) continue;
                    const long ho = hn / st;
                    if (ho >= Ho) continue;
                    for (long b = 0; b < kw; ++b) {
                        const long wn = w + pad - b;
                        if (wn < 0 || wn % st != 0) continue;
                        const long wo = wn / st;
                        if (wo >= Wo) continue;
                        const double* dTp = dT + ((nn * Ho + ho) * Wo + wo) * R;
                        for (long c = 0; c < C; ++c) {
                            const double* Uc = U + ((a * kw + b) * C + c) * R;
                            double acc = 0.0;
                            for (long j = 0; j < R; ++j) acc += dTp[j] * Uc[j];
                            dXp[c] += acc;
                        }
                    }
                }
            }
        }
    }
}

/* Flat gradient buffer (Section 4.1): offsets[0] = 0, offsets[i+1] = offsets[i] + numel_i,
 * flat[offsets[i] + e] = grads_i[e] bit for bit; tight packing, caller's list order. */
void pf_oracle_pack(const void* const* grads, const long* numels, int count, int elem_bytes,
                    void* flat, long* offsets) {
    offsets[0] = 0;
    for (int i = 0; i < count; ++i) {
        const unsigned char* src = (const unsigned char*)grads[i];
        unsigned char* dst = (unsigned char*)flat + (size_t)offsets[i] * (size_t)elem_bytes;
        for (long e = 0; e < numels[i] * (long)elem_bytes; ++e) dst[e] = src[e];
        offsets[i + 1] = offsets[i] + numels[i];
    }
}
