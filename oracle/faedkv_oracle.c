/*
 * FAEDKV / IWDFT reference oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, float64 CPU statement of what the IWDFT hot path computes:
 * the pruned DFT of a K/V cache along the token axis, the per-token IWDFT
 * update, the pruned inverse DFT, and single-query softmax attention on the
 * reconstructed cache.  Every function is the textbook definition written out
 * as loops; there is no blocking, no fast transform, no recurrence for the
 * twiddles.  Phases are reduced exactly in 64-bit integers, m = (k*n) mod P,
 * before cos/sin are taken, so long sequences lose no accuracy.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call
 * this file.  It shares no code, header, table or constant with the CUDA path.
 * OpenMP pragmas only distribute independent output elements over cores; they
 * do not change any arithmetic or summation order of a single output.
 *
 * Notation: P = DFT grid size (the paper's N / N_DFT), bins[] = ascending
 * retained one-sided bin indices in [0, P/2], M = number of bins, d = channels
 * of one (batch, head) unit, t = tokens folded so far.
 *
 * Readings of the paper fixed here (each is tested by the oracle's pins):
 *  - state = start-referenced, unnormalised pruned DFT (Eq. 4); the
 *    IWDFT update adds x[t] * exp(-j*2*pi*k*t/P) (stationary-frame form of
 *    Eq. 9; the printed rotating-frame and running-mean recursions are
 *    kept below as cross-checks, never as the product's target);
 *  - real signals => one-sided bins with implied Hermitian mirror, weight
 *    w_k = 1 for k = 0 and k = P/2 (P even), else 2;
 *  - positions wrap modulo P; reconstruction length L = min(t, P).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

/* ------------------------------------------------------------------ helpers */

/* exact phase index (k*n) mod P in 64-bit integers */
static inline int64_t phase_index(int64_t k, int64_t n, int64_t P) {
    int64_t kk = k % P, nn = n % P;
    return (kk * nn) % P; /* kk, nn < 2^31  =>  product < 2^62 */
}

/* angle 2*pi*m/P of a reduced phase index */
static inline double phase_angle(int64_t m, int64_t P) {
    return 2.0 * M_PI * (double)m / (double)P;
}

/* Hermitian weight of a one-sided bin: the bin and its mirror P-k coincide for
 * k = 0 and, when P is even, k = P/2; otherwise the mirror doubles the term. */
double orc_weight(int P, int k) {
    if (k == 0) return 1.0;
    if ((P % 2 == 0) && (k == P / 2)) return 1.0;
    return 2.0;
}

/* ------------------------------------------------------------- plan / masks */

/* Retained-bin list of a one-sided mask (Eq. 6 as a keep-list):
 * ascending k in [0, P/2] with mask[k] != 0.  Returns M. */
int orc_plan(int P, const uint8_t *mask, int32_t *bins) {
    int M = 0;
    for (int k = 0; k <= P / 2; ++k)
        if (mask[k]) bins[M++] = k;
    return M;
}

/* Fold a two-sided mask over {0..P-1} (the paper's chunks partition the full
 * spectrum) onto one-sided bins: a one-sided bin is kept when either it or its
 * mirror is kept. */
void orc_fold_two_sided(int P, const uint8_t *mask2, uint8_t *mask1) {
    for (int k = 0; k <= P / 2; ++k) {
        int mirror = (P - k) % P;
        mask1[k] = (uint8_t)((mask2[k] != 0) || (mask2[mirror] != 0));
    }
}

/* Low-pass mask: bins 0..M-1. */
int orc_mask_lowpass(int P, int M, uint8_t *mask) {
    int n1 = P / 2 + 1;
    if (M < 0 || M > n1) return -1;
    for (int k = 0; k < n1; ++k) mask[k] = (uint8_t)(k < M);
    return 0;
}

/* Layer-wise mixed mask standing in for the per-layer top chunks of the
 * ablation study: chunks of 16 bins; the lowest n_low = floor(M/2 / 16) * 16
 * bins are always kept; the remaining (M - n_low)/16 chunks are drawn from
 * the chunks in [n_low/16, floor((P/2)/16)) by a Fisher-Yates shuffle driven
 * by a 64-bit LCG seeded from (seed, layer). */
int orc_mask_mixed(int P, int M, int layer, uint64_t seed, uint8_t *mask) {
    const int g = 16;
    int n1 = P / 2 + 1;
    if (M <= 0 || M % g != 0) return -1;
    int n_low = ((M / 2) / g) * g;
    int first = n_low / g;
    int end = (P / 2) / g; /* candidate chunks: first .. end-1 */
    int n_cand = end - first;
    int n_take = (M - n_low) / g;
    if (n_cand < n_take) return -1;
    memset(mask, 0, (size_t)n1);
    for (int k = 0; k < n_low; ++k) mask[k] = 1;
    int *cand = (int *)malloc(sizeof(int) * (size_t)(n_cand > 0 ? n_cand : 1));
    for (int i = 0; i < n_cand; ++i) cand[i] = first + i;
    uint64_t s = seed * 2654435761ULL + (uint64_t)layer;
    for (int i = 0; i < n_take; ++i) {
        s = s * 6364136223846793005ULL + 1442695040888963407ULL;
        uint64_t draw = s >> 33;
        int j = i + (int)(draw % (uint64_t)(n_cand - i));
        int tmp = cand[i]; cand[i] = cand[j]; cand[j] = tmp;
        for (int b = 0; b < g; ++b) mask[cand[i] * g + b] = 1;
    }
    free(cand);
    return 0;
}

/* ------------------------------------------------------ O2: pruned DFT (Eq. 4 + Eq. 6) */

/* C[k,c] = sum_{n<T} x[n,c] * exp(-j*2*pi*bins[k]*(pos0+n)/P), one unit.
 * x is [T][d]; Cre, Cim are [M][d].  pos0 is the position of x[0]. */
void orc_compress(const double *x, int T, int d, int P, const int32_t *bins, int M,
                  int64_t pos0, double *Cre, double *Cim) {
#pragma omp parallel for schedule(static)
    for (int ki = 0; ki < M; ++ki) {
        double *re = Cre + (size_t)ki * d, *im = Cim + (size_t)ki * d;
        for (int c = 0; c < d; ++c) { re[c] = 0.0; im[c] = 0.0; }
        for (int n = 0; n < T; ++n) {
            double a = phase_angle(phase_index(bins[ki], pos0 + n, P), P);
            double co = cos(a), si = sin(a);
            const double *xr = x + (size_t)n * d;
            for (int c = 0; c < d; ++c) {
                re[c] += xr[c] * co;
                im[c] -= xr[c] * si;
            }
        }
    }
}

/* The same over U independent units: x [U][T][d] -> C [U][M][d]. */
void orc_compress_units(const double *x, int U, int T, int d, int P, const int32_t *bins,
                        int M, int64_t pos0, double *Cre, double *Cim) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int u = 0; u < U; ++u)
        for (int ki = 0; ki < M; ++ki) {
            double *re = Cre + ((size_t)u * M + ki) * d, *im = Cim + ((size_t)u * M + ki) * d;
            for (int c = 0; c < d; ++c) { re[c] = 0.0; im[c] = 0.0; }
            for (int n = 0; n < T; ++n) {
                double a = phase_angle(phase_index(bins[ki], pos0 + n, P), P);
                double co = cos(a), si = sin(a);
                const double *xr = x + ((size_t)u * T + n) * d;
                for (int c = 0; c < d; ++c) {
                    re[c] += xr[c] * co;
                    im[c] -= xr[c] * si;
                }
            }
        }
}

/* ------------------------------------------------------ O3: IWDFT update (Eq. 9 / Eq. 12) */

/* Fold the token at position t into the retained coefficients with unit
 * weight: C[k,c] += x[c] * exp(-j*2*pi*bins[k]*t/P).  Only retained bins are
 * touched, which is "update all bins, then re-prune". */
void orc_append(double *Cre, double *Cim, int M, int d, int P, const int32_t *bins,
                int64_t t, const double *xnew) {
#pragma omp parallel for schedule(static)
    for (int ki = 0; ki < M; ++ki) {
        double a = phase_angle(phase_index(bins[ki], t, P), P);
        double co = cos(a), si = sin(a);
        for (int c = 0; c < d; ++c) {
            Cre[(size_t)ki * d + c] += xnew[c] * co;
            Cim[(size_t)ki * d + c] -= xnew[c] * si;
        }
    }
}

/* ------------------------------------------------------ O4: pruned inverse DFT (Eq. 5 on retained bins) */

/* out[n,c] = (1/P) * sum_k w_k * (Re C[k,c]*cos(2*pi*k*n/P) - Im C[k,c]*sin(2*pi*k*n/P)),
 * n < L.  This is Eq. 5 with every pruned bin zero and the mirror
 * bins P-k supplied by conjugate symmetry of a real signal. */
void orc_reconstruct(const double *Cre, const double *Cim, int M, int d, int P,
                     const int32_t *bins, int L, double *out) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < L; ++n) {
        double *o = out + (size_t)n * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int ki = 0; ki < M; ++ki) {
            double a = phase_angle(phase_index(bins[ki], n, P), P);
            double w = orc_weight(P, bins[ki]);
            double co = w * cos(a), si = w * sin(a);
            const double *re = Cre + (size_t)ki * d, *im = Cim + (size_t)ki * d;
            for (int c = 0; c < d; ++c) o[c] += re[c] * co - im[c] * si;
        }
        for (int c = 0; c < d; ++c) o[c] /= (double)P;
    }
}

/* The same sum at the listed positions only: out[i,c] = xtilde[rows[i], c].  (Eq. 5 on the retained bins,
 * position by position; lets a caller check single rows of a long reconstruction.) */
void orc_reconstruct_rows(const double *Cre, const double *Cim, int M, int d, int P,
                          const int32_t *bins, const int32_t *rows, int n_rows, double *out) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n_rows; ++i) {
        const int64_t n = rows[i];
        double *o = out + (size_t)i * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int ki = 0; ki < M; ++ki) {
            double a = phase_angle(phase_index(bins[ki], n, P), P);
            double w = orc_weight(P, bins[ki]);
            double co = w * cos(a), si = w * sin(a);
            const double *re = Cre + (size_t)ki * d, *im = Cim + (size_t)ki * d;
            for (int c = 0; c < d; ++c) o[c] += re[c] * co - im[c] * si;
        }
        for (int c = 0; c < d; ++c) o[c] /= (double)P;
    }
}

/* ------------------------------------------------------ O5: decode attention (Eq. 3 on Eq. 11) */

/* Textbook single-query attention on the materialised reconstruction:
 * out[g,:] = softmax_n(scale * q[g,:] . Ktilde[n,:]) * Vtilde.  q is [G][d]
 * for the G query heads that share this kv head.  Ktilde, Vtilde are [L][d]. */
void orc_attention_dense(const double *q, int G, const double *Kt, const double *Vt,
                         int L, int d, double scale, double *out) {
    double *s = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
    for (int g = 0; g < G; ++g) {
        double mx = -INFINITY;
        for (int n = 0; n < L; ++n) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += q[(size_t)g * d + c] * Kt[(size_t)n * d + c];
            s[n] = acc * scale;
            if (s[n] > mx) mx = s[n];
        }
        double den = 0.0;
        for (int n = 0; n < L; ++n) { s[n] = exp(s[n] - mx); den += s[n]; }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int n = 0; n < L; ++n) acc += s[n] * Vt[(size_t)n * d + c];
            /* L = 0: Eq. 3 sums over no token at all; the empty sum is read as the zero vector */
            out[(size_t)g * d + c] = L > 0 ? acc / den : 0.0;
        }
    }
    free(s);
}

/* Reconstruct K and V of one kv head, then attend. */
void orc_decode_attn(const double *q, int G, const double *CKre, const double *CKim,
                     const double *CVre, const double *CVim, int M, int d, int P,
                     const int32_t *bins, int L, double scale, double *out) {
    double *Kt = (double *)malloc(sizeof(double) * (size_t)L * d);
    double *Vt = (double *)malloc(sizeof(double) * (size_t)L * d);
    orc_reconstruct(CKre, CKim, M, d, P, bins, L, Kt);
    orc_reconstruct(CVre, CVim, M, d, P, bins, L, Vt);
    orc_attention_dense(q, G, Kt, Vt, L, d, scale, out);
    free(Kt);
    free(Vt);
}

/* ------------------------------------------------------ printed recursions, kept as cross-checks only */

/* Eq. 9 with the normalisation dropped, literally: R <- W_k * (R + x),
 * W_k = exp(-j*2*pi*k/P).  (Rotating-frame state.) */
void orc_rotating_frame_step(double *Rre, double *Rim, int M, int d, int P,
                             const int32_t *bins, const double *xnew) {
    for (int ki = 0; ki < M; ++ki) {
        double a = phase_angle(bins[ki] % P, P);
        double wr = cos(a), wi = -sin(a);
        for (int c = 0; c < d; ++c) {
            double ar = Rre[(size_t)ki * d + c] + xnew[c];
            double ai = Rim[(size_t)ki * d + c];
            Rre[(size_t)ki * d + c] = wr * ar - wi * ai;
            Rim[(size_t)ki * d + c] = wr * ai + wi * ar;
        }
    }
}

/* Eq. 8 literally: S <- W_k * (S - x_out + x_in). */
void orc_sliding_window_step(double *Sre, double *Sim, int M, int d, int P,
                             const int32_t *bins, const double *x_out, const double *x_in) {
    for (int ki = 0; ki < M; ++ki) {
        double a = phase_angle(bins[ki] % P, P);
        double wr = cos(a), wi = -sin(a);
        for (int c = 0; c < d; ++c) {
            double ar = Sre[(size_t)ki * d + c] - x_out[c] + x_in[c];
            double ai = Sim[(size_t)ki * d + c];
            Sre[(size_t)ki * d + c] = wr * ar - wi * ai;
            Sim[(size_t)ki * d + c] = wr * ai + wi * ar;
        }
    }
}

/* Eq. 9's normalisation with the exact factors, in the stationary
 * frame: S_{t+1} = (t/(t+1)) * S_t + x * exp(-j*2*pi*k*t/P) / (t+1), so that
 * S_t = C_t / t (a running mean).  t is the token count before the step. */
void orc_running_mean_step(double *Sre, double *Sim, int M, int d, int P,
                           const int32_t *bins, int64_t t, const double *xnew) {
    double keep = (double)t / (double)(t + 1), add = 1.0 / (double)(t + 1);
    for (int ki = 0; ki < M; ++ki) {
        double a = phase_angle(phase_index(bins[ki], t, P), P);
        double co = cos(a), si = sin(a);
        for (int c = 0; c < d; ++c) {
            Sre[(size_t)ki * d + c] = keep * Sre[(size_t)ki * d + c] + add * xnew[c] * co;
            Sim[(size_t)ki * d + c] = keep * Sim[(size_t)ki * d + c] - add * xnew[c] * si;
        }
    }
}
