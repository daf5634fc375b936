/*
 * CPU oracle for the SCAP activation-pruned fully-connected layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of
 * what the path computes, written from the paper's definitions.  It shares no code, header,
 * table or helper with the CUDA library and must never be linked into or called from it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * Conventions (paper notation in brackets):
 *   K  input channels  [IC]      N  output channels [OC]      B  batch rows [N in Eq. 1]
 *   x[B,K]  row-major activations, stored fp16 or bf16 (16-bit patterns), or fp32 ("xf")
 *   W[K,N]  row-major, row k = all outputs of input channel k   [W in R^{IC x OC}, Eq. 1]
 *   m[K]    per-channel mode (binary32); the paper's scalar eta is the constant vector [Eq. 4-6]
 *   tau     pruning threshold (binary32)                                       [Eq. 2]
 * Floating point: the keep/drop decision is taken in binary32 with one subtraction and one
 * compare, exactly as written below; every sum is accumulated in binary64 in ascending k.
 * Build with -O2 -ffp-contract=off (no fused multiply-add, no fast-math).
 *
 * Pins: every function here is pinned by the CPU tests (closed forms, brute force on tiny
 * inputs, textbook special cases, library quantile/matmul cross-checks, the paper's printed
 * FFN-sparsity rows) EXCEPT the following, which are "parity unpinned" because the paper
 * prints nothing that fixes them:
 *   - the accuracy of the histogram mode estimator (its definition is pinned on hand-built cases
 *     and against a library histogram on samples away from bin edges);
 *   - the mixture-of-experts router convention (softmax, top-k, renormalise, ties to lower index).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SCAP_ORACLE_F16 0
#define SCAP_ORACLE_BF16 1

/* ---------------------------------------------------------------- storage widening (exact) */

static float widen_bf16(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static float widen_f16(uint16_t h) {
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    int32_t e = (h >> 10) & 0x1f;
    uint32_t frac = h & 0x3ffu;
    double v;
    if (e == 0) {
        v = ldexp((double)frac, -24); /* subnormal: frac * 2^-10 * 2^-14 */
    } else if (e == 31) {
        v = frac ? NAN : INFINITY;
    } else {
        v = ldexp(1.0 + (double)frac / 1024.0, e - 15);
    }
    return (float)(sign ? -v : v); /* every fp16 value is exactly representable in binary32 */
}

float scap_oracle_widen(uint16_t bits, int dt) { return dt == SCAP_ORACLE_F16 ? widen_f16(bits) : widen_bf16(bits); }

void scap_oracle_widen_array(const uint16_t *bits, int dt, long n, float *out) {
    for (long i = 0; i < n; ++i) out[i] = scap_oracle_widen(bits[i], dt);
}

/* ---------------------------------------------------------------- Eq. 2 / Alg. 3: centre + threshold
 * d = xf - m[k]  (one binary32 subtraction);  keep iff |d| >= tau  (Alg. 2/3 use >=; a NaN compares
 * false and is dropped).  m == NULL means no centring.  Outputs (any may be NULL):
 *   keep[B,K]  per-element decision;   d_out[B,K] the centred value (not zeroed);
 *   U[K] = OR over rows (the channels whose weight row must be fetched for this batch);
 *   idx = ascending list of k with U[k];  returns nnz = |idx|.                                  */
int scap_oracle_mask(const float *xf, const float *m, float tau, int B, int K,
                     uint8_t *keep, float *d_out, uint8_t *U, uint32_t *idx) {
    int nnz = 0;
    for (int k = 0; k < K; ++k) {
        int any = 0;
        for (int b = 0; b < B; ++b) {
            float x = xf[(long)b * K + k];
            volatile float d = m ? x - m[k] : x;
            int kp = (fabsf(d) >= tau) ? 1 : 0;
            if (keep) keep[(long)b * K + k] = (uint8_t)kp;
            if (d_out) d_out[(long)b * K + k] = d;
            any |= kp;
        }
        if (U) U[k] = (uint8_t)any;
        if (any) {
            if (idx) idx[nnz] = (uint32_t)k;
            ++nnz;
        }
    }
    return nnz;
}

/* ---------------------------------------------------------------- Eq. 3 / Alg. 3: sparse FC
 * y[b,n] = b_fused[n] + sum_k keep[b,k] * (xf[b,k] - m[k]) * W[k,n], ascending k, binary64.
 * Pruning is per element (Eq. 2 is written over X_ij): a row whose own |x'| < tau contributes
 * nothing for that channel even when another row of the batch kept it.
 * The product uses the exact real difference of the two binary32 operands (computed in
 * binary64, where it is exact up to one rounding), not the rounded binary32 d.             */
void scap_oracle_sparse_fc(const float *xf, const uint16_t *W, int dt, const float *m, float tau,
                           const float *b_fused, int B, int K, int N, double *y) {
    uint8_t *keep = (uint8_t *)malloc((size_t)B * K);
    scap_oracle_mask(xf, m, tau, B, K, keep, NULL, NULL, NULL);
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < N; ++n) y[(long)b * N + n] = b_fused ? (double)b_fused[n] : 0.0;
    for (int k = 0; k < K; ++k) {
        for (int b = 0; b < B; ++b) {
            if (!keep[(long)b * K + k]) continue;
            double xc = (double)xf[(long)b * K + k] - (m ? (double)m[k] : 0.0);
            const uint16_t *wr = W + (long)k * N;
            double *yr = y + (long)b * N;
            for (int n = 0; n < N; ++n) yr[n] += xc * (double)scap_oracle_widen(wr[n], dt);
        }
    }
    free(keep);
}

/* Same sum restricted to output columns [n0, n1): lets a caller spread columns over threads or
 * sample a few columns of a large layer.  y has B rows of (n1 - n0) entries.                */
void scap_oracle_sparse_fc_cols(const float *xf, const uint16_t *W, int dt, const float *m, float tau,
                                const float *b_fused, int B, int K, int N, int n0, int n1, double *y) {
    int w = n1 - n0;
    uint8_t *keep = (uint8_t *)malloc((size_t)B * K);
    scap_oracle_mask(xf, m, tau, B, K, keep, NULL, NULL, NULL);
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < w; ++n) y[(long)b * w + n] = b_fused ? (double)b_fused[n0 + n] : 0.0;
    for (int k = 0; k < K; ++k) {
        for (int b = 0; b < B; ++b) {
            if (!keep[(long)b * K + k]) continue;
            double xc = (double)xf[(long)b * K + k] - (m ? (double)m[k] : 0.0);
            const uint16_t *wr = W + (long)k * N + n0;
            double *yr = y + (long)b * w;
            for (int n = 0; n < w; ++n) yr[n] += xc * (double)scap_oracle_widen(wr[n], dt);
        }
    }
    free(keep);
}

/* ---------------------------------------------------------------- Eq. 1: dense FC, y = xW + b */
void scap_oracle_dense_fc(const float *xf, const uint16_t *W, int dt, const float *b,
                          int B, int K, int N, double *y) {
    for (int bb = 0; bb < B; ++bb)
        for (int n = 0; n < N; ++n) y[(long)bb * N + n] = b ? (double)b[n] : 0.0;
    for (int k = 0; k < K; ++k)
        for (int bb = 0; bb < B; ++bb) {
            double xv = (double)xf[(long)bb * K + k];
            const uint16_t *wr = W + (long)k * N;
            double *yr = y + (long)bb * N;
            for (int n = 0; n < N; ++n) yr[n] += xv * (double)scap_oracle_widen(wr[n], dt);
        }
}

/* ---------------------------------------------------------------- Eq. 5-6: b_fused = b + m W
 * b is in the storage dtype (nullable = zero bias).  Result in binary64.                    */
void scap_oracle_fold_bias(const uint16_t *W, int dt, const float *m, const uint16_t *b,
                           int K, int N, double *b_fused) {
    for (int n = 0; n < N; ++n) b_fused[n] = b ? (double)scap_oracle_widen(b[n], dt) : 0.0;
    for (int k = 0; k < K; ++k) {
        double mk = (double)m[k];
        const uint16_t *wr = W + (long)k * N;
        for (int n = 0; n < N; ++n) b_fused[n] += mk * (double)scap_oracle_widen(wr[n], dt);
    }
}

/* ---------------------------------------------------------------- mode by histogram arg-max
 * The paper estimates the mode offline from a density estimate and reads off its peak
 * (Section 3, "Determination of mode value"); the estimator here is a fixed-width histogram
 * per channel.  All arithmetic is binary32, each operation rounded separately:
 *   lo = min_t x, hi = max_t x;  hi == lo -> m = lo.
 *   scale = nbins / (hi - lo);  bin(x) = min(nbins-1, floor((x - lo) * scale));
 *   i* = lowest bin with the largest count;  w = (hi - lo) * (1/nbins);  m = lo + (i* + 0.5) * w. */
void scap_oracle_mode(const float *xf /*[T,K]*/, int T, int K, int nbins, float *m_out) {
    int *cnt = (int *)malloc(sizeof(int) * (size_t)nbins);
    for (int k = 0; k < K; ++k) {
        float lo = xf[k], hi = xf[k];
        for (int t = 1; t < T; ++t) {
            float v = xf[(long)t * K + k];
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
        if (hi == lo) {
            m_out[k] = lo;
            continue;
        }
        volatile float range = hi - lo;
        volatile float scale = (float)nbins / range;
        memset(cnt, 0, sizeof(int) * (size_t)nbins);
        for (int t = 0; t < T; ++t) {
            volatile float off = xf[(long)t * K + k] - lo;
            volatile float pos = off * scale;
            int i = (int)floorf(pos);
            if (i > nbins - 1) i = nbins - 1;
            if (i < 0) i = 0;
            cnt[i]++;
        }
        int best = 0;
        for (int i = 1; i < nbins; ++i)
            if (cnt[i] > cnt[best]) best = i;
        volatile float inv = 1.0f / (float)nbins;
        volatile float w = range * inv;
        volatile float c = (float)best + 0.5f;
        volatile float step = c * w;
        volatile float mm = lo + step;
        m_out[k] = mm;
    }
    free(cnt);
}

/* ---------------------------------------------------------------- Eq. 2: tau = Quantile(|X - m|, s)
 * Importance is pooled over the whole calibration tensor of this FC input: v = sorted
 * |xf[t,k] - m[k]| (binary32 subtraction as in scap_oracle_mask), M = T*K values.
 * Linear-interpolation quantile: pos = s (M-1), j = floor(pos), f = pos - j,
 * tau = v[j] + f (v[j+1] - v[j]) in binary64, rounded once to binary32.  s <= 0 -> tau = 0.   */
static int cmp_float(const void *a, const void *b) {
    float x = *(const float *)a, y = *(const float *)b;
    return (x > y) - (x < y);
}

/* ---------------------------------------------------------------- mode by mean or median
 * Section 3 ("Determination of mode value"): a fast estimate of the mode is the empirical mean or
 * the median of the calibration activations.  Per channel k:
 *   mean:    m[k] = ( sum_{t = 0 .. T-1, in this order} x[t,k] ) / T   in binary64, rounded once to binary32;
 *   median:  v = the column sorted ascending, m[k] = ( v[(T-1)/2] + v[T/2] ) / 2 in binary64, rounded once
 *            (the middle value for odd T, the mean of the two middle values for even T).
 * A result of -0 is returned as +0.                                                             */
void scap_oracle_mean(const float *xf /*[T,K]*/, int T, int K, float *m_out) {
    for (int k = 0; k < K; ++k) {
        double acc = 0.0;
        for (int t = 0; t < T; ++t) acc += (double)xf[(long)t * K + k];
        m_out[k] = (float)(acc / (double)T) + 0.0f;
    }
}

void scap_oracle_median(const float *xf /*[T,K]*/, int T, int K, float *m_out) {
    float *v = (float *)malloc(sizeof(float) * (size_t)T);
    for (int k = 0; k < K; ++k) {
        for (int t = 0; t < T; ++t) v[t] = xf[(long)t * K + k];
        qsort(v, (size_t)T, sizeof(float), cmp_float);
        volatile double mid = ((double)v[(T - 1) / 2] + (double)v[T / 2]) / 2.0;
        m_out[k] = (float)mid + 0.0f;
    }
    free(v);
}

/* Mode as the peak of a kernel density estimate (Section 3, "Determination of mode value", names KDE next to the
 * mean and the median and leaves its parameters to a statistics package).  Reading taken, per channel, all in
 * binary64: Gaussian kernel; bandwidth h = sigma * T^(-1/5) (Scott's rule) with sigma the sample standard
 * deviation (divisor T - 1) about the mean, both summed in row order; the density is evaluated on G points
 * g_i = lo + i (hi - lo) / (G - 1), i = 0 .. G-1, between the channel's smallest and largest value,
 *   dens_i = sum_t exp( -((g_i - x_t) / h)^2 / 2 )      (the common factor 1 / (T h sqrt(2 pi)) is left out),
 * and the mode is the first g_i of largest density, rounded once to binary32.  A constant channel returns its
 * constant.  dens_out (optional) receives the G densities of channel k_dens.                           */
void scap_oracle_kde(const float *xf /*[T,K]*/, int T, int K, int G, float *m_out, int k_dens, double *dens_out /*[G] or NULL*/) {
    for (int k = 0; k < K; ++k) {
        float lo = xf[k], hi = xf[k];
        double sum = 0.0;
        for (int t = 0; t < T; ++t) {
            const float v = xf[(long)t * K + k];
            if (v < lo) lo = v;
            if (v > hi) hi = v;
            sum += (double)v;
        }
        if (hi == lo) {
            m_out[k] = lo + 0.0f;
            if (dens_out && k == k_dens) for (int i = 0; i < G; ++i) dens_out[i] = (double)T;
            continue;
        }
        const double mu = sum / (double)T;
        double ss = 0.0;
        for (int t = 0; t < T; ++t) {
            const double d = (double)xf[(long)t * K + k] - mu;
            ss += d * d;
        }
        const double sigma = sqrt(ss / (double)(T - 1));
        const double h = sigma * pow((double)T, -0.2);
        const double step = ((double)hi - (double)lo) / (double)(G - 1);
        double best = -1.0;
        int best_i = 0;
        for (int i = 0; i < G; ++i) {
            const double g = (double)lo + (double)i * step;
            double dens = 0.0;
            for (int t = 0; t < T; ++t) {
                const double u = (g - (double)xf[(long)t * K + k]) / h;
                dens += exp(-0.5 * (u * u));
            }
            if (dens_out && k == k_dens) dens_out[i] = dens;
            if (dens > best) { best = dens; best_i = i; }
        }
        m_out[k] = (float)((double)lo + (double)best_i * step) + 0.0f;
    }
}

/* Scalar eta for the whole FC input (the paper's eta is one scalar per layer), from all T*K values:
 *   mean:    the per-channel sums above (each over t in order), added over k = 0 .. K-1 in this order in
 *            binary64, divided by T*K, rounded once to binary32;
 *   median and histogram mode: the per-channel definitions applied to the tensor read as one channel of
 *            T*K values (callers pass T*K, 1).                                                   */
float scap_oracle_eta_mean(const float *xf /*[T,K]*/, int T, int K) {
    double total = 0.0;
    for (int k = 0; k < K; ++k) {
        double acc = 0.0;
        for (int t = 0; t < T; ++t) acc += (double)xf[(long)t * K + k];
        total += acc;
    }
    return (float)(total / ((double)T * (double)K)) + 0.0f;
}

float scap_oracle_tau(const float *xf /*[T,K]*/, int T, int K, const float *m, double s,
                      float *vj_out, float *vj1_out) {
    long M = (long)T * K;
    if (vj_out) *vj_out = 0.0f;
    if (vj1_out) *vj1_out = 0.0f;
    if (s <= 0.0 || M <= 0) return 0.0f;
    float *v = (float *)malloc(sizeof(float) * (size_t)M);
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < K; ++k) {
            volatile float d = m ? xf[(long)t * K + k] - m[k] : xf[(long)t * K + k];
            v[(long)t * K + k] = fabsf(d);
        }
    qsort(v, (size_t)M, sizeof(float), cmp_float);
    double pos = s * (double)(M - 1);
    long j = (long)floor(pos);
    if (j > M - 1) j = M - 1;
    double f = pos - (double)j;
    long j1 = j + 1 < M ? j + 1 : M - 1;
    volatile double diff = (double)v[j1] - (double)v[j];
    volatile double prod = f * diff;
    volatile double t64 = (double)v[j] + prod;
    if (vj_out) *vj_out = v[j];
    if (vj1_out) *vj1_out = v[j1];
    free(v);
    return (float)t64;
}

/* ---------------------------------------------------------------- 8-bit weights (Table 4 applies SCAP to 8-bit models)
 * Storage reading: Wq[K,N] signed 8-bit, one binary32 scale per input channel, W[k,n] = scale[k] * Wq[k,n]
 * (symmetric, no zero point).  The sparse FC and the bias folding are Eq. 2-3 and Eq. 5-6 on that W, in binary64. */
void scap_oracle_sparse_fc_q8(const float *xf, const signed char *Wq, const float *scale, const float *m, float tau,
                              const float *b_fused, int B, int K, int N, double *y) {
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < N; ++n) {
            double acc = b_fused ? (double)b_fused[n] : 0.0;
            for (int k = 0; k < K; ++k) {
                volatile float d = m ? xf[(long)b * K + k] - m[k] : xf[(long)b * K + k];   /* the decision: binary32 */
                double xc = (double)xf[(long)b * K + k] - (m ? (double)m[k] : 0.0);      /* the product: exact difference */
                if (fabsf(d) >= tau) acc += xc * ((double)scale[k] * (double)Wq[(long)k * N + n]);
            }
            y[(long)b * N + n] = acc;
        }
}

void scap_oracle_fold_bias_q8(const signed char *Wq, const float *scale, const float *m, const float *b /*[N] nullable*/,
                              int K, int N, double *b_fused) {
    for (int n = 0; n < N; ++n) {
        double acc = b ? (double)b[n] : 0.0;
        for (int k = 0; k < K; ++k) acc += (double)m[k] * ((double)scale[k] * (double)Wq[(long)k * N + n]);
        b_fused[n] = acc;
    }
}

/* ---------------------------------------------------------------- group-wise 4-bit weights (Table 4: the AWQ rows)
 * Storage reading (the paper names the models, not a layout): unsigned 4-bit codes q[k,n] in 0..15, two per byte in
 * Wq[K, N/2] (row-major like W; column 2j in the low nibble of byte j, column 2j+1 in the high nibble); groups of
 * `group` consecutive INPUT channels share, per output column, one binary32 scale and one zero point in 0..15:
 *     W[k,n] = scale[k / group, n] * (q[k,n] - zero[k / group, n]).
 * The sparse FC and the bias folding are Eq. 2-3 and Eq. 5-6 on that W, in binary64, ascending k.            */
static double q4_weight(const uint8_t *Wq, const float *scale, const uint8_t *zero, int N, int group, int k, int n) {
    const uint8_t byte = Wq[(long)k * (N / 2) + n / 2];
    const int q = (n & 1) ? (byte >> 4) : (byte & 15);
    const long g = k / group;
    return (double)scale[g * N + n] * (double)(q - (int)zero[g * N + n]);
}

void scap_oracle_sparse_fc_q4(const float *xf, const uint8_t *Wq, const float *scale, const uint8_t *zero, int group,
                              const float *m, float tau, const float *b_fused, int B, int K, int N, double *y) {
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < N; ++n) {
            double acc = b_fused ? (double)b_fused[n] : 0.0;
            for (int k = 0; k < K; ++k) {
                volatile float d = m ? xf[(long)b * K + k] - m[k] : xf[(long)b * K + k];   /* the decision: binary32 */
                double xc = (double)xf[(long)b * K + k] - (m ? (double)m[k] : 0.0);      /* the product: exact difference */
                if (fabsf(d) >= tau) acc += xc * q4_weight(Wq, scale, zero, N, group, k, n);
            }
            y[(long)b * N + n] = acc;
        }
}

void scap_oracle_fold_bias_q4(const uint8_t *Wq, const float *scale, const uint8_t *zero, int group, const float *m,
                              const float *b /*[N] nullable*/, int K, int N, double *b_fused) {
    for (int n = 0; n < N; ++n) {
        double acc = b ? (double)b[n] : 0.0;
        for (int k = 0; k < K; ++k) acc += (double)m[k] * q4_weight(Wq, scale, zero, N, group, k, n);
        b_fused[n] = acc;
    }
}

/* ---------------------------------------------------------------- Alg. 2: SwiGLU block
 * Wgu[D,2F]: columns 0..F-1 are the gate projection, F..2F-1 the up projection; both read the
 * same pruned input (one tau_x, one mask).  z = up * silu(gate), silu(g) = g / (1 + exp(-g)),
 * in binary64.  The down projection reads z stored as binary32 (z32) and prunes it with
 * (m2, tau2).  If z_in is non-NULL it replaces the computed z32 (teacher forcing for a
 * stage-wise comparison).  Outputs: y[B,D] binary64; z_out[B,F] binary32 (nullable).        */
void scap_oracle_glu_ffn(const float *hf /*[B,D]*/, const uint16_t *Wgu, const uint16_t *Wd, int dt,
                         const float *m1, float tau1, const float *bgu_fused /*[2F] nullable*/,
                         const float *m2, float tau2, const float *bd_fused /*[D] nullable*/,
                         int B, int D, int F, const float *z_in, double *y, float *z_out) {
    float *z32 = (float *)malloc(sizeof(float) * (size_t)B * F);
    if (z_in) {
        memcpy(z32, z_in, sizeof(float) * (size_t)B * F);
    } else {
        double *gu = (double *)malloc(sizeof(double) * (size_t)B * 2 * F);
        scap_oracle_sparse_fc(hf, Wgu, dt, m1, tau1, bgu_fused, B, D, 2 * F, gu);
        for (int b = 0; b < B; ++b)
            for (int f = 0; f < F; ++f) {
                double g = gu[(long)b * 2 * F + f];
                double u = gu[(long)b * 2 * F + F + f];
                double z = u * (g / (1.0 + exp(-g)));
                z32[(long)b * F + f] = (float)z;
            }
        free(gu);
    }
    if (z_out) memcpy(z_out, z32, sizeof(float) * (size_t)B * F);
    scap_oracle_sparse_fc(z32, Wd, dt, m2, tau2, bd_fused, B, F, D, y);
    free(z32);
}

/* ---------------------------------------------------------------- non-GLU FFN (Section 4.3, ablation of mode centring)
 * Falcon / MPT-style block: u = sparse_fc(h; Wu, m1, tau1, bu_fused) [B,F]; z = gelu(u) with the exact
 * GELU, gelu(v) = v/2 (1 + erf(v / sqrt 2)), in binary64; the down projection reads z stored as binary32
 * and prunes it with (m2, tau2) - the input whose mode centring the paper's ablation is about.  z_in, if
 * non-NULL, replaces the computed z (teacher forcing for a stage-wise comparison).                     */
void scap_oracle_gelu_ffn(const float *hf /*[B,D]*/, const uint16_t *Wu /*[D,F]*/, const uint16_t *Wd /*[F,D]*/, int dt,
                          const float *m1, float tau1, const float *bu_fused /*[F] nullable*/,
                          const float *m2, float tau2, const float *bd_fused /*[D] nullable*/,
                          int B, int D, int F, const float *z_in, double *y, float *z_out) {
    float *z32 = (float *)malloc(sizeof(float) * (size_t)B * F);
    if (z_in) {
        memcpy(z32, z_in, sizeof(float) * (size_t)B * F);
    } else {
        double *u = (double *)malloc(sizeof(double) * (size_t)B * F);
        scap_oracle_sparse_fc(hf, Wu, dt, m1, tau1, bu_fused, B, D, F, u);
        for (long i = 0; i < (long)B * F; ++i) z32[i] = (float)(0.5 * u[i] * (1.0 + erf(u[i] / sqrt(2.0))));
        free(u);
    }
    if (z_out) memcpy(z_out, z32, sizeof(float) * (size_t)B * F);
    scap_oracle_sparse_fc(z32, Wd, dt, m2, tau2, bd_fused, B, F, D, y);
    free(z32);
}

/* ---------------------------------------------------------------- MoE router (convention: see header)
 * p = softmax(logits[b, 0..E-1]) in binary64; the top_k largest p (ties -> lower index) are
 * selected and their weights renormalised to sum to one.                                     */
void scap_oracle_router(const float *logits /*[B,E]*/, int B, int E, int top_k,
                        int *expert_out /*[B,top_k]*/, double *weight_out /*[B,top_k]*/) {
    double *p = (double *)malloc(sizeof(double) * (size_t)E);
    uint8_t *used = (uint8_t *)malloc((size_t)E);
    for (int b = 0; b < B; ++b) {
        double mx = -INFINITY, sum = 0.0;
        for (int e = 0; e < E; ++e)
            if ((double)logits[(long)b * E + e] > mx) mx = (double)logits[(long)b * E + e];
        for (int e = 0; e < E; ++e) {
            p[e] = exp((double)logits[(long)b * E + e] - mx);
            sum += p[e];
        }
        for (int e = 0; e < E; ++e) p[e] /= sum;
        memset(used, 0, (size_t)E);
        double tot = 0.0;
        for (int j = 0; j < top_k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!used[e] && (best < 0 || p[e] > p[best])) best = e;
            used[best] = 1;
            expert_out[(long)b * top_k + j] = best;
            weight_out[(long)b * top_k + j] = p[best];
            tot += p[best];
        }
        for (int j = 0; j < top_k; ++j) weight_out[(long)b * top_k + j] /= tot;
    }
    free(p);
    free(used);
}

/* ---------------------------------------------------------------- Section B: FFN sparsity accounting
 * A SwiGLU FFN has three equal-size FCs, so its sparsity is the mean of the three input
 * sparsities: (s_up + s_gate + s_down) / 3 (= 2/3 s_x + 1/3 s_gated when up and gate share s_x). */
double scap_oracle_ffn_sparsity(double s_up, double s_gate, double s_down) {
    return (s_up + s_gate + s_down) / 3.0;
}
