/*
 * CPU oracle for the CDL quantized layer ("Coded Deep Learning: Framework and
 * Algorithm", arXiv 2501.09849).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, direct
 * transcription of the paper's definitions in double precision.  Nothing in it
 * is blocked, fused, windowed by shortcut or reordered, so that each function
 * can be checked against the cited equation by eye.  It shares no code with
 * the CUDA library; only tests, the smoke check and the benchmark's CPU
 * baseline call it.  The "omp parallel for" lines split independent elements
 * (or output rows) over host threads and change no arithmetic.
 *
 * Notation (Sec. IV-A, V-A): theta is a weight or an activation; the index set
 * is {lo, ..., hi} (the paper's A = {-2^(b-1)..2^(b-1)-1} for weights and
 * B = {0..2^b-1} for activations are instances); the reproduction alphabet is
 * {i*q}; alpha > 0 is the CPMF parameter (beta for activations).
 *
 * Readings of points the paper leaves open (each is listed in the design
 * notes of the repository as well):
 *  - hard index: the uniform quantizer Q_u (Remark of Sec. IV-A, end of
 *    Sec. IV-B) evaluated as clamp(round-half-even(theta / q), lo, hi) with the
 *    quotient taken in IEEE binary32, because an integer decision needs one
 *    arithmetic definition shared by every implementation.
 *  - truncated activation CPMF (Sec. VI-B.1, five entries kept): keep the
 *    `window` largest CPMF entries (equal entries: the lower index first), set
 *    the rest to 0, renormalise.
 *  - entropy is in bits (log base 2), Sec. V-C speaks of bits per weight.
 *  - d Q_d / d alpha is not printed; it is derived with the steps of
 *    Appendix B:  dP_i/dalpha = P_i ( -(theta-iq)^2 + sum_j P_j (theta-jq)^2 )
 *    so  dQ_d/dalpha = -Cov(X, (theta-X)^2) = 2 theta Var{X} - Skew_u{X}.
 *  - derivative of the total bits n*H w.r.t. theta (Sec. V-D states that it
 *    has a closed form without printing it): with level probabilities pbar
 *    held as given,
 *    d(nH)/dtheta = - sum_k dP_k/dtheta log2 pbar_k and, from Appendix B,
 *    dP_k/dtheta = 2 alpha P_k (kq - Q_d).  log2 of a probability below 2^-30
 *    is taken as -30.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define CDL_ORACLE_MAX_LEVELS 256

int cdl_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Number of host threads the parallel loops use from now on (timing at one thread and at all cores); changes
 * no arithmetic.  Returns the count in effect. */
int cdl_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}

/* ---------------------------------------------------------------------------
 * CPMF of Sec. IV-A, Eq. (4) and its softmax form Eq. (6) (per layer: Eqs. (12), (13)):
 *  P[i-lo] = softmax_i( -alpha (theta - i q)^2 ).
 * window > 0 and window < nlev applies the top-`window` rule of Sec. VI-B.1.
 * ------------------------------------------------------------------------- */
void cdl_oracle_cpmf(double theta, double q, int lo, int hi, double alpha,
                     int window, double *P)
{
    const int nlev = hi - lo + 1;
    double logit[CDL_ORACLE_MAX_LEVELS];
    double top = -INFINITY;
    for (int i = 0; i < nlev; ++i) {
        const double d = theta - (double)(lo + i) * q;
        logit[i] = -alpha * d * d;
        if (logit[i] > top) top = logit[i];
    }
    double sum = 0.0;
    for (int i = 0; i < nlev; ++i) {
        P[i] = exp(logit[i] - top);
        sum += P[i];
    }
    for (int i = 0; i < nlev; ++i) P[i] /= sum;

    if (window > 0 && window < nlev) {
        int keep[CDL_ORACLE_MAX_LEVELS];
        memset(keep, 0, sizeof keep);
        for (int r = 0; r < window; ++r) {
            int best = -1;
            for (int i = 0; i < nlev; ++i)       /* strict '>' : lower index wins ties */
                if (!keep[i] && (best < 0 || logit[i] > logit[best])) best = i;
            keep[best] = 1;
        }
        double kept = 0.0;
        for (int i = 0; i < nlev; ++i) {
            if (!keep[i]) P[i] = 0.0;
            kept += P[i];
        }
        for (int i = 0; i < nlev; ++i) P[i] /= kept;
    }
}

/* Moments of X = Q_p(theta) under a CPMF P: E, Var, Skew_u (Lemma 1). */
static void moments(const double *P, double q, int lo, int hi,
                    double *E, double *Var, double *Skewu)
{
    const int nlev = hi - lo + 1;
    double e1 = 0.0, e2 = 0.0, e3 = 0.0;
    for (int i = 0; i < nlev; ++i) {
        const double x = (double)(lo + i) * q;
        e1 += P[i] * x;
        e2 += P[i] * x * x;
        e3 += P[i] * x * x * x;
    }
    double var = 0.0;
    for (int i = 0; i < nlev; ++i) {
        const double x = (double)(lo + i) * q;
        var += P[i] * (x - e1) * (x - e1);
    }
    *E = e1;
    *Var = var;
    *Skewu = e3 - e1 * e2;
}

/* ---------------------------------------------------------------------------
 * Soft deterministic quantizer of Sec. IV-B, Eq. (8) (per layer: Eq. (15)):
 *  Q_d(theta) = sum_i P(iq|theta) iq.
 * ------------------------------------------------------------------------- */
void cdl_oracle_soft(const float *x, int64_t n, float q, int lo, int hi,
                     float alpha, int window, double *y)
{
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double P[CDL_ORACLE_MAX_LEVELS];
        cdl_oracle_cpmf((double)x[e], (double)q, lo, hi, (double)alpha, window, P);
        double acc = 0.0;
        for (int i = 0; i <= hi - lo; ++i) acc += P[i] * ((double)(lo + i) * (double)q);
        y[e] = acc;
    }
}

/* ---------------------------------------------------------------------------
 * Per-element partial derivatives of Q_d.
 *   d/dtheta = 2 alpha Var                                      Lemma 1, Eq. (9a)
 *   d/dq     = ( E + 2 alpha theta Var - 2 alpha Skew_u ) / q   Lemma 1, Eq. (9b)
 *   d/dalpha = 2 theta Var - Skew_u                   derived, see the header
 * Any output pointer may be NULL.  var_out receives Var{Q_p | theta}.
 * ------------------------------------------------------------------------- */
void cdl_oracle_partials(const float *x, int64_t n, float q, int lo, int hi,
                         float alpha, int window, double *d_theta, double *d_q,
                         double *d_alpha, double *var_out)
{
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double P[CDL_ORACLE_MAX_LEVELS];
        const double th = (double)x[e], a = (double)alpha, qq = (double)q;
        cdl_oracle_cpmf(th, qq, lo, hi, a, window, P);
        double E, Var, Sk;
        moments(P, qq, lo, hi, &E, &Var, &Sk);
        if (d_theta) d_theta[e] = 2.0 * a * Var;
        if (d_q) d_q[e] = (E + 2.0 * a * th * Var - 2.0 * a * Sk) / qq;
        if (d_alpha) d_alpha[e] = 2.0 * th * Var - Sk;
        if (var_out) var_out[e] = Var;
    }
}

/* ---------------------------------------------------------------------------
 * Hard index = uniform quantizer Q_u (nearest level), binary32 quotient,
 * round-half-even, clamped; a NaN quotient takes the lowest level lo.
 * hist (nullable, nlev counters) is incremented, not cleared.
 * ------------------------------------------------------------------------- */
void cdl_oracle_hard(const float *x, int64_t n, float q, int lo, int hi,
                     int32_t *idx, uint64_t *hist)
{
    for (int64_t e = 0; e < n; ++e) {
        const float u = x[e] / q;            /* IEEE binary32 division */
        float r = nearbyintf(u);             /* default mode: ties to even */
        if (!(r >= (float)lo)) r = (float)lo;    /* also catches NaN */
        if (r > (float)hi) r = (float)hi;
        const int k = (int)r;
        if (idx) idx[e] = k;
        if (hist) hist[k - lo] += 1;
    }
}

/* ---------------------------------------------------------------------------
 * Soft histogram of Sec. V-C, Eq. (25): sums[k] = sum_i P_alpha(k q | x[i]); divided by n it is the marginal
 * PMF of the randomly quantized tensor, whose entropy is the average number of bits per entry.
 * ------------------------------------------------------------------------- */
void cdl_oracle_mpmf(const float *x, int64_t n, float q, int lo, int hi, float alpha, int window, double *sums)
{
    const int nlev = hi - lo + 1;
    double acc[CDL_ORACLE_MAX_LEVELS];
    for (int k = 0; k < CDL_ORACLE_MAX_LEVELS; ++k) acc[k] = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : acc[:CDL_ORACLE_MAX_LEVELS])
    for (int64_t e = 0; e < n; ++e) {
        double P[CDL_ORACLE_MAX_LEVELS];
        cdl_oracle_cpmf((double)x[e], (double)q, lo, hi, (double)alpha, window, P);
        for (int k = 0; k < nlev; ++k) acc[k] += P[k];
    }
    for (int k = 0; k < nlev; ++k) sums[k] = acc[k];
}

/* ---------------------------------------------------------------------------
 * Counter-based generator Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as
 * 1, 2, 3", SC 2011), written from its published definition: ten rounds of
 *   (c0,c1,c2,c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
 * with the key (k0,k1) advanced by the Weyl constants (W0,W1) between rounds.
 * ------------------------------------------------------------------------- */
void cdl_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += W0;
            k1 += W1;
        }
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0;
        c1 = n1;
        c2 = n2;
        c3 = n3;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

/* The uniform number in [0,1) that element number e of a tensor draws under `seed`: word (e mod 4) of the
 * Philox block with counter (e div 4, 0) and key = seed, top 24 bits scaled by 2^-24. */
double cdl_oracle_uniform(uint64_t seed, uint64_t e)
{
    const uint64_t blk = e >> 2;
    const uint32_t ctr[4] = {(uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t r[4];
    cdl_oracle_philox4x32_10(ctr, key, r);
    return (double)(r[e & 3] >> 8) * (1.0 / 16777216.0);
}

/* ---------------------------------------------------------------------------
 * Probabilistic quantizer Q_p of Sec. IV-A, Eq. (7): theta is mapped to level i with probability
 * P_alpha(iq | theta).  Sampling by inversion: with u the element's uniform number, the index is the first
 * level, in increasing order, whose cumulative probability exceeds u.  cdf_lo / cdf_hi (nullable) receive the
 * cumulative probability just below and through the chosen level, u_out the uniform number.
 * ------------------------------------------------------------------------- */
void cdl_oracle_sample(const float *x, int64_t n, float q, int lo, int hi, float alpha, int window,
                       uint64_t seed, uint64_t first_index, int32_t *idx, double *u_out,
                       double *cdf_lo, double *cdf_hi)
{
    const int nlev = hi - lo + 1;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double P[CDL_ORACLE_MAX_LEVELS];
        cdl_oracle_cpmf((double)x[e], (double)q, lo, hi, (double)alpha, window, P);
        const double u = cdl_oracle_uniform(seed, first_index + (uint64_t)e);
        double cum = 0.0, below = 0.0;
        int k = -1;
        for (int i = 0; i < nlev; ++i) {
            if (P[i] == 0.0) continue;
            below = cum;
            cum += P[i];
            k = i;
            if (cum > u) break;
        }
        idx[e] = lo + k;
        if (u_out) u_out[e] = u;
        if (cdf_lo) cdf_lo[e] = below;
        if (cdf_hi) cdf_hi[e] = cum;
    }
}

/* ---------------------------------------------------------------------------
 * Entropy of the empirical level distribution, H(P) = -sum_c P[c] log2 P[c]
 * (Sec. III-A with base 2; Sec. V-C), P[c] = hist[c] / n, 0 log 0 = 0.
 * ------------------------------------------------------------------------- */
void cdl_oracle_entropy(const uint64_t *hist, int nlev, double *H_bits,
                        double *level_prob, uint64_t *n_out)
{
    uint64_t n = 0;
    for (int c = 0; c < nlev; ++c) n += hist[c];
    double H = 0.0;
    for (int c = 0; c < nlev; ++c) {
        const double p = n ? (double)hist[c] / (double)n : 0.0;
        if (level_prob) level_prob[c] = p;
        if (p > 0.0) H -= p * log2(p);
    }
    *H_bits = H;
    if (n_out) *n_out = n;
}

/* ---------------------------------------------------------------------------
 * Backward of the quantizer with the gradient proxy of Sec. V-B:
 *   grad_x[e]  = g[e] * dQ_d/dtheta (Eqs. (18), (20))
 *                + rate_weight * d(nH)/dtheta_e        (rate term, see header)
 *   grad_q     = sum_e g[e] * dQ_d/dq      (Eqs. (21), (22))
 *   grad_alpha = sum_e g[e] * dQ_d/dalpha  (Eqs. (23), (24))
 * level_prob == NULL or rate_weight == 0: no rate term.
 * Two scales for comparing the reduced sums with a lower-precision result
 * (all nullable): abs_q / abs_alpha receive sum_e |g[e] * partial|, and
 * mag_q / mag_alpha receive sum_e |g[e]| * (sum of the magnitudes of the terms
 * of the printed formula: |E| + |2 alpha theta Var| + |2 alpha Skew_u|, over q;
 * |2 theta Var| + |Skew_u|), which bounds what cancellation between those
 * terms can cost.
 * ------------------------------------------------------------------------- */
void cdl_oracle_backward(const float *x, const float *g, int64_t n, float q,
                         int lo, int hi, float alpha, int window,
                         float rate_weight, const double *level_prob,
                         double *grad_x, double *grad_q, double *grad_alpha,
                         double *abs_q, double *abs_alpha,
                         double *mag_q, double *mag_alpha)
{
    const int nlev = hi - lo + 1;
    double log2p[CDL_ORACLE_MAX_LEVELS];
    const int with_rate = (level_prob != NULL) && (rate_weight != 0.0f);
    for (int i = 0; i < nlev; ++i) {
        double p = with_rate ? level_prob[i] : 1.0;
        log2p[i] = (p < ldexp(1.0, -30)) ? -30.0 : log2(p);
    }
    double sq = 0.0, sa = 0.0, aq = 0.0, aa = 0.0, mq = 0.0, ma = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : sq, sa, aq, aa, mq, ma)
    for (int64_t e = 0; e < n; ++e) {
        double P[CDL_ORACLE_MAX_LEVELS];
        const double th = (double)x[e], a = (double)alpha, qq = (double)q;
        const double ge = (double)g[e];
        cdl_oracle_cpmf(th, qq, lo, hi, a, window, P);
        double E, Var, Sk;
        moments(P, qq, lo, hi, &E, &Var, &Sk);
        double gx = ge * (2.0 * a * Var);
        if (with_rate) {
            double s_lx = 0.0, s_l = 0.0;
            for (int i = 0; i < nlev; ++i) {
                s_lx += P[i] * log2p[i] * ((double)(lo + i) * qq);
                s_l += P[i] * log2p[i];
            }
            gx += (double)rate_weight * (-2.0 * a * (s_lx - s_l * E));
        }
        if (grad_x) grad_x[e] = gx;
        const double tq = ge * ((E + 2.0 * a * th * Var - 2.0 * a * Sk) / qq);
        const double ta = ge * (2.0 * th * Var - Sk);
        sq += tq;
        sa += ta;
        aq += fabs(tq);
        aa += fabs(ta);
        mq += fabs(ge) * (fabs(E) + fabs(2.0 * a * th * Var) + fabs(2.0 * a * Sk)) / qq;
        ma += fabs(ge) * (fabs(2.0 * th * Var) + fabs(Sk));
    }
    if (grad_q) *grad_q = sq;
    if (grad_alpha) *grad_alpha = sa;
    if (abs_q) *abs_q = aq;
    if (abs_alpha) *abs_alpha = aa;
    if (mag_q) *mag_q = mq;
    if (mag_alpha) *mag_alpha = ma;
}

/* ---------------------------------------------------------------------------
 * Layer products over the integer indices (Sec. V-A: forward and backward
 * passes run on the quantized weights and activations).  Indices are bytes;
 * a_unsigned selects uint8 for the activation operand (index set B), weights
 * and gradient indices are int8.  Row-major with explicit leading dimensions.
 * Accumulators are int64 so that the caller can check the int32 range.
 *   fwd : ACC[m,n] = sum_k A[m,k] W[k,n]
 *   dX  : ACC[m,k] = sum_n G[m,n] W[k,n]
 *   dW  : ACC[k,n] = sum_m A[m,k] G[m,n]
 * ------------------------------------------------------------------------- */
static inline int64_t ld_idx(const void *p, int64_t off, int is_unsigned)
{
    return is_unsigned ? (int64_t)((const uint8_t *)p)[off]
                       : (int64_t)((const int8_t *)p)[off];
}

void cdl_oracle_gemm_fwd(const void *A, int64_t lda, int a_unsigned,
                         const int8_t *W, int64_t ldw, int M, int N, int K,
                         int64_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int k = 0; k < K; ++k)
                s += ld_idx(A, (int64_t)m * lda + k, a_unsigned) * (int64_t)W[(int64_t)k * ldw + n];
            acc[(int64_t)m * N + n] = s;
        }
}

void cdl_oracle_gemm_dx(const int8_t *G, int64_t ldg, const int8_t *W,
                        int64_t ldw, int M, int N, int K, int64_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) {
            int64_t s = 0;
            for (int n = 0; n < N; ++n)
                s += (int64_t)G[(int64_t)m * ldg + n] * (int64_t)W[(int64_t)k * ldw + n];
            acc[(int64_t)m * K + k] = s;
        }
}

void cdl_oracle_gemm_dw(const void *A, int64_t lda, int a_unsigned,
                        const int8_t *G, int64_t ldg, int M, int N, int K,
                        int64_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k)
        for (int n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int m = 0; m < M; ++m)
                s += ld_idx(A, (int64_t)m * lda + k, a_unsigned) * (int64_t)G[(int64_t)m * ldg + n];
            acc[(int64_t)k * N + n] = s;
        }
}

/* -------------------------------------------------------------------------
 * Convolutional layer products on index tensors.  The paper's networks are CNNs (Sec. VI-C, VI-D: ResNets, whose
 * stages begin with stride-2 layers) whose layers apply the quantized weights to the quantized activations
 * (Algorithm 1, forward and backward over the quantized tensors); the convolution itself is the textbook strided
 * cross-correlation with zero padding:
 *   X [N,H,W,C] (index bytes), Wt [(r*S+s)*C + c, co] (int8, row pitch ldw), G [N,P,Q,CO] (int8),
 *   P = (H + 2 pad_h - R) / stride + 1,  Q = (W + 2 pad_w - S) / stride + 1   (integer division)
 *   fwd : Y [n,p,q,co]        = sum_{r,s,c}  X[n, p*stride-pad_h+r, q*stride-pad_w+s, c] * Wt[(r*S+s)*C+c, co]
 *   dX  : dX[n,h,w,c]         = sum over (r,s,co) and the (p,q) with p*stride-pad_h+r = h, q*stride-pad_w+s = w
 *                               of G[n,p,q,co] * Wt[(r*S+s)*C+c, co]
 *   dW  : dW[(r*S+s)*C+c, co] = sum_{n,p,q}  X[n, p*stride-pad_h+r, q*stride-pad_w+s, c] * G[n,p,q,co]
 * (a term whose spatial position falls outside the tensor is zero).  dX and dW are the adjoints of fwd in X and
 * in Wt.  Sums are int64.
 * ------------------------------------------------------------------------- */
void cdl_oracle_conv_fwd(const void *X, int x_unsigned, const int8_t *Wt, int64_t ldw, int N, int H, int W, int C,
                         int R, int S, int pad_h, int pad_w, int CO, int stride, int64_t *acc)
{
    const int P = (H + 2 * pad_h - R) / stride + 1, Q = (W + 2 * pad_w - S) / stride + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int co = 0; co < CO; ++co) {
                    int64_t sum = 0;
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride - pad_h + r;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int w = q * stride - pad_w + s;
                            if (w < 0 || w >= W) continue;
                            for (int c = 0; c < C; ++c)
                                sum += ld_idx(X, (((int64_t)n * H + h) * W + w) * C + c, x_unsigned) *
                                       (int64_t)Wt[((int64_t)(r * S + s) * C + c) * ldw + co];
                        }
                    }
                    acc[(((int64_t)n * P + p) * Q + q) * CO + co] = sum;
                }
}

void cdl_oracle_conv_dx(const int8_t *G, const int8_t *Wt, int64_t ldw, int N, int H, int W, int C,
                        int R, int S, int pad_h, int pad_w, int CO, int stride, int64_t *acc)
{
    const int P = (H + 2 * pad_h - R) / stride + 1, Q = (W + 2 * pad_w - S) / stride + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int w = 0; w < W; ++w)
                for (int c = 0; c < C; ++c) {
                    int64_t sum = 0;
                    for (int r = 0; r < R; ++r) {
                        const int ph = h + pad_h - r;            /* = p * stride for the output row that reads h at tap r */
                        if (ph < 0 || ph % stride != 0 || ph / stride >= P) continue;
                        const int p = ph / stride;
                        for (int s = 0; s < S; ++s) {
                            const int qw = w + pad_w - s;
                            if (qw < 0 || qw % stride != 0 || qw / stride >= Q) continue;
                            const int q = qw / stride;
                            for (int co = 0; co < CO; ++co)
                                sum += (int64_t)G[(((int64_t)n * P + p) * Q + q) * CO + co] *
                                       (int64_t)Wt[((int64_t)(r * S + s) * C + c) * ldw + co];
                        }
                    }
                    acc[(((int64_t)n * H + h) * W + w) * C + c] = sum;
                }
}

void cdl_oracle_conv_dw(const void *X, int x_unsigned, const int8_t *G, int N, int H, int W, int C,
                        int R, int S, int pad_h, int pad_w, int CO, int stride, int64_t *acc)
{
    const int P = (H + 2 * pad_h - R) / stride + 1, Q = (W + 2 * pad_w - S) / stride + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (int r = 0; r < R; ++r)
        for (int s = 0; s < S; ++s)
            for (int c = 0; c < C; ++c)
                for (int co = 0; co < CO; ++co) {
                    int64_t sum = 0;
                    for (int n = 0; n < N; ++n)
                        for (int p = 0; p < P; ++p) {
                            const int h = p * stride - pad_h + r;
                            if (h < 0 || h >= H) continue;
                            for (int q = 0; q < Q; ++q) {
                                const int w = q * stride - pad_w + s;
                                if (w < 0 || w >= W) continue;
                                sum += ld_idx(X, (((int64_t)n * H + h) * W + w) * C + c, x_unsigned) *
                                       (int64_t)G[(((int64_t)n * P + p) * Q + q) * CO + co];
                            }
                        }
                    acc[((int64_t)(r * S + s) * C + c) * CO + co] = sum;
                }
}
