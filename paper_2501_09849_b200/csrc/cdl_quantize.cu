// Quantizer kernels of the CDL layer for sm_100a: hard index + histogram, soft value Q_d,
// analytic backward.  One pass over the tensor each; HBM-bound by design.
//
// Arithmetic (per element theta, Sec. IV of the paper):
//   k0  = rint(clamp(theta / q, lo, hi))         the hard index (binary32 quotient, ties to even).  Rounding
//         is done by adding 1.5 * 2^23 (no conversion instruction); the integer is read from the mantissa.
//   d   = theta - kn q, kn the reference level (k0, or the exact nearest level when a window is used).
//   e_j = exp(-alpha ((d - j q)^2 - d^2)) = 2^(j (B - A j)),  A = alpha q^2 log2 e, B = 2 alpha q d log2 e:
//         the CPMF of Eq. (4) relative to level kn, P_{kn+j} = e_j / sum e_j, e_0 = 1, e_j <= 1 (no max pass).
//   Moments of the index offset under that CPMF give everything else:
//   Q_d = kn q + q E J                                                   (Eq. (8))
//   dQ_d/dtheta = 2 alpha q^2 Var J                                      (Lemma 1, Eq. (9a))
//   dQ_d/dq     = kn + E J + 2 alpha q ((d - kn q) Var J - q Cov(J, J^2)) (Eq. (9b), re-centred on kn)
//   dQ_d/dalpha = q^2 (2 d Var J - q Cov(J, J^2))                        (Appendix B steps, re-centred)
//   rate term   = rate_weight * (-2 alpha q) * Cov(L, J),  L = log2 of the level probability.
// The re-centred forms equal the printed ones (expand X = q (kn + J)) without their cancellation.
//
// Four evaluation paths, chosen per launch from alpha q^2 and the window (both uniform over the tensor):
//   NEAR3  alpha q^2 > 12: levels two or more steps from the nearest one weigh < e^-24; only kn-1, kn, kn+1 are
//          summed.  Here d must be exact next to the midpoints (dQ_d/dtheta ~ alpha q^2 / 2 there), so d is
//          carried as an unevaluated sum dh + dl of two floats: k0 q is split exactly with one fma and
//          theta - fl(k0 q) is exact (operands within a factor of two).
//   WIN5   alpha q^2 <= 12, window of 5 (Sec. VI-B.1): the five in-range levels nearest theta, st .. st+4, each
//          with its own ex2; moments are taken about st with compile-time weights 0..4 and shifted to kn.
//          The window needs the exact nearest level (ties: the lower one), decided from dh + dl on a rarely
//          taken branch.
//   LOOP   everything else (whole index set, or another odd window): a loop over the levels within jmax
//          steps of kn (further ones weigh < 2^-40), one ex2 per level.
//   LATTICE  whole index set, vector region of the soft and backward passes: e_j = G_j b^j with G_j = 2^(-A j^2)
//          the same for every element (a shared-memory table that also holds j G_j, j^2 G_j, j^3 G_j) and
//          b = 2^B per element, so a level costs a few multiply-adds and no ex2.  b^j is carried as
//          1 + beta_j, beta_(j+1) = beta_j + (beta_j beta + beta): for small alpha q^2 b is so close to 1 that
//          a binary32 b would lose B (its relative error, times j, would shift theta by far more than the
//          tolerance), while beta = 2^B - 1 keeps it to full relative precision.  The four elements of a load
//          walk the levels together on the packed instructions, the levels above and below kn separately and
//          outwards.  Taken when the window of +-jmax levels is narrower than the index set and no rate term is
//          asked for, by the warps all of whose elements have jmax levels on either side (the others take LOOP);
//          1.3x the LOOP form on the soft pass, 1.4x on the backward pass.
#include "cdl_internal.h"

#include <math.h>

namespace cdl {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 2;            // float4 loads in flight per thread
constexpr int kHistCluster = 8;      // CTAs per cluster in launches that fill a histogram (portable cluster size)
// streaming accesses: every element is touched once, so loads and stores bypass the usual cache retention
#define CDL_LD(p) __ldcs(p)
#define CDL_ST(p, v) __stcs(p, v)
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr int kMagicBits = 0x4B400000;
// |quotient - nearest integer| above this may be a rounding tie once the 3-ulp error of the reciprocal product is
// allowed for: indices lie in [-128, 255], where an ulp is at most 2^-16; 0.5 - 2^-12 leaves 16 ulp of margin.
constexpr float kTieGuard = 0.5f - 0.000244140625f;

enum QuantPath { PATH_NEAR3 = 0, PATH_WIN5 = 1, PATH_LOOP = 2, PATH_LATTICE = 3 };

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Philox4x32-10 (Salmon et al., SC 2011) from its definition: ten rounds of
//   (c0,c1,c2,c3) <- (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)),  key += (W0, W1) between rounds.
// Counter = (block number, 0), key = seed; the block's four words serve elements 4 b .. 4 b + 3.
__device__ __forceinline__ uint4 philox4x32_10(unsigned long long block, unsigned long long seed)
{
    const unsigned int M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    unsigned int c0 = (unsigned int)block, c1 = (unsigned int)(block >> 32), c2 = 0u, c3 = 0u;
    unsigned int k0 = (unsigned int)seed, k1 = (unsigned int)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) {
            k0 += W0;
            k1 += W1;
        }
        const unsigned int n0 = __umulhi(M1, c2) ^ c1 ^ k0;
        const unsigned int n1 = M1 * c2;
        const unsigned int n2 = __umulhi(M0, c0) ^ c3 ^ k1;
        const unsigned int n3 = M0 * c0;
        c0 = n0;
        c1 = n1;
        c2 = n2;
        c3 = n3;
    }
    return make_uint4(c0, c1, c2, c3);
}
// top 24 bits of a word as a uniform number in [0, 1)
__device__ __forceinline__ float u01(unsigned int w) { return (float)(w >> 8) * 5.9604644775390625e-8f; }
__device__ __forceinline__ float philox_uniform(unsigned long long seed, unsigned long long e)
{
    const uint4 r = philox4x32_10(e >> 2, seed);
    const unsigned int k = (unsigned int)e & 3u;
    return u01(k == 0 ? r.x : k == 1 ? r.y : k == 2 ? r.z : r.w);
}

// Adds P (a CPMF entry in [0,1]) to the soft-histogram bin of `level` in units of 2^-32: integer sums are exact and
// independent of the order in which elements arrive.
__device__ __forceinline__ void mp_add(unsigned long long *mp_s, int bin, int lane, float P)
{
    // a reduction on a 32-bit shared-window address (no result, no generic-address arithmetic)
    const unsigned int a = (unsigned int)__cvta_generic_to_shared(mp_s) + (unsigned int)(((bin << 5) + lane) << 3);
    asm volatile("red.shared.add.u64 [%0], %1;" ::"r"(a), "l"((unsigned long long)__float2uint_rn(P * 4294967296.0f)) : "memory");
}

struct ElemOut {
    int k0;       // hard index
    float y;      // Q_d
    float gx;     // grad wrt theta
    float tq;     // g * dQ_d/dq
    float ta;     // g * dQ_d/dalpha
};

// d = x - k q as dh + dl (dl: what dh lost), k an integer-valued float near x / q
__device__ __forceinline__ void residual2(float x, float k, float q, float &dh, float &dl)
{
    const float ph = __fmul_rn(k, q);
    const float pl = __fmaf_rn(k, q, -ph);
    const float s = __fsub_rn(x, ph);
    dh = __fsub_rn(s, pl);
    dl = __fsub_rn(__fsub_rn(s, dh), pl);
}

// Moves (kn, ki, dh) to the exact nearest in-range level; of two equally near levels the lower one.
__device__ __noinline__ void nearest_fixup(const QuantDev &P, float &kn, int &ki, float &dh, float dl)
{
    if ((dh > P.half_q || (dh == P.half_q && dl > 0.0f)) && kn < P.fhi) {
        kn += 1.0f;
        ki += 1;
        dh = __fsub_rn(dh, P.q);
    } else if ((dh < -P.half_q || (dh == -P.half_q && dl <= 0.0f)) && kn > P.flo) {
        kn -= 1.0f;
        ki -= 1;
        dh = __fadd_rn(dh, P.q);
    }
}

template <int MODE, int PATH, bool RATE>
__device__ __forceinline__ ElemOut quant_elem(const QuantDev &P, const float *__restrict__ Ltab, float x, float g,
                                              unsigned long long *mp_s = nullptr, int lane = 0)
{
    // the third template flag means "rate term" in the backward pass and "soft histogram" in the soft pass
    constexpr bool kRate = RATE && MODE == MODE_BWD;
    constexpr bool kSoftHist = RATE && MODE == MODE_SOFT;
    ElemOut o;
    const float q = P.q;
    // ---- hard index: rint(clamp(RN(x / q))), a NaN quotient clamps to lo.  x * RN(1/q) is within 3 ulp of the
    // correctly rounded quotient, so both round to the same integer unless the quotient lies within a few ulp
    // of a half-integer; only then (about 5 elements in 10^4) is the IEEE division itself evaluated.
    float c = fminf(fmaxf(P.fast_div ? __fmul_rn(x, P.rq) : __fdiv_rn(x, q), P.flo), P.fhi);
    float t = __fadd_rn(c, kMagic);
    float kn = __fsub_rn(t, kMagic);
    if (P.fast_div && fabsf(__fsub_rn(c, kn)) > kTieGuard) {
        c = fminf(fmaxf(__fdiv_rn(x, q), P.flo), P.fhi);
        t = __fadd_rn(c, kMagic);
        kn = __fsub_rn(t, kMagic);
    }
    int ki = __float_as_int(t) - kMagicBits;
    o.k0 = ki;
    o.y = 0.0f;
    o.gx = 0.0f;
    o.tq = 0.0f;
    o.ta = 0.0f;
    if (MODE == MODE_HARD) return o;

    float m1, varj = 0.0f, covj = 0.0f, rate = 0.0f, dh;   // moments of J about kn
    if (PATH == PATH_NEAR3) {
        float dl;
        residual2(x, kn, q, dh, dl);
        const float m2d = -2.0f * dh, dl2 = 2.0f * dl;
        const float w1 = __fsub_rn(__fadd_rn(q, m2d), dl2);   // (q - 2 dh) - 2 dl, exact near the midpoint
        const float wm = __fadd_rn(__fsub_rn(q, m2d), dl2);   // (q + 2 dh) + 2 dl
        float e1 = ex2_approx(-P.c1 * w1);
        float em = ex2_approx(-P.c1 * wm);
        e1 = (kn < P.fhi) ? e1 : 0.0f;
        em = (kn > P.flo) ? em : 0.0f;
        if (MODE == MODE_SAMPLE) {
            // inversion in increasing level order: kn-1 (em), kn (1), kn+1 (e1); g carries the uniform number
            const float S = 1.0f + e1 + em;
            const float tt = fminf(g * S, S * 0.99999994f);
            const int ks = ki + ((tt >= em + 1.0f) ? 1 : 0) - ((tt < em) ? 1 : 0);
            o.k0 = ks;
            o.y = __fmul_rn((float)ks, q);
            return o;
        }
        const float rS = rcp_approx(1.0f + e1 + em);
        m1 = (e1 - em) * rS;
        o.y = __fmaf_rn(kn, q, __fmul_rn(q, m1));
        if (kSoftHist) {
            mp_add(mp_s, ki - P.lo, lane, rS);
            if (e1 > 0.0f) mp_add(mp_s, ki + 1 - P.lo, lane, e1 * rS);
            if (em > 0.0f) mp_add(mp_s, ki - 1 - P.lo, lane, em * rS);
        }
        if (MODE == MODE_BWD) {
            const float m2 = (e1 + em) * rS;         // E J^2; E J^3 = E J
            varj = fmaf(-m1, m1, m2);
            covj = m1 - m1 * m2;
            if (kRate) {
                const float Lc = Ltab[ki - P.lo];
                const float l1 = (Ltab[min(ki + 1, P.hi) - P.lo] - Lc) * e1;
                const float lm = (Ltab[max(ki - 1, P.lo) - P.lo] - Lc) * em;
                rate = ((l1 - lm) - m1 * (l1 + lm)) * rS;
            }
        }
    } else if (PATH == PATH_WIN5) {
        float dl;
        residual2(x, kn, q, dh, dl);
        if (fabsf(dh) >= P.half_q) nearest_fixup(P, kn, ki, dh, dl);
        const float stf = fminf(fmaxf(kn - 2.0f, P.flo), P.fhi - 4.0f);
        const float j0 = stf - kn;                    // -4 .. 0
        const float B = P.c1x2 * dh;
        float T0 = 0.0f, T1 = 0.0f, T2 = 0.0f, T3 = 0.0f, R0 = 0.0f, R1 = 0.0f;
        float ev[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
        const float *Lp = Ltab;
        float Lc = 0.0f;
        if (kRate) {
            Lc = Ltab[ki - P.lo];
            Lp = Ltab + (min(max(ki - 2, P.lo), P.hi - 4) - P.lo);
        }
#pragma unroll
        for (int i = 0; i < 5; ++i) {
            const float jf = j0 + (float)i;
            const float e = ex2_approx(jf * fmaf(-P.A, jf, B));
            if (MODE == MODE_SAMPLE || kSoftHist) ev[i] = e;
            T0 += e;
            if (i > 0) T1 = fmaf((float)i, e, T1);
            if (MODE == MODE_BWD) {
                if (i > 0) {
                    T2 = fmaf((float)(i * i), e, T2);
                    T3 = fmaf((float)(i * i * i), e, T3);
                }
                if (kRate) {
                    const float le = (Lp[i] - Lc) * e;
                    R0 += le;
                    if (i > 0) R1 = fmaf((float)i, le, R1);
                }
            }
        }
        if (MODE == MODE_SAMPLE) {
            const float tt = fminf(g * T0, T0 * 0.99999994f);
            float cum = 0.0f;
            int cnt = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                cum += ev[i];
                cnt += (cum <= tt) ? 1 : 0;
            }
            const int ks = min(max(ki - 2, P.lo), P.hi - 4) + cnt;
            o.k0 = ks;
            o.y = __fmul_rn((float)ks, q);
            return o;
        }
        const float rT = rcp_approx(T0);
        const float mi = T1 * rT;                      // E I, I = level - st
        o.y = __fmaf_rn(stf, q, __fmul_rn(q, mi));
        if (kSoftHist) {
            const int b0 = min(max(ki - 2, P.lo), P.hi - 4) - P.lo;
#pragma unroll
            for (int i = 0; i < 5; ++i) mp_add(mp_s, b0 + i, lane, ev[i] * rT);
        }
        m1 = mi + j0;
        if (MODE == MODE_BWD) {
            const float m2i = T2 * rT, m3i = T3 * rT;
            varj = fmaf(-mi, mi, m2i);
            covj = fmaf(-mi, m2i, m3i) + 2.0f * j0 * varj;   // Cov(J, J^2) with J = I + j0
            if (kRate) rate = (R1 - mi * R0) * rT;
        }
    } else {
        int jlo, jhi;
        if (P.window > 0) {
            float dl;
            residual2(x, kn, q, dh, dl);
            if (fabsf(dh) >= P.half_q) nearest_fixup(P, kn, ki, dh, dl);
            const int st = min(max(ki - (P.window >> 1), P.lo), P.hi - P.window + 1);
            jlo = st - ki;
            jhi = jlo + P.window - 1;
        } else {
            dh = __fmaf_rn(-kn, q, x);
            jlo = max(P.lo - ki, -P.jmax);
            jhi = min(P.hi - ki, P.jmax);
        }
        const float B = P.c1x2 * dh;
        float S = 0.0f, S1 = 0.0f, S2 = 0.0f, S3 = 0.0f, R0 = 0.0f, R1 = 0.0f;
        const float Lc = kRate ? Ltab[ki - P.lo] : 0.0f;
        const float *Lp = Ltab + (ki - P.lo);
        float jf = (float)jlo;
        for (int j = jlo; j <= jhi; ++j, jf += 1.0f) {
            const float e = ex2_approx(jf * fmaf(-P.A, jf, B));
            S += e;
            S1 = fmaf(jf, e, S1);
            if (MODE == MODE_BWD) {
                const float j2 = jf * jf;
                S2 = fmaf(j2, e, S2);
                S3 = fmaf(j2 * jf, e, S3);
                if (kRate) {
                    const float le = (Lp[j] - Lc) * e;
                    R0 += le;
                    R1 = fmaf(jf, le, R1);
                }
            }
        }
        if (MODE == MODE_SAMPLE) {
            // second pass over the same levels: first one whose running sum exceeds u * S
            const float tt = fminf(g * S, S * 0.99999994f);
            float cum = 0.0f, jj = (float)jlo;
            int ks = ki + jhi;
            for (int j = jlo; j <= jhi; ++j, jj += 1.0f) {
                cum += ex2_approx(jj * fmaf(-P.A, jj, B));
                if (cum > tt) {
                    ks = ki + j;
                    break;
                }
            }
            o.k0 = ks;
            o.y = __fmul_rn((float)ks, q);
            return o;
        }
        const float rS = rcp_approx(S);
        m1 = S1 * rS;
        o.y = __fmaf_rn(kn, q, __fmul_rn(q, m1));
        if (kSoftHist) {
            float jj = (float)jlo;
            for (int j = jlo; j <= jhi; ++j, jj += 1.0f)
                mp_add(mp_s, ki + j - P.lo, lane, ex2_approx(jj * fmaf(-P.A, jj, B)) * rS);
        }
        if (MODE == MODE_BWD) {
            const float m2 = S2 * rS, m3 = S3 * rS;
            varj = fmaf(-m1, m1, m2);
            covj = fmaf(-m1, m2, m3);
            if (kRate) rate = (R1 - m1 * R0) * rS;
        }
    }
    if (MODE == MODE_BWD) {
        float gx = g * (P.a2 * varj);
        if (kRate) gx = fmaf(P.rate_c, rate, gx);
        o.gx = gx;
        const float dmk = fmaf(-kn, q, dh);            // d - kn q
        const float dq = (kn + m1) + P.two_aq * (dmk * varj - q * covj);
        const float da = P.q2 * (2.0f * dh * varj - q * covj);
        o.tq = g * dq;
        o.ta = g * da;
    }
    return o;
}

// ---- two elements at a time on the NEAR3 path, with the packed binary32 instructions of sm_100 (one issue slot
// per pair of multiplies, adds or fused multiply-adds).  The passes are issue-bound before they are HBM-bound, and
// three quarters of an element's arithmetic is of that kind.  Every packed operation rounds exactly like the scalar
// one it replaces, and the sequence is the scalar path's, so both give the same bits.
struct PairOut {
    int k0[2];
    float2 y, gx, tq, ta;
};
__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __ffma2_rn(b, f2(-1.0f), a); }   // a - b, one rounding

// hard indices of two elements (see quant_elem for the arithmetic)
__device__ __forceinline__ void hard_pair(const QuantDev &P, float2 x, int &k0, int &k1)
{
    const float q = P.q;
    float2 c = P.fast_div ? __fmul2_rn(x, f2(P.rq)) : make_float2(__fdiv_rn(x.x, q), __fdiv_rn(x.y, q));
    c.x = fminf(fmaxf(c.x, P.flo), P.fhi);
    c.y = fminf(fmaxf(c.y, P.flo), P.fhi);
    float2 t = __fadd2_rn(c, f2(kMagic));
    if (P.fast_div) {
        const float2 df = sub2(c, __fadd2_rn(t, f2(-kMagic)));
        if (fabsf(df.x) > kTieGuard || fabsf(df.y) > kTieGuard) {
            c.x = fminf(fmaxf(__fdiv_rn(x.x, q), P.flo), P.fhi);
            c.y = fminf(fmaxf(__fdiv_rn(x.y, q), P.flo), P.fhi);
            t = __fadd2_rn(c, f2(kMagic));
        }
    }
    k0 = __float_as_int(t.x) - kMagicBits;
    k1 = __float_as_int(t.y) - kMagicBits;
}

template <int MODE, bool RATE>
__device__ __forceinline__ PairOut quant_pair_near3(const QuantDev &P, const float2 *__restrict__ Dtab, float2 x, float2 g)
{
    constexpr bool kRate = RATE && MODE == MODE_BWD;
    PairOut o;
    const float q = P.q;
    // hard index (see quant_elem): reciprocal product, clamp, magic-number rounding, exact quotient near ties
    float2 c = __fmul2_rn(x, f2(P.rq));
    if (!P.fast_div) c = make_float2(__fdiv_rn(x.x, q), __fdiv_rn(x.y, q));
    c.x = fminf(fmaxf(c.x, P.flo), P.fhi);
    c.y = fminf(fmaxf(c.y, P.flo), P.fhi);
    float2 t = __fadd2_rn(c, f2(kMagic));
    float2 kn = __fadd2_rn(t, f2(-kMagic));
    if (P.fast_div) {
        const float2 df = sub2(c, kn);
        if (fabsf(df.x) > kTieGuard || fabsf(df.y) > kTieGuard) {
            c.x = fminf(fmaxf(__fdiv_rn(x.x, q), P.flo), P.fhi);
            c.y = fminf(fmaxf(__fdiv_rn(x.y, q), P.flo), P.fhi);
            t = __fadd2_rn(c, f2(kMagic));
            kn = __fadd2_rn(t, f2(-kMagic));
        }
    }
    const int k0 = __float_as_int(t.x) - kMagicBits, k1 = __float_as_int(t.y) - kMagicBits;
    o.k0[0] = k0;
    o.k0[1] = k1;
    // d = x - kn q as dh + dl
    // logits of the two neighbours relative to the nearest level: -alpha q (q -+ 2 d)
    float2 dh, w1, wm;
    if (P.res1 && MODE != MODE_SAMPLE) {   // (the sampled index keeps the two-float residual of the one-by-one path)
        // moderate alpha q^2: the correctly rounded residual of one fused multiply-add is accurate enough (its 2^-25 q
        // moves a logit by at most 2 alpha q^2 2^-25 < 4e-6)
        dh = __ffma2_rn(kn, f2(-q), x);
        w1 = __ffma2_rn(dh, f2(-2.0f), f2(q));
        wm = __ffma2_rn(dh, f2(2.0f), f2(q));
    } else {
        const float2 nph = __fmul2_rn(kn, f2(-q));            // -(kn q) rounded
        const float2 pl = __ffma2_rn(kn, f2(q), nph);         // kn q - RN(kn q), exact
        const float2 sx = __fadd2_rn(x, nph);
        dh = sub2(sx, pl);
        const float2 dl = sub2(sub2(sx, dh), pl);
        w1 = __ffma2_rn(dl, f2(-2.0f), __ffma2_rn(dh, f2(-2.0f), f2(q)));
        wm = __ffma2_rn(dl, f2(2.0f), __ffma2_rn(dh, f2(2.0f), f2(q)));
    }
    const float2 a1 = __fmul2_rn(w1, f2(-P.c1)), am = __fmul2_rn(wm, f2(-P.c1));
    float2 e1 = make_float2(ex2_approx(a1.x), ex2_approx(a1.y));
    float2 em = make_float2(ex2_approx(am.x), ex2_approx(am.y));
    e1.x = (kn.x < P.fhi) ? e1.x : 0.0f;
    e1.y = (kn.y < P.fhi) ? e1.y : 0.0f;
    em.x = (kn.x > P.flo) ? em.x : 0.0f;
    em.y = (kn.y > P.flo) ? em.y : 0.0f;
    const float2 S = __fadd2_rn(__fadd2_rn(f2(1.0f), e1), em);
    if (MODE == MODE_SAMPLE) {
        // inversion in increasing level order: kn-1 (em), kn (1), kn+1 (e1); g carries the uniform numbers
        const float2 gs = __fmul2_rn(g, S), cap = __fmul2_rn(S, f2(0.99999994f)), em1 = __fadd2_rn(em, f2(1.0f));
        const float tx = fminf(gs.x, cap.x), ty = fminf(gs.y, cap.y);
        const int s0 = k0 + ((tx >= em1.x) ? 1 : 0) - ((tx < em.x) ? 1 : 0);
        const int s1 = k1 + ((ty >= em1.y) ? 1 : 0) - ((ty < em.y) ? 1 : 0);
        o.k0[0] = s0;
        o.k0[1] = s1;
        o.y = __fmul2_rn(make_float2((float)s0, (float)s1), f2(q));
        o.gx = o.tq = o.ta = f2(0.0f);
        return o;
    }
    const float2 rS = make_float2(rcp_approx(S.x), rcp_approx(S.y));
    const float2 m1 = __fmul2_rn(sub2(e1, em), rS);
    o.y = __ffma2_rn(kn, f2(q), __fmul2_rn(f2(q), m1));
    o.gx = o.tq = o.ta = f2(0.0f);
    if (MODE == MODE_BWD) {
        const float2 m2 = __fmul2_rn(__fadd2_rn(e1, em), rS);          // E J^2; E J^3 = E J
        const float2 varj = __ffma2_rn(__fmul2_rn(m1, f2(-1.0f)), m1, m2);
        const float2 covj = sub2(m1, __fmul2_rn(m1, m2));
        float2 gx = __fmul2_rn(g, __fmul2_rn(f2(P.a2), varj));
        if (kRate) {
            // log2 p of the upper / lower neighbour relative to the level's own: one 8-byte table entry per element
            const float2 d0 = Dtab[k0 - P.lo], d1 = Dtab[k1 - P.lo];
            const float2 l1 = __fmul2_rn(make_float2(d0.x, d1.x), e1);
            const float2 lm = __fmul2_rn(make_float2(d0.y, d1.y), em);
            const float2 rate = __fmul2_rn(sub2(sub2(l1, lm), __fmul2_rn(m1, __fadd2_rn(l1, lm))), rS);
            gx = __ffma2_rn(f2(P.rate_c), rate, gx);
        }
        o.gx = gx;
        const float2 qc = __fmul2_rn(f2(q), covj);
        const float2 dmk = __ffma2_rn(kn, f2(-q), dh);                 // d - kn q
        const float2 dq = __ffma2_rn(f2(P.two_aq), sub2(__fmul2_rn(dmk, varj), qc), __fadd2_rn(kn, m1));
        const float2 da = __fmul2_rn(f2(P.q2), sub2(__fmul2_rn(__fmul2_rn(f2(2.0f), dh), varj), qc));
        o.tq = dq;          // the caller accumulates g * dq and g * da
        o.ta = da;
    }
    return o;
}

// ---- whole index set without an ex2 per level (see LATTICE in the header comment): the four elements of a
// 128-bit load as two packed pairs that walk the levels together, so that one table load serves all four.
struct LatPair {
    float2 kn, dh, bu, bd;          // reference level, residual, 2^B - 1, 2^-B - 1
    int k0, k1;
    float2 A0, A1, A2, A3;          // sums over the levels other than kn of j^m e_j, m = 0..3
};

// hard indices of a pair (see quant_elem: reciprocal product, clamp, magic-number rounding, exact quotient near ties)
__device__ __forceinline__ void lattice_index(const QuantDev &P, float2 x, LatPair &s)
{
    const float q = P.q;
    float2 c = __fmul2_rn(x, f2(P.rq));
    if (!P.fast_div) c = make_float2(__fdiv_rn(x.x, q), __fdiv_rn(x.y, q));
    c.x = fminf(fmaxf(c.x, P.flo), P.fhi);
    c.y = fminf(fmaxf(c.y, P.flo), P.fhi);
    float2 t = __fadd2_rn(c, f2(kMagic));
    float2 kn = __fadd2_rn(t, f2(-kMagic));
    if (P.fast_div) {
        const float2 df = sub2(c, kn);
        if (fabsf(df.x) > kTieGuard || fabsf(df.y) > kTieGuard) {
            c.x = fminf(fmaxf(__fdiv_rn(x.x, q), P.flo), P.fhi);
            c.y = fminf(fmaxf(__fdiv_rn(x.y, q), P.flo), P.fhi);
            t = __fadd2_rn(c, f2(kMagic));
            kn = __fadd2_rn(t, f2(-kMagic));
        }
    }
    s.kn = kn;
    s.k0 = __float_as_int(t.x) - kMagicBits;
    s.k1 = __float_as_int(t.y) - kMagicBits;
}

__device__ __forceinline__ void lattice_setup(const QuantDev &P, float2 x, LatPair &s)
{
    const float q = P.q;
    const float2 kn = s.kn;
    s.dh = __ffma2_rn(kn, f2(-q), x);
    // B = 2 alpha q d log2 e, limited to +-64: beyond that the element lies far outside the index set and the
    // levels on the side that still exists weigh < 2^-64 either way
    float2 B = __fmul2_rn(s.dh, f2(P.c1x2));
    B.x = fminf(fmaxf(B.x, -64.0f), 64.0f);
    B.y = fminf(fmaxf(B.y, -64.0f), 64.0f);
    // beta = 2^B - 1 upwards, 2^-B - 1 downwards.  |B| < 1: expm1 of a quarter of the argument by its series
    // (|z| < 0.174, remainder < 5e-9 relative), then (1 + beta)^2 - 1 = beta (2 + beta) twice; the downward one
    // from -beta / (1 + beta).  Otherwise from ex2 directly (b is then far enough from 1).
    const float2 z = __fmul2_rn(B, f2(0.25f * 0.693147180559945f));
    float2 pz = __ffma2_rn(z, f2(1.0f / 720.0f), f2(1.0f / 120.0f));
    pz = __ffma2_rn(z, pz, f2(1.0f / 24.0f));
    pz = __ffma2_rn(z, pz, f2(1.0f / 6.0f));
    pz = __ffma2_rn(z, pz, f2(0.5f));
    pz = __ffma2_rn(z, pz, f2(1.0f));
    pz = __fmul2_rn(z, pz);
    pz = __fmul2_rn(pz, __fadd2_rn(pz, f2(2.0f)));
    pz = __fmul2_rn(pz, __fadd2_rn(pz, f2(2.0f)));
    const float2 pd1 = __fadd2_rn(pz, f2(1.0f));
    const float2 pd = __fmul2_rn(__fmul2_rn(pz, f2(-1.0f)), make_float2(rcp_approx(pd1.x), rcp_approx(pd1.y)));
    s.bu.x = fabsf(B.x) < 1.0f ? pz.x : ex2_approx(B.x) - 1.0f;
    s.bu.y = fabsf(B.y) < 1.0f ? pz.y : ex2_approx(B.y) - 1.0f;
    s.bd.x = fabsf(B.x) < 1.0f ? pd.x : ex2_approx(-B.x) - 1.0f;
    s.bd.y = fabsf(B.y) < 1.0f ? pd.y : ex2_approx(-B.y) - 1.0f;
    s.A0 = s.A1 = s.A2 = s.A3 = f2(0.0f);
}

// adds level kn + DIR * j with weight G_j * w to the sums of one pair
template <bool BWD, int DIR>
__device__ __forceinline__ void lattice_add(LatPair &s, float4 ga, float4 ha, float2 w)
{
    s.A0 = __ffma2_rn(make_float2(ga.x, ga.y), w, s.A0);
    s.A1 = __ffma2_rn(make_float2(DIR * ga.z, DIR * ga.w), w, s.A1);
    if (BWD) {
        s.A2 = __ffma2_rn(make_float2(ha.x, ha.y), w, s.A2);
        s.A3 = __ffma2_rn(make_float2(DIR * ha.z, DIR * ha.w), w, s.A3);
    }
}

// One side of the sums for both pairs: levels kn + DIR * j, j = 1 .. jmax (all of them inside the index set).
template <bool BWD, int DIR>
__device__ __forceinline__ void lattice_side(const float4 *__restrict__ Gtab, const float4 *__restrict__ Htab, LatPair &s0,
                                             LatPair &s1, int jmax)
{
    const float2 one = f2(1.0f);
    const float2 b0 = DIR > 0 ? s0.bu : s0.bd, b1 = DIR > 0 ? s1.bu : s1.bd;
    float2 w0 = b0, w1 = b1;               // b^j - 1
    for (int j = 1; j <= jmax; ++j) {
        const float4 ga = Gtab[j];
        const float4 ha = BWD ? Htab[j] : ga;
        lattice_add<BWD, DIR>(s0, ga, ha, __fadd2_rn(w0, one));
        lattice_add<BWD, DIR>(s1, ga, ha, __fadd2_rn(w1, one));
        w0 = __fadd2_rn(w0, __ffma2_rn(w0, b0, b0));
        w1 = __fadd2_rn(w1, __ffma2_rn(w1, b1, b1));
    }
}

template <int MODE>
__device__ __forceinline__ PairOut lattice_finish(const QuantDev &P, const LatPair &s, float2 g)
{
    PairOut o;
    const float q = P.q;
    o.k0[0] = s.k0;
    o.k0[1] = s.k1;
    const float2 S = __fadd2_rn(s.A0, f2(1.0f));
    const float2 rS = make_float2(rcp_approx(S.x), rcp_approx(S.y));
    const float2 m1 = __fmul2_rn(s.A1, rS);
    // (0 * residual: zero for finite input; a NaN or infinite input, whose B was clamped above, still gives NaN)
    o.y = __ffma2_rn(s.kn, f2(q), __ffma2_rn(f2(q), m1, __fmul2_rn(s.dh, f2(0.0f))));
    o.gx = o.tq = o.ta = f2(0.0f);
    if (MODE == MODE_BWD) {
        const float2 m2 = __fmul2_rn(s.A2, rS), m3 = __fmul2_rn(s.A3, rS);
        const float2 nm1 = __fmul2_rn(m1, f2(-1.0f));
        const float2 varj = __ffma2_rn(nm1, m1, m2);
        const float2 covj = __ffma2_rn(nm1, m2, m3);
        o.gx = __fmul2_rn(g, __fmul2_rn(f2(P.a2), varj));
        const float2 qc = __fmul2_rn(f2(q), covj);
        const float2 dmk = __ffma2_rn(s.kn, f2(-q), s.dh);             // d - kn q
        o.tq = __ffma2_rn(f2(P.two_aq), sub2(__fmul2_rn(dmk, varj), qc), __fadd2_rn(s.kn, m1));
        o.ta = __fmul2_rn(f2(P.q2), sub2(__fmul2_rn(__fmul2_rn(f2(2.0f), s.dh), varj), qc));
    }
    return o;
}

// the four elements of a load whose hard indices s0, s1 already hold; all four have jmax levels on either side
template <int MODE>
__device__ __forceinline__ void quant_quad_lattice(const QuantDev &P, const float4 *__restrict__ Gtab,
                                                   const float4 *__restrict__ Htab, const float (&xs)[4],
                                                   const float (&gs)[4], LatPair &s0, LatPair &s1, PairOut (&o)[2])
{
    constexpr bool kBwd = MODE == MODE_BWD;
    lattice_setup(P, make_float2(xs[0], xs[1]), s0);
    lattice_setup(P, make_float2(xs[2], xs[3]), s1);
    lattice_side<kBwd, 1>(Gtab, Htab, s0, s1, P.jmax);
    lattice_side<kBwd, -1>(Gtab, Htab, s0, s1, P.jmax);
    o[0] = lattice_finish<MODE>(P, s0, make_float2(gs[0], gs[1]));
    o[1] = lattice_finish<MODE>(P, s1, make_float2(gs[2], gs[3]));
}

// ---- thread-block cluster helpers (a launch without a cluster attribute is a cluster of one CTA)
__device__ __forceinline__ unsigned int cluster_ctarank()
{
    unsigned int r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned int cluster_nctarank()
{
    unsigned int r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the 64-bit word at the same shared-memory offset as `p` in CTA `rank` of the cluster
__device__ __forceinline__ unsigned long long ld_cluster_u64(const unsigned long long *p, unsigned int rank)
{
    unsigned long long v;
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %1, %2;\n\t"
        "ld.shared::cluster.u64 %0, [ra];\n\t}"
        : "=l"(v)
        : "r"((unsigned int)__cvta_generic_to_shared(p)), "r"(rank)
        : "memory");
    return v;
}

// One more element at level k.  hist_a is the 32-bit shared-window address of this lane's counter of level 0 (the
// counters of one level are 32 consecutive words, one per lane, so a warp never meets a bank conflict): one address
// computation and one reduction per element.
__device__ __forceinline__ void hist_inc(unsigned int hist_a, int k)
{
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(hist_a + ((unsigned int)k << 7)), "r"(1u) : "memory");
}

// Vector region: elements [head, head + 4 n4); the remaining head + tail elements are done one by one.
// When the pointers do not allow 128-bit access the host passes n4 = 0 and everything is scalar.
template <int MODE, int PATH, bool RATE>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const QuantDev P, const float *__restrict__ x, const float *__restrict__ g, int64_t n,
                int64_t head, int64_t n4, float *__restrict__ y, unsigned char *__restrict__ idx,
                unsigned long long *__restrict__ hist, float *__restrict__ gx,
                double *__restrict__ gq, double *__restrict__ ga, unsigned long long *__restrict__ mp)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Ltab = reinterpret_cast<float *>(smem_raw);                       // CDL_MAX_LEVELS floats
    unsigned int *hist_s = reinterpret_cast<unsigned int *>(smem_raw + CDL_MAX_LEVELS * sizeof(float));
    const int lane = threadIdx.x & 31;
    const bool do_hist = hist != nullptr;
    // soft histogram (sum of CPMFs per level, fixed point): bins behind the index histogram's, only when asked for
    unsigned long long *mp_s = nullptr;
    if (MODE == MODE_SOFT && RATE) {
        mp_s = reinterpret_cast<unsigned long long *>(smem_raw + CDL_MAX_LEVELS * sizeof(float) +
                                                      (do_hist ? (size_t)P.nlev * 32 * sizeof(unsigned int) : 0));
        for (int k = threadIdx.x; k < P.nlev * 32; k += kThreads) mp_s[k] = 0ull;
    }

    // LATTICE: (G_j, G_j, j G_j, j G_j) and (j^2 G_j, j^2 G_j, j^3 G_j, j^3 G_j), G_j = 2^(-A j^2), for the level j steps
    // from the nearest one; every entry twice so that a 128-bit load yields two packed operands
    __shared__ float4 Gtab[PATH == PATH_LATTICE ? CDL_MAX_LEVELS : 1];
    __shared__ float4 Htab[(PATH == PATH_LATTICE && MODE == MODE_BWD) ? CDL_MAX_LEVELS : 1];
    if (PATH == PATH_LATTICE) {
        for (int j = threadIdx.x; j < CDL_MAX_LEVELS; j += kThreads) {
            const float jf = (float)j;
            const float G = exp2f(__fmul_rn(__fmul_rn(-P.A, jf), jf)), jG = __fmul_rn(jf, G), j2G = __fmul_rn(jf, jG);
            Gtab[j] = make_float4(G, G, jG, jG);
            if (MODE == MODE_BWD) {
                const float j3G = __fmul_rn(jf, j2G);
                Htab[j] = make_float4(j2G, j2G, j3G, j3G);
            }
        }
    }
    constexpr bool kPairRate = MODE == MODE_BWD && RATE && PATH == PATH_NEAR3;
    __shared__ float2 Dtab[kPairRate ? CDL_MAX_LEVELS : 1];     // (L[k+1] - L[k], L[k-1] - L[k]), clamped at the ends
    if (MODE == MODE_BWD && RATE) {
        auto log2p = [&](int k) {
            const float p = P.level_prob[k];
            return (p < 9.31322574615478515625e-10f) ? -30.0f : log2f(p);   // 2^-30
        };
        for (int k = threadIdx.x; k < P.nlev; k += kThreads) {
            const float Lk = log2p(k);
            Ltab[k] = Lk;
            if (kPairRate) Dtab[k] = make_float2(log2p(min(k + 1, P.nlev - 1)) - Lk, log2p(max(k - 1, 0)) - Lk);
        }
    }
    if (do_hist)
        for (int k = threadIdx.x; k < P.nlev * 32; k += kThreads) hist_s[k] = 0u;
    if (RATE || do_hist || PATH == PATH_LATTICE) __syncthreads();

    // this lane's column of the index histogram, addressed by level: level k sits at hist_a + 128 k
    const unsigned int hist_a = (unsigned int)__cvta_generic_to_shared(hist_s) + (unsigned int)((lane - P.lo * 32) * 4);
    double acc_q = 0.0, acc_a = 0.0;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;

    const float4 *x4 = reinterpret_cast<const float4 *>(x + head);
    const float4 *g4 = reinterpret_cast<const float4 *>(g + head);
    float4 *y4 = reinterpret_cast<float4 *>(y + head);
    float4 *gx4 = reinterpret_cast<float4 *>(gx + head);
    unsigned int *idx4 = reinterpret_cast<unsigned int *>(idx + head);

    // One 128-bit group (four elements): quantize, store, count.  The running sums of the scalar gradients are kept
    // across the groups of a batch and flushed to double precision after it.
    float part_q = 0.0f, part_a = 0.0f;
    float2 part_q2 = make_float2(0.0f, 0.0f), part_a2 = make_float2(0.0f, 0.0f);    // pair path: two running sums each
    auto group = [&](const float4 xq, const float4 gq, const int64_t i, float4 *yp, float4 *gxp, unsigned int *ip) {
        const float xs[4] = {xq.x, xq.y, xq.z, xq.w};
        float gs[4] = {0.f, 0.f, 0.f, 0.f};
        if (MODE == MODE_BWD) {
            gs[0] = gq.x;
            gs[1] = gq.y;
            gs[2] = gq.z;
            gs[3] = gq.w;
        }
        if (MODE == MODE_SAMPLE) {
            // the uniform numbers of elements e0 .. e0+3: one Philox block when e0 is a multiple of 4
            const unsigned long long e0 = P.first_index + (unsigned long long)(head + 4 * i);
            if ((e0 & 3ull) == 0ull) {
                const uint4 r = philox4x32_10(e0 >> 2, P.seed);
                gs[0] = u01(r.x);
                gs[1] = u01(r.y);
                gs[2] = u01(r.z);
                gs[3] = u01(r.w);
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) gs[c] = philox_uniform(P.seed, e0 + c);
            }
        }
        float ys[4], gxs[4];
        unsigned int packed = 0u;
        constexpr bool kPairs = (PATH == PATH_NEAR3 && (MODE == MODE_BWD || MODE == MODE_SAMPLE || (MODE == MODE_SOFT && !RATE))) ||
                                (PATH == PATH_LATTICE && !RATE && (MODE == MODE_BWD || MODE == MODE_SOFT));
        // LATTICE: the table form serves a warp all of whose elements have jmax levels on either side of
        // their nearest one; a warp with an element near the edge of the index set (or outside it) takes
        // the level loop, which visits exactly each element's levels
        bool use_pairs = kPairs;
        PairOut quad[2];
        if (PATH == PATH_LATTICE && kPairs) {
            LatPair s0, s1;
            lattice_index(P, make_float2(xs[0], xs[1]), s0);
            lattice_index(P, make_float2(xs[2], xs[3]), s1);
            const int klo = P.lo + P.jmax, khi = P.hi - P.jmax;
            const bool inner = min(min(s0.k0, s0.k1), min(s1.k0, s1.k1)) >= klo &&
                               max(max(s0.k0, s0.k1), max(s1.k0, s1.k1)) <= khi;
            use_pairs = __all_sync(__activemask(), inner);
            if (use_pairs) quant_quad_lattice<MODE>(P, Gtab, Htab, xs, gs, s0, s1, quad);
        }
        if (kPairs && use_pairs) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float2 xp = make_float2(xs[2 * h], xs[2 * h + 1]), gp = make_float2(gs[2 * h], gs[2 * h + 1]);
                const PairOut o = PATH == PATH_LATTICE ? quad[h] : quant_pair_near3<MODE, RATE>(P, Dtab, xp, gp);
                ys[2 * h] = o.y.x;
                ys[2 * h + 1] = o.y.y;
                gxs[2 * h] = o.gx.x;
                gxs[2 * h + 1] = o.gx.y;
                if (MODE == MODE_BWD) {
                    const float2 gg = make_float2(gs[2 * h], gs[2 * h + 1]);
                    part_q2 = __ffma2_rn(gg, o.tq, part_q2);
                    part_a2 = __ffma2_rn(gg, o.ta, part_a2);
                }
                packed = h == 0 ? __byte_perm((unsigned int)o.k0[0], (unsigned int)o.k0[1], 0x0040)
                                : __byte_perm(packed, __byte_perm((unsigned int)o.k0[0], (unsigned int)o.k0[1], 0x0040), 0x5410);
                if (MODE != MODE_BWD && do_hist) {
                    hist_inc(hist_a, o.k0[0]);
                    hist_inc(hist_a, o.k0[1]);
                }
            }
        }
        if (MODE == MODE_HARD) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                int k0, k1;
                hard_pair(P, make_float2(xs[2 * h], xs[2 * h + 1]), k0, k1);
                packed = h == 0 ? __byte_perm((unsigned int)k0, (unsigned int)k1, 0x0040)
                                : __byte_perm(packed, __byte_perm((unsigned int)k0, (unsigned int)k1, 0x0040), 0x5410);
                if (do_hist) {
                    hist_inc(hist_a, k0);
                    hist_inc(hist_a, k1);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < (((kPairs && PATH != PATH_LATTICE) || MODE == MODE_HARD) ? 0 : 4); ++c) {
            if (kPairs && use_pairs) break;      // (only LATTICE decides this at run time; the bound stays constant)
            const ElemOut o = quant_elem<MODE, PATH, RATE>(P, Ltab, xs[c], gs[c], mp_s, lane);
            ys[c] = o.y;
            gxs[c] = o.gx;
            part_q += o.tq;
            part_a += o.ta;
            packed |= ((unsigned int)o.k0 & 0xffu) << (8 * c);
            if (MODE != MODE_BWD && do_hist) hist_inc(hist_a, o.k0);
        }
        if (MODE == MODE_SOFT || (MODE == MODE_SAMPLE && y != nullptr)) CDL_ST(yp, make_float4(ys[0], ys[1], ys[2], ys[3]));
        if (MODE == MODE_BWD && gx != nullptr) CDL_ST(gxp, make_float4(gxs[0], gxs[1], gxs[2], gxs[3]));
        if (MODE != MODE_BWD && idx != nullptr) *ip = packed;
    };
    auto flush_partials = [&]() {
        if (MODE == MODE_BWD) {
            acc_q += (double)(part_q + (part_q2.x + part_q2.y));
            acc_a += (double)(part_a + (part_a2.x + part_a2.y));
            part_q = part_a = 0.0f;
            part_q2 = part_a2 = make_float2(0.0f, 0.0f);
        }
    };

    // Whole batches first (kBatch loads in flight, no bounds checks inside), then the at most kBatch - 1 groups left
    // over; every stream is walked with a running pointer, so a step costs additions, not 64-bit address arithmetic.
    {
        int64_t i = tid;
        const float4 *xp = x4 + i, *gp = g4 + i;
        float4 *yp = y4 + i, *gxp = gx4 + i;
        unsigned int *ip = idx4 + i;
        // (The level-loop paths have a long body that the arithmetic, not the loads, paces: they take the one-group
        // loop below for everything, which keeps a single copy of that body in the instruction cache.)
        constexpr bool kLongBody = MODE != MODE_HARD && (PATH == PATH_LOOP || PATH == PATH_LATTICE);
        const int64_t last_full = kLongBody ? 0 : n4 - (kBatch - 1) * stride;       // a batch starting below this is whole
        for (; i < last_full; i += kBatch * stride) {
            float4 xv[kBatch], gv[kBatch];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                xv[b] = CDL_LD(xp + b * stride);
                if (MODE == MODE_BWD) gv[b] = CDL_LD(gp + b * stride);
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b)
                group(xv[b], MODE == MODE_BWD ? gv[b] : make_float4(0.f, 0.f, 0.f, 0.f), i + b * stride, yp + b * stride, gxp + b * stride, ip + b * stride);
            flush_partials();
            xp += kBatch * stride;
            gp += kBatch * stride;
            yp += kBatch * stride;
            gxp += kBatch * stride;
            ip += kBatch * stride;
        }
        for (; i < n4; i += stride) {
            const float4 xq = CDL_LD(xp);
            const float4 gq = MODE == MODE_BWD ? CDL_LD(gp) : make_float4(0.f, 0.f, 0.f, 0.f);
            group(xq, gq, i, yp, gxp, ip);
            flush_partials();
            xp += stride;
            gp += stride;
            yp += stride;
            gxp += stride;
            ip += stride;
        }
    }

    // scalar remainder: elements [0, head) and [head + 4 n4, n)
    const int64_t tail0 = head + 4 * n4;
    const int64_t nrem = head + (n - tail0);
    for (int64_t t = tid; t < nrem; t += stride) {
        const int64_t i = (t < head) ? t : (tail0 + (t - head));
        const float gi = (MODE == MODE_BWD) ? g[i]
                         : (MODE == MODE_SAMPLE) ? philox_uniform(P.seed, P.first_index + (unsigned long long)i) : 0.0f;
        const ElemOut o = quant_elem<MODE, PATH, RATE>(P, Ltab, x[i], gi, mp_s, lane);
        if (MODE == MODE_SOFT || (MODE == MODE_SAMPLE && y != nullptr)) y[i] = o.y;
        if (MODE == MODE_BWD) {
            if (gx != nullptr) gx[i] = o.gx;
            acc_q += (double)o.tq;
            acc_a += (double)o.ta;
        } else {
            if (idx != nullptr) idx[i] = (unsigned char)((unsigned int)o.k0 & 0xffu);
            if (do_hist) hist_inc(hist_a, o.k0);
        }
    }

    // Histograms leave the CTA in two steps.  Each CTA adds up its 32 lane-private columns; then the CTAs of a
    // thread-block cluster (kHistCluster of them when a histogram is asked for) read one another's totals through
    // distributed shared memory, every CTA taking the bins congruent to its rank, and only these cluster sums go to
    // global memory.  All blocks hit the same few addresses there, and those reductions are served one at a time:
    // with one reduction per bin per CTA they cost as much as a quarter of a launch on a 13 M-element tensor.
    const bool do_mp = MODE == MODE_SOFT && RATE;   // RATE doubles as "soft histogram requested" in the soft pass
    if (MODE != MODE_BWD && (do_hist || do_mp)) {
        unsigned long long *tot_c = reinterpret_cast<unsigned long long *>(
            smem_raw + CDL_MAX_LEVELS * sizeof(float) + (do_hist ? (size_t)P.nlev * 32 * sizeof(unsigned int) : 0) +
            (do_mp ? (size_t)P.nlev * 32 * sizeof(unsigned long long) : 0));
        unsigned long long *tot_m = tot_c + P.nlev;
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp; b < P.nlev; b += kThreads / 32) {
            if (do_hist) {
                const unsigned int c = __reduce_add_sync(0xffffffffu, hist_s[b * 32 + lane]);
                if (lane == 0) tot_c[b] = c;
            }
            if (do_mp) {
                unsigned long long c = mp_s[b * 32 + lane];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) c += __shfl_down_sync(0xffffffffu, c, off);
                if (lane == 0) tot_m[b] = c;
            }
        }
        cluster_sync_all();                        // every CTA's totals are in place (also orders them within the CTA)
        const unsigned int csize = cluster_nctarank(), crank = cluster_ctarank();
        for (int b = threadIdx.x; b < P.nlev; b += kThreads) {
            if ((unsigned int)b % csize != crank) continue;
            if (do_hist) {
                unsigned long long sum = 0ull;
                for (unsigned int r = 0; r < csize; ++r) sum += ld_cluster_u64(&tot_c[b], r);
                if (sum != 0ull) atomicAdd(&hist[b], sum);
            }
            if (do_mp) {
                unsigned long long sum = 0ull;
                for (unsigned int r = 0; r < csize; ++r) sum += ld_cluster_u64(&tot_m[b], r);
                if (sum != 0ull) atomicAdd(&mp[b], sum);
            }
        }
        cluster_sync_all();                        // no CTA leaves while another may still read its totals
    }
    if (MODE == MODE_BWD && (gq != nullptr || ga != nullptr)) {
        __shared__ double red[2][kThreads / 32];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            acc_q += __shfl_down_sync(0xffffffffu, acc_q, off);
            acc_a += __shfl_down_sync(0xffffffffu, acc_a, off);
        }
        if (lane == 0) {
            red[0][threadIdx.x >> 5] = acc_q;
            red[1][threadIdx.x >> 5] = acc_a;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            double sq = 0.0, sa = 0.0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) {
                sq += red[0][w];
                sa += red[1][w];
            }
            if (gq != nullptr) atomicAdd(gq, sq);
            if (ga != nullptr) atomicAdd(ga, sa);
        }
    }
}

template <int MODE, int PATH, bool RATE>
int launch_t(const QuantDev &qd, const float *x, const float *g, int64_t n, int64_t head, int64_t n4,
             float *y, unsigned char *idx, unsigned long long *hist, float *gx, double *gq, double *ga,
             unsigned long long *mp, cudaStream_t stream)
{
    const bool histo = MODE != MODE_BWD && (hist != nullptr || mp != nullptr);
    const size_t smem = CDL_MAX_LEVELS * sizeof(float) + (hist ? (size_t)qd.nlev * 32 * sizeof(unsigned int) : 0) +
                        (mp ? (size_t)qd.nlev * 32 * sizeof(unsigned long long) : 0) +
                        (histo ? 2 * (size_t)qd.nlev * sizeof(unsigned long long) : 0);     // per-CTA totals of both histograms
    auto kern = quantize_kernel<MODE, PATH, RATE>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, smem) != cudaSuccess || per_sm < 1) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    // one float4 group (or one scalar element) per thread until the device is full, then kBatch in flight each
    const int64_t work = (n4 > 0) ? n4 : n;
    int64_t blocks = (work + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)sms * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (!histo) {
        kern<<<(unsigned int)blocks, kThreads, smem, stream>>>(qd, x, g, n, head, n4, y, idx, hist, gx, gq, ga, mp);
        return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
    }
    // histogram launches: clusters of kHistCluster CTAs (CTAs without elements still take part in the reduction)
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kHistCluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned int)(cap / kHistCluster * kHistCluster));
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg) != cudaSuccess || max_clusters < 1) {
        (void)cudaGetLastError();
        max_clusters = (int)(cap / kHistCluster) > 0 ? (int)(cap / kHistCluster) : 1;
    }
    int64_t clusters = (blocks + kHistCluster - 1) / kHistCluster;
    if (clusters > max_clusters) clusters = max_clusters;
    cfg.gridDim = dim3((unsigned int)(clusters * kHistCluster));
    if (cudaLaunchKernelEx(&cfg, kern, qd, x, g, n, head, n4, y, idx, hist, gx, gq, ga, mp) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    return CDL_OK;
}

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

int launch_quantize(int mode, const float *x, const float *grad_out, int64_t n, const QuantDev &qd,
                    float *y, void *idx, unsigned long long *hist, bool hist_accumulate,
                    float *grad_x, double *grad_q, double *grad_alpha, unsigned long long *soft_hist,
                    cudaStream_t stream)
{
    if (soft_hist != nullptr && !hist_accumulate) {
        if (cudaMemsetAsync(soft_hist, 0, (size_t)qd.nlev * sizeof(unsigned long long), stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }
    if (hist != nullptr && !hist_accumulate) {
        if (cudaMemsetAsync(hist, 0, (size_t)qd.nlev * sizeof(unsigned long long), stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }
    if (mode == MODE_BWD) {
        if (grad_q != nullptr && grad_alpha == grad_q + 1) {       // adjacent scalars: one clear
            if (cudaMemsetAsync(grad_q, 0, 2 * sizeof(double), stream) != cudaSuccess) return CDL_ERR_LAUNCH;
        } else {
            if (grad_q && cudaMemsetAsync(grad_q, 0, sizeof(double), stream) != cudaSuccess) return CDL_ERR_LAUNCH;
            if (grad_alpha && cudaMemsetAsync(grad_alpha, 0, sizeof(double), stream) != cudaSuccess) return CDL_ERR_LAUNCH;
        }
    }
    if (n == 0) return CDL_OK;

    // 128-bit path: skip `head` elements so that x is 16-byte aligned; every other stream must then be
    // aligned at the same element offset (16 bytes for floats, 4 bytes for the packed index bytes).
    int64_t head = (int64_t)((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4;
    if (head > n) head = n;
    bool vec = true;
    if (mode == MODE_SOFT || (mode == MODE_SAMPLE && y != nullptr)) vec = vec && aligned_to(y + head, 16);
    if (mode == MODE_BWD) {
        vec = vec && aligned_to(grad_out + head, 16);
        if (grad_x) vec = vec && aligned_to(grad_x + head, 16);
    }
    if (mode != MODE_BWD && idx) vec = vec && aligned_to(static_cast<unsigned char *>(idx) + head, 4);
    int64_t n4 = vec ? (n - head) / 4 : 0;
    if (n4 == 0) head = 0;

    unsigned char *ib = static_cast<unsigned char *>(idx);
    // NEAR3 sums the nearest level and its two neighbours whatever the window: right for the whole index set and for
    // any window of three or more (what it leaves out weighs < e^-24), wrong for a window of one, which keeps the
    // nearest level alone (zero variance and gradient): that one takes the level loop, which honours the window.
    const int path = (qd.near3 && qd.window != 1) ? PATH_NEAR3 : (qd.window == 5 ? PATH_WIN5 : PATH_LOOP);
    const bool rate = (mode == MODE_BWD) && qd.level_prob != nullptr && qd.rate_c != 0.0f;
    // Whole index set, a window of +-jmax levels that is narrower than the index set and wide enough to pay for the
    // per-element set-up (jmax >= 8), vector region present, no soft histogram and no rate term: the table form of
    // the level sums for the warps whose elements all lie jmax levels inside the index set.  (Measured: with the
    // rate term - two more per-lane table loads per level - it was no faster; letting elements near the edges take
    // part, with per-element level counts and masks, made a warp walk both sides to its longest lane's end and
    // lost more than it gained on heavy-tailed data.)
    const bool lattice = path == PATH_LOOP && qd.window == 0 && n4 > 0 && qd.jmax >= 8 && 2 * qd.jmax + 1 < qd.nlev && !rate &&
                         ((mode == MODE_SOFT && soft_hist == nullptr) || mode == MODE_BWD);
#define CDL_Q(M, PTH, RT) \
    launch_t<M, PTH, RT>(qd, x, grad_out, n, head, n4, y, ib, hist, grad_x, grad_q, grad_alpha, soft_hist, stream)
    switch (mode) {
        case MODE_HARD:
            return CDL_Q(MODE_HARD, PATH_LOOP, false);
        case MODE_SOFT:
            if (soft_hist != nullptr)
                return path == PATH_NEAR3 ? CDL_Q(MODE_SOFT, PATH_NEAR3, true)
                     : path == PATH_WIN5 ? CDL_Q(MODE_SOFT, PATH_WIN5, true)
                                         : CDL_Q(MODE_SOFT, PATH_LOOP, true);
            if (lattice) return CDL_Q(MODE_SOFT, PATH_LATTICE, false);
            return path == PATH_NEAR3 ? CDL_Q(MODE_SOFT, PATH_NEAR3, false)
                 : path == PATH_WIN5 ? CDL_Q(MODE_SOFT, PATH_WIN5, false)
                                     : CDL_Q(MODE_SOFT, PATH_LOOP, false);
        case MODE_SAMPLE:
            return path == PATH_NEAR3 ? CDL_Q(MODE_SAMPLE, PATH_NEAR3, false)
                 : path == PATH_WIN5 ? CDL_Q(MODE_SAMPLE, PATH_WIN5, false)
                                     : CDL_Q(MODE_SAMPLE, PATH_LOOP, false);
        case MODE_BWD:
            if (lattice) return CDL_Q(MODE_BWD, PATH_LATTICE, false);
            if (rate)
                return path == PATH_NEAR3 ? CDL_Q(MODE_BWD, PATH_NEAR3, true)
                     : path == PATH_WIN5 ? CDL_Q(MODE_BWD, PATH_WIN5, true)
                                         : CDL_Q(MODE_BWD, PATH_LOOP, true);
            return path == PATH_NEAR3 ? CDL_Q(MODE_BWD, PATH_NEAR3, false)
                 : path == PATH_WIN5 ? CDL_Q(MODE_BWD, PATH_WIN5, false)
                                     : CDL_Q(MODE_BWD, PATH_LOOP, false);
        default:
            return CDL_ERR_ARG;
    }
#undef CDL_Q
}

// ------------------------------------------------------------------------------------------------
// Entropy of a level histogram (Sec. III-A definition, base 2): one CTA, fixed-order tree reduction,
// double precision.  nlev <= 256.
namespace {
__global__ void __launch_bounds__(CDL_MAX_LEVELS)
entropy_kernel(const unsigned long long *__restrict__ hist, int nlev, double *__restrict__ H,
               float *__restrict__ prob, unsigned long long *__restrict__ n_out)
{
    __shared__ unsigned long long cnt[CDL_MAX_LEVELS];
    __shared__ double term[CDL_MAX_LEVELS];
    const int t = threadIdx.x;
    const unsigned long long c = (t < nlev) ? hist[t] : 0ull;
    cnt[t] = c;
    __syncthreads();
    for (int s = CDL_MAX_LEVELS / 2; s > 0; s >>= 1) {
        if (t < s) cnt[t] += cnt[t + s];
        __syncthreads();
    }
    const unsigned long long n = cnt[0];
    const double p = (n != 0ull) ? (double)c / (double)n : 0.0;
    term[t] = (p > 0.0) ? -p * log2(p) : 0.0;
    if (prob != nullptr && t < nlev) prob[t] = (float)p;
    __syncthreads();
    for (int s = CDL_MAX_LEVELS / 2; s > 0; s >>= 1) {
        if (t < s) term[t] += term[t + s];
        __syncthreads();
    }
    if (t == 0) {
        *H = term[0];
        if (n_out != nullptr) *n_out = n;
    }
}
}  // namespace

int launch_entropy(const unsigned long long *hist, int nlev, double *H, float *prob,
                   unsigned long long *n_out, cudaStream_t stream)
{
    entropy_kernel<<<1, CDL_MAX_LEVELS, 0, stream>>>(hist, nlev, H, prob, n_out);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace cdl
