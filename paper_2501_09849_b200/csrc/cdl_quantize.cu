// Quantizer kernels of the CDL layer for sm_100a: hard index + histogram, soft value Q_d,
// analytic backward.  One pass over the tensor each; HBM-bound by design.
//
// Arithmetic (per element theta, Sec. IV of the paper):
//   k0  = clamp(rint(theta / q))                 the hard index (binary32 quotient, ties to even)
//   d   = theta - kn q  as an unevaluated sum dh + dl of two floats (kn = nearest in-range level):
//         k0 q is split exactly with one fma, theta - fl(k0 q) is exact (operands within a factor
//         of two), so d carries ~48 bits.  This matters next to the midpoints between levels when
//         alpha q^2 is large: there dQ_d/dtheta ~ alpha q^2 / 2 and a 2^-24 error in d is visible.
//   e_j = exp(-alpha ((d - j q)^2 - d^2)) = 2^(-c1 j (j q - 2 d)),  c1 = alpha q log2 e,
//         the CPMF of Eq. (4) relative to level kn: P_{kn+j} = e_j / sum_j e_j, e_0 = 1, e_j <= 1.
//   J   = index offset from kn under that CPMF; moments m1 = E J, m2 = E J^2, m3 = E J^3.
//   Q_d = kn q + q m1                                                   (Eq. (8))
//   dQ_d/dtheta = 2 alpha q^2 Var J                                      (Lemma 1, Eq. (9a))
//   dQ_d/dq     = kn + m1 + 2 alpha q ((d - kn q) Var J - q Cov(J, J^2)) (Eq. (9b), re-centred on kn)
//   dQ_d/dalpha = q^2 (2 d Var J - q Cov(J, J^2))                        (Appendix B steps, re-centred)
//   rate term   = rate_weight * (-2 alpha q) * (E[L J] - m1 E[L]),  L = log2 of the level probability.
// The re-centred forms equal the printed ones (expand X = q (kn + J)) without their cancellation.
//
// Window of 5 (Sec. VI-B.1): the five in-range levels nearest theta form a contiguous block that
// contains kn.  Their e_j come from two ex2 (j = +1, -1) and the lattice recurrence
// e_{j+1} = e_j r_j, r_{j+1} = r_j exp(-2 alpha q^2), which keeps the MUFU count at 2 per element.
#include "cdl_internal.h"

#include <math.h>

namespace cdl {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 4;  // float4 loads in flight per thread

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct ElemOut {
    int k0;       // hard index
    float y;      // Q_d
    float gx;     // grad wrt theta
    float tq;     // g * dQ_d/dq
    float ta;     // g * dQ_d/dalpha
};

template <int MODE, bool WIN5, bool RATE>
__device__ __forceinline__ ElemOut quant_elem(const QuantDev &P, const float *__restrict__ Ltab, float x, float g)
{
    ElemOut o;
    // ---- hard index: the defining binary32 expression
    const float u = __fdiv_rn(x, P.q);
    float r = rintf(u);
    r = (r != r) ? 0.0f : r;
    const float k0 = fminf(fmaxf(r, P.flo), P.fhi);
    o.k0 = (int)k0;
    o.y = 0.0f;
    o.gx = 0.0f;
    o.tq = 0.0f;
    o.ta = 0.0f;
    if (MODE == MODE_HARD) return o;

    // ---- d = theta - k0 q as dh + dl
    const float q = P.q;
    const float ph = __fmul_rn(k0, q);
    const float pl = __fmaf_rn(k0, q, -ph);
    const float s = __fsub_rn(x, ph);
    float dh = __fsub_rn(s, pl);
    const float dl = __fsub_rn(__fsub_rn(s, dh), pl);
    float kn = k0;
    int jlo, jhi;
    if (P.window > 0) {
        // exact nearest level; of two equally near levels the lower one
        const bool up = (dh > P.half_q || (dh == P.half_q && dl > 0.0f)) && (kn < P.fhi);
        if (up) {
            kn += 1.0f;
            dh = __fsub_rn(dh, q);
        }
        const bool dn = (dh < -P.half_q || (dh == -P.half_q && dl <= 0.0f)) && (kn > P.flo);
        if (dn) {
            kn -= 1.0f;
            dh = __fadd_rn(dh, q);
        }
        const int kni = (int)kn;
        const int st = min(max(kni - (P.window >> 1), P.lo), P.hi - P.window + 1);
        jlo = st - kni;
        jhi = jlo + P.window - 1;
    } else {
        const int kni = (int)kn;
        jlo = max(P.lo - kni, -P.jmax);
        jhi = min(P.hi - kni, P.jmax);
    }
    const int kni = (int)kn;
    const float m2d = -2.0f * dh;
    const float dl2 = 2.0f * dl;

    // The rate term is a covariance with L, so L may be shifted by a constant: measuring it from the
    // nearest level's value makes the j = 0 term vanish and a flat L give exactly zero.
    float S = 1.0f, S1 = 0.0f, S2 = 0.0f, S3 = 0.0f, R0 = 0.0f, R1 = 0.0f;
    const float Lc = RATE ? Ltab[kni - P.lo] : 0.0f;

    if (WIN5) {
        const float w1 = __fsub_rn(__fadd_rn(q, m2d), dl2);   // (q - 2 dh) - 2 dl
        const float wm = __fadd_rn(__fsub_rn(q, m2d), dl2);   // (q + 2 dh) + 2 dl
        const float e1 = ex2_approx(-P.c1 * w1);
        const float em = ex2_approx(-P.c1 * wm);
        const int nneg = -jlo;  // levels below kn in the window: 0..4
        float e = 1.0f, rr = em;
#pragma unroll
        for (int i = 1; i <= 4; ++i) {
            if (i == nneg + 1) {  // switch from the downward to the upward chain
                e = 1.0f;
                rr = e1;
            }
            e *= rr;
            rr *= P.decay;
            const int j = (i <= nneg) ? -i : (i - nneg);
            const float jf = (float)j;
            S += e;
            S1 = fmaf(jf, e, S1);
            if (MODE == MODE_BWD) {
                const float j2 = jf * jf;
                S2 = fmaf(j2, e, S2);
                S3 = fmaf(j2 * jf, e, S3);
                if (RATE) {
                    const float le = (Ltab[kni - P.lo + j] - Lc) * e;
                    R0 += le;
                    R1 = fmaf(jf, le, R1);
                }
            }
        }
    } else {
        for (int j = jlo; j <= jhi; ++j) {
            if (j == 0) continue;
            const float jf = (float)j;
            const float w = __fsub_rn(__fmaf_rn(jf, q, m2d), dl2);   // (j q - 2 dh) - 2 dl
            const float e = ex2_approx((-P.c1 * jf) * w);
            S += e;
            S1 = fmaf(jf, e, S1);
            if (MODE == MODE_BWD) {
                const float j2 = jf * jf;
                S2 = fmaf(j2, e, S2);
                S3 = fmaf(j2 * jf, e, S3);
                if (RATE) {
                    const float le = (Ltab[kni - P.lo + j] - Lc) * e;
                    R0 += le;
                    R1 = fmaf(jf, le, R1);
                }
            }
        }
    }
    const float rS = __frcp_rn(S);
    const float m1 = S1 * rS;
    o.y = __fmaf_rn(kn, q, __fmul_rn(q, m1));
    if (MODE == MODE_BWD) {
        const float m2 = S2 * rS;
        const float m3 = S3 * rS;
        const float varj = fmaf(-m1, m1, m2);
        const float cov3 = fmaf(-m1, m2, m3);
        float gx = g * (P.a2 * varj);
        if (RATE) gx = fmaf(P.rate_c, (R1 - m1 * R0) * rS, gx);
        o.gx = gx;
        const float dmk = fmaf(-kn, q, dh);  // d - kn q
        const float dq = (kn + m1) + P.two_aq * (dmk * varj - q * cov3);
        const float da = P.q2 * (2.0f * dh * varj - q * cov3);
        o.tq = g * dq;
        o.ta = g * da;
    }
    return o;
}

__device__ __forceinline__ void hist_add(unsigned int *hist_s, int bin, int lane)
{
    atomicAdd(&hist_s[bin * 32 + lane], 1u);
}

// Vector region: elements [head, head + 4 n4); the remaining head + tail elements are done one by one.
// When the pointers do not allow 128-bit access the host passes n4 = 0 and everything is scalar.
template <int MODE, bool WIN5, bool RATE>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const QuantDev P, const float *__restrict__ x, const float *__restrict__ g, int64_t n,
                int64_t head, int64_t n4, float *__restrict__ y, unsigned char *__restrict__ idx,
                unsigned long long *__restrict__ hist, float *__restrict__ gx,
                double *__restrict__ gq, double *__restrict__ ga)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Ltab = reinterpret_cast<float *>(smem_raw);                       // CDL_MAX_LEVELS floats
    unsigned int *hist_s = reinterpret_cast<unsigned int *>(smem_raw + CDL_MAX_LEVELS * sizeof(float));
    const int lane = threadIdx.x & 31;
    const bool do_hist = hist != nullptr;

    if (RATE) {
        for (int k = threadIdx.x; k < P.nlev; k += kThreads) {
            const float p = P.level_prob[k];
            Ltab[k] = (p < 9.31322574615478515625e-10f) ? -30.0f : log2f(p);   // 2^-30
        }
    }
    if (do_hist)
        for (int k = threadIdx.x; k < P.nlev * 32; k += kThreads) hist_s[k] = 0u;
    if (RATE || do_hist) __syncthreads();

    double acc_q = 0.0, acc_a = 0.0;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;

    const float4 *x4 = reinterpret_cast<const float4 *>(x + head);
    const float4 *g4 = reinterpret_cast<const float4 *>(g + head);
    float4 *y4 = reinterpret_cast<float4 *>(y + head);
    float4 *gx4 = reinterpret_cast<float4 *>(gx + head);
    unsigned int *idx4 = reinterpret_cast<unsigned int *>(idx + head);

    for (int64_t base = tid; base < n4; base += stride * kBatch) {
        float4 xv[kBatch], gv[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int64_t i = base + b * stride;
            if (i < n4) {
                xv[b] = __ldcs(x4 + i);
                if (MODE == MODE_BWD) gv[b] = __ldcs(g4 + i);
            }
        }
        float part_q = 0.0f, part_a = 0.0f;
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int64_t i = base + b * stride;
            if (i < n4) {
                const float xs[4] = {xv[b].x, xv[b].y, xv[b].z, xv[b].w};
                float gs[4] = {0.f, 0.f, 0.f, 0.f};
                if (MODE == MODE_BWD) {
                    gs[0] = gv[b].x;
                    gs[1] = gv[b].y;
                    gs[2] = gv[b].z;
                    gs[3] = gv[b].w;
                }
                float ys[4], gxs[4];
                unsigned int packed = 0u;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const ElemOut o = quant_elem<MODE, WIN5, RATE>(P, Ltab, xs[c], gs[c]);
                    ys[c] = o.y;
                    gxs[c] = o.gx;
                    part_q += o.tq;
                    part_a += o.ta;
                    packed |= ((unsigned int)o.k0 & 0xffu) << (8 * c);
                    if (MODE != MODE_BWD && do_hist) hist_add(hist_s, o.k0 - P.lo, lane);
                }
                if (MODE == MODE_SOFT) __stcs(y4 + i, make_float4(ys[0], ys[1], ys[2], ys[3]));
                if (MODE == MODE_BWD && gx != nullptr) __stcs(gx4 + i, make_float4(gxs[0], gxs[1], gxs[2], gxs[3]));
                if (MODE != MODE_BWD && idx != nullptr) idx4[i] = packed;
            }
        }
        if (MODE == MODE_BWD) {
            acc_q += (double)part_q;
            acc_a += (double)part_a;
        }
    }

    // scalar remainder: elements [0, head) and [head + 4 n4, n)
    const int64_t tail0 = head + 4 * n4;
    const int64_t nrem = head + (n - tail0);
    for (int64_t t = tid; t < nrem; t += stride) {
        const int64_t i = (t < head) ? t : (tail0 + (t - head));
        const float gi = (MODE == MODE_BWD) ? g[i] : 0.0f;
        const ElemOut o = quant_elem<MODE, WIN5, RATE>(P, Ltab, x[i], gi);
        if (MODE == MODE_SOFT) y[i] = o.y;
        if (MODE == MODE_BWD) {
            if (gx != nullptr) gx[i] = o.gx;
            acc_q += (double)o.tq;
            acc_a += (double)o.ta;
        } else {
            if (idx != nullptr) idx[i] = (unsigned char)((unsigned int)o.k0 & 0xffu);
            if (do_hist) hist_add(hist_s, o.k0 - P.lo, lane);
        }
    }

    if (MODE != MODE_BWD && do_hist) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp; b < P.nlev; b += kThreads / 32) {
            const unsigned int c = __reduce_add_sync(0xffffffffu, hist_s[b * 32 + lane]);
            if (lane == 0 && c != 0u) atomicAdd(&hist[b], (unsigned long long)c);
        }
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

template <int MODE, bool WIN5, bool RATE>
int launch_t(const QuantDev &qd, const float *x, const float *g, int64_t n, int64_t head, int64_t n4,
             float *y, unsigned char *idx, unsigned long long *hist, float *gx, double *gq, double *ga,
             cudaStream_t stream)
{
    const size_t smem = CDL_MAX_LEVELS * sizeof(float) + (hist ? (size_t)qd.nlev * 32 * sizeof(unsigned int) : 0);
    auto kern = quantize_kernel<MODE, WIN5, RATE>;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, smem) != cudaSuccess || per_sm < 1) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    const int64_t work = (n4 > 0) ? n4 : n;   // float4 groups, or single elements on the scalar path
    int64_t blocks = (work + (int64_t)kThreads * kBatch - 1) / ((int64_t)kThreads * kBatch);
    const int64_t cap = (int64_t)sms * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    kern<<<(unsigned int)blocks, kThreads, smem, stream>>>(qd, x, g, n, head, n4, y, idx, hist, gx, gq, ga);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

int launch_quantize(int mode, const float *x, const float *grad_out, int64_t n, const QuantDev &qd,
                    float *y, void *idx, unsigned long long *hist, bool hist_accumulate,
                    float *grad_x, double *grad_q, double *grad_alpha, cudaStream_t stream)
{
    if (hist != nullptr && !hist_accumulate) {
        if (cudaMemsetAsync(hist, 0, (size_t)qd.nlev * sizeof(unsigned long long), stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }
    if (mode == MODE_BWD) {
        if (grad_q && cudaMemsetAsync(grad_q, 0, sizeof(double), stream) != cudaSuccess) return CDL_ERR_LAUNCH;
        if (grad_alpha && cudaMemsetAsync(grad_alpha, 0, sizeof(double), stream) != cudaSuccess) return CDL_ERR_LAUNCH;
    }
    if (n == 0) return CDL_OK;

    // 128-bit path: skip `head` elements so that x is 16-byte aligned; every other stream must then be
    // aligned at the same element offset (16 bytes for floats, 4 bytes for the packed index bytes).
    int64_t head = (int64_t)((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4;
    if (head > n) head = n;
    bool vec = true;
    if (mode == MODE_SOFT) vec = vec && aligned_to(y + head, 16);
    if (mode == MODE_BWD) {
        vec = vec && aligned_to(grad_out + head, 16);
        if (grad_x) vec = vec && aligned_to(grad_x + head, 16);
    }
    if (mode != MODE_BWD && idx) vec = vec && aligned_to(static_cast<unsigned char *>(idx) + head, 4);
    int64_t n4 = vec ? (n - head) / 4 : 0;
    if (n4 == 0) head = 0;

    unsigned char *ib = static_cast<unsigned char *>(idx);
    const bool win5 = qd.window == 5;
    const bool rate = (mode == MODE_BWD) && qd.level_prob != nullptr && qd.rate_c != 0.0f;
    switch (mode) {
        case MODE_HARD:
            return launch_t<MODE_HARD, false, false>(qd, x, nullptr, n, head, n4, nullptr, ib, hist, nullptr, nullptr, nullptr, stream);
        case MODE_SOFT:
            return win5 ? launch_t<MODE_SOFT, true, false>(qd, x, nullptr, n, head, n4, y, ib, hist, nullptr, nullptr, nullptr, stream)
                        : launch_t<MODE_SOFT, false, false>(qd, x, nullptr, n, head, n4, y, ib, hist, nullptr, nullptr, nullptr, stream);
        case MODE_BWD:
            if (win5)
                return rate ? launch_t<MODE_BWD, true, true>(qd, x, grad_out, n, head, n4, nullptr, nullptr, nullptr, grad_x, grad_q, grad_alpha, stream)
                            : launch_t<MODE_BWD, true, false>(qd, x, grad_out, n, head, n4, nullptr, nullptr, nullptr, grad_x, grad_q, grad_alpha, stream);
            return rate ? launch_t<MODE_BWD, false, true>(qd, x, grad_out, n, head, n4, nullptr, nullptr, nullptr, grad_x, grad_q, grad_alpha, stream)
                        : launch_t<MODE_BWD, false, false>(qd, x, grad_out, n, head, n4, nullptr, nullptr, nullptr, grad_x, grad_q, grad_alpha, stream);
        default:
            return CDL_ERR_ARG;
    }
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
