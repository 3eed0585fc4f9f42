// extern "C" entry points of libcdl.so: argument validation and launch plumbing.  See include/cdl.h
// for the contract of every call.
#include <math.h>
#include <string.h>

#include "cdl_internal.h"

namespace cdl {

namespace {
constexpr int kMaxDevices = 64;
int g_dev_ok[kMaxDevices];    // 0 unknown, 1 supported, -1 unsupported (cached device properties only)
int g_dev_sms[kMaxDevices];
}  // namespace

int check_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    if (dev < 0 || dev >= kMaxDevices) return CDL_ERR_UNSUPPORTED;
    if (g_dev_ok[dev] == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
        g_dev_sms[dev] = sms;
        g_dev_ok[dev] = (major == 10) ? 1 : -1;
    }
    return g_dev_ok[dev] == 1 ? CDL_OK : CDL_ERR_UNSUPPORTED;
}

int read_status_block(void *block, cudaStream_t st)
{
    int32_t words[3] = {0, 0, 0};
    if (cudaMemcpyAsync(words, block, sizeof words, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    // kernels write nothing but a complete record into the block; anything else (a fresh allocation) is "no record"
    if (words[0] != CDL_ERR_TIMEOUT || (unsigned int)words[1] != kStatusTag1 || (unsigned int)words[2] != kStatusTag2)
        return CDL_OK;
    if (cudaMemsetAsync(block, 0, sizeof words, st) != cudaSuccess) (void)cudaGetLastError();
    return CDL_ERR_TIMEOUT;
}

int sm_count()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    return g_dev_sms[dev];
}

int make_quant_dev(const cdl_quant_params *p, bool need_alpha, QuantDev *out)
{
    if (p == nullptr) return CDL_ERR_ARG;
    if (p->flags & ~CDL_HIST_ACCUMULATE) return CDL_ERR_ARG;
    if (!(p->q > 0.0f) || !isfinite(p->q)) return CDL_ERR_RANGE;
    if (p->hi < p->lo) return CDL_ERR_RANGE;
    const int64_t nlev = (int64_t)p->hi - (int64_t)p->lo + 1;
    if (nlev > CDL_MAX_LEVELS) return CDL_ERR_RANGE;
    if (p->lo < 0) {
        if (p->lo < -128 || p->hi > 127) return CDL_ERR_RANGE;
    } else if (p->hi > 255) {
        return CDL_ERR_RANGE;
    }
    QuantDev d;
    memset(&d, 0, sizeof d);
    d.q = p->q;
    d.half_q = 0.5f * p->q;
    d.rq = (float)(1.0 / (double)p->q);
    d.fast_div = (p->q > 1e-30f && p->q < 1e30f) ? 1 : 0;
    d.lo = p->lo;
    d.hi = p->hi;
    d.nlev = (int)nlev;
    d.flo = (float)p->lo;
    d.fhi = (float)p->hi;
    if (need_alpha) {
        if (!(p->alpha > 0.0f) || !isfinite(p->alpha)) return CDL_ERR_RANGE;
        if (!(p->rate_weight >= 0.0f) || !isfinite(p->rate_weight)) return CDL_ERR_RANGE;
        if (p->window < 0) return CDL_ERR_ARG;
        if (p->window > 0 && (p->window & 1) == 0) return CDL_ERR_ARG;
        const double q = (double)p->q, al = (double)p->alpha;
        const double a = al * q * q;
        d.c1 = (float)(al * q * 1.4426950408889634074);
        d.A = (float)(a * 1.4426950408889634074);
        d.c1x2 = (float)(2.0 * al * q * 1.4426950408889634074);
        d.near3 = a > 12.0 ? 1 : 0;
        d.res1 = a <= 64.0 ? 1 : 0;
        d.a2 = (float)(2.0 * a);
        d.two_aq = (float)(2.0 * al * q);
        d.q2 = (float)(q * q);
        d.rate_c = (float)((double)p->rate_weight * (-2.0 * al * q));
        if (!isfinite(d.c1) || !isfinite(d.c1x2) || !isfinite(d.A) || !isfinite(d.a2) || !isfinite(d.two_aq) || !isfinite(d.rate_c) || !(d.q2 > 0.0f))
            return CDL_ERR_RANGE;
        d.window = (p->window >= (int)nlev) ? 0 : p->window;
        // e_j <= 2^(-a log2e j (j - 1)) for the levels j steps beyond the nearest one: below 2^-40 past jmax
        double jm = ceil(0.5 + sqrt(0.25 + 40.0 * 0.69314718055994530942 / a)) + 1.0;
        if (!(jm < 256.0)) jm = 256.0;
        d.jmax = (int)jm;
        d.level_prob = p->level_prob;
    }
    *out = d;
    return CDL_OK;
}

namespace {

inline bool bad_f32_ptr(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3u) != 0; }

struct IndexRange {
    bool is_unsigned;
    int64_t absmax;
};

int index_range(const cdl_index_desc *d, IndexRange *r)
{
    if (d == nullptr) return CDL_ERR_ARG;
    if (!(d->q > 0.0f) || !isfinite(d->q)) return CDL_ERR_RANGE;
    if (d->hi < d->lo) return CDL_ERR_RANGE;
    if (d->lo < 0) {
        if (d->lo < -128 || d->hi > 127) return CDL_ERR_RANGE;
    } else if (d->hi > 255) {
        return CDL_ERR_RANGE;
    }
    r->is_unsigned = d->lo >= 0;
    const int64_t a = d->lo < 0 ? -(int64_t)d->lo : (int64_t)d->lo;
    const int64_t b = d->hi < 0 ? -(int64_t)d->hi : (int64_t)d->hi;
    r->absmax = a > b ? a : b;
    return CDL_OK;
}

inline bool overflow_risk(int64_t terms, const IndexRange &x, const IndexRange &y)
{
    return terms * x.absmax * y.absmax >= (int64_t)1 << 31;
}

constexpr size_t kStatusBytes = 256;

// float output of accumulators that were summed outside a product call (across ranks): one conversion, one multiply
template <typename T>
__global__ void __launch_bounds__(256) rescale_acc_kernel(const T *__restrict__ acc, long long n, float scale, float *__restrict__ out)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float v = sizeof(T) == 8 ? __ll2float_rn((long long)acc[i]) : (float)(int)acc[i];
        out[i] = __fmul_rn(v, scale);
    }
}

}  // namespace
}  // namespace cdl

using namespace cdl;

extern "C" {

int cdl_version(void) { return CDL_VERSION; }

const char *cdl_strerror(int status)
{
    switch (status) {
        case CDL_OK: return "ok";
        case CDL_ERR_ARG: return "invalid argument";
        case CDL_ERR_ALIGN: return "pointer or leading dimension not aligned as required";
        case CDL_ERR_RANGE: return "parameter out of range";
        case CDL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CDL_ERR_OVERFLOW_RISK: return "int32 accumulator could overflow for these sizes and index ranges";
        case CDL_ERR_LAUNCH: return "CUDA launch or runtime call failed";
        case CDL_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case CDL_ERR_UNSUPPORTED: return "device is not compute capability 10.x";
        case CDL_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

int cdl_quantize_hard(const float *x, int64_t n, const cdl_quant_params *p, void *idx_out, uint64_t *hist,
                      void *stream)
{
    if (n < 0 || (n > 0 && x == nullptr)) return CDL_ERR_ARG;
    if (bad_f32_ptr(x) || (reinterpret_cast<uintptr_t>(hist) & 7u)) return CDL_ERR_ALIGN;
    QuantDev qd;
    int rc = make_quant_dev(p, false, &qd);
    if (rc != CDL_OK) return rc;
    if ((rc = check_device()) != CDL_OK) return rc;
    return launch_quantize(MODE_HARD, x, nullptr, n, qd, nullptr, idx_out,
                           reinterpret_cast<unsigned long long *>(hist), (p->flags & CDL_HIST_ACCUMULATE) != 0,
                           nullptr, nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int cdl_quantize_soft(const float *x, int64_t n, const cdl_quant_params *p, float *y_soft, void *idx_out,
                      uint64_t *hist, uint64_t *soft_hist, void *stream)
{
    if (n < 0 || (n > 0 && (x == nullptr || y_soft == nullptr))) return CDL_ERR_ARG;
    if (bad_f32_ptr(x) || bad_f32_ptr(y_soft) || (reinterpret_cast<uintptr_t>(hist) & 7u) ||
        (reinterpret_cast<uintptr_t>(soft_hist) & 7u))
        return CDL_ERR_ALIGN;
    QuantDev qd;
    int rc = make_quant_dev(p, true, &qd);
    if (rc != CDL_OK) return rc;
    if ((rc = check_device()) != CDL_OK) return rc;
    return launch_quantize(MODE_SOFT, x, nullptr, n, qd, y_soft, idx_out,
                           reinterpret_cast<unsigned long long *>(hist), (p->flags & CDL_HIST_ACCUMULATE) != 0,
                           nullptr, nullptr, nullptr, reinterpret_cast<unsigned long long *>(soft_hist),
                           static_cast<cudaStream_t>(stream));
}

int cdl_quantize_sample(const float *x, int64_t n, const cdl_quant_params *p, uint64_t seed, uint64_t first_index,
                        void *idx_out, float *y_out, uint64_t *hist, void *stream)
{
    if (n < 0 || (n > 0 && x == nullptr)) return CDL_ERR_ARG;
    if (bad_f32_ptr(x) || bad_f32_ptr(y_out) || (reinterpret_cast<uintptr_t>(hist) & 7u)) return CDL_ERR_ALIGN;
    QuantDev qd;
    int rc = make_quant_dev(p, true, &qd);
    if (rc != CDL_OK) return rc;
    qd.seed = seed;
    qd.first_index = first_index;
    if ((rc = check_device()) != CDL_OK) return rc;
    return launch_quantize(MODE_SAMPLE, x, nullptr, n, qd, y_out, idx_out,
                           reinterpret_cast<unsigned long long *>(hist), (p->flags & CDL_HIST_ACCUMULATE) != 0,
                           nullptr, nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int cdl_quantize_backward(const float *x, const float *grad_out, int64_t n, const cdl_quant_params *p,
                          float *grad_x, double *grad_q, double *grad_alpha, void *stream)
{
    if (n < 0 || (n > 0 && (x == nullptr || grad_out == nullptr))) return CDL_ERR_ARG;
    if (bad_f32_ptr(x) || bad_f32_ptr(grad_out) || bad_f32_ptr(grad_x)) return CDL_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(grad_q) & 7u) || (reinterpret_cast<uintptr_t>(grad_alpha) & 7u)) return CDL_ERR_ALIGN;
    QuantDev qd;
    int rc = make_quant_dev(p, true, &qd);
    if (rc != CDL_OK) return rc;
    if (bad_f32_ptr(qd.level_prob)) return CDL_ERR_ALIGN;
    if ((rc = check_device()) != CDL_OK) return rc;
    return launch_quantize(MODE_BWD, x, grad_out, n, qd, nullptr, nullptr, nullptr, false, grad_x, grad_q,
                           grad_alpha, nullptr, static_cast<cudaStream_t>(stream));
}

int cdl_index_entropy(const uint64_t *hist, int32_t nlev, double *H_bits, float *level_prob, uint64_t *n_out,
                      void *stream)
{
    if (hist == nullptr || H_bits == nullptr) return CDL_ERR_ARG;
    if (nlev < 1 || nlev > CDL_MAX_LEVELS) return CDL_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(hist) & 7u) || (reinterpret_cast<uintptr_t>(H_bits) & 7u) ||
        (reinterpret_cast<uintptr_t>(n_out) & 7u) || bad_f32_ptr(level_prob))
        return CDL_ERR_ALIGN;
    int rc = check_device();
    if (rc != CDL_OK) return rc;
    return launch_entropy(reinterpret_cast<const unsigned long long *>(hist), nlev, H_bits, level_prob,
                          reinterpret_cast<unsigned long long *>(n_out), static_cast<cudaStream_t>(stream));
}

int cdl_huffman_lengths(const uint64_t *hist, int32_t nlev, uint8_t *lengths, uint64_t *total_bits, double *avg_bits,
                        void *stream)
{
    if (hist == nullptr || (lengths == nullptr && total_bits == nullptr && avg_bits == nullptr)) return CDL_ERR_ARG;
    if (nlev < 1 || nlev > CDL_MAX_LEVELS) return CDL_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(hist) & 7u) || (reinterpret_cast<uintptr_t>(total_bits) & 7u) ||
        (reinterpret_cast<uintptr_t>(avg_bits) & 7u))
        return CDL_ERR_ALIGN;
    int rc = check_device();
    if (rc != CDL_OK) return rc;
    return launch_huffman(reinterpret_cast<const unsigned long long *>(hist), nlev, lengths,
                          reinterpret_cast<unsigned long long *>(total_bits), avg_bits, static_cast<cudaStream_t>(stream));
}

size_t cdl_workspace_bytes(int32_t op, int32_t M, int32_t N, int32_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    switch (op) {
        case CDL_OP_QLINEAR_FWD: return kStatusBytes + tc_gemm_scratch_bytes(M, N, K);
        case CDL_OP_QLINEAR_BWD: {
            const size_t dx = tc_gemm_scratch_bytes(M, K, N), dw = tc_gemm_scratch_bytes(K, N, M);
            size_t need = dx > dw ? dx : dw;
            const size_t skinny = skinny_dw_ok(M, N, K) ? skinny_dw_scratch_bytes(N, K) : 0;
            if (skinny > need) need = skinny;
            return kStatusBytes + need;
        }
        default: return 0;
    }
}

int cdl_workspace_status(void *ws, void *stream)
{
    if (ws == nullptr) return CDL_ERR_WORKSPACE;
    return read_status_block(ws, static_cast<cudaStream_t>(stream));
}

namespace {
// next layer's quantizer for the fused index output; CDL_OK with out->idx_out == nullptr when none is requested
int next_quant(const cdl_index_desc *next, void *idx_next, cdl::NextQuant *out)
{
    out->idx_out = nullptr;
    if (idx_next == nullptr) return CDL_OK;
    if (next == nullptr) return CDL_ERR_ARG;
    cdl::IndexRange r;
    int rc = cdl::index_range(next, &r);
    if (rc != CDL_OK) return rc;
    out->idx_out = idx_next;
    out->q = next->q;
    out->rq = (float)(1.0 / (double)next->q);
    out->flo = (float)next->lo;
    out->fhi = (float)next->hi;
    out->fast_div = (next->q > 1e-30f && next->q < 1e30f) ? 1 : 0;
    return CDL_OK;
}
}  // namespace

int cdl_qlinear_fwd_next(const void *A_idx, int64_t lda, const cdl_index_desc *a, const void *W_idx, int64_t ldw,
                         const cdl_index_desc *w, int32_t M, int32_t N, int32_t K, int32_t *acc_out, float *y_out,
                         const float *bias, const cdl_index_desc *next, void *idx_next, void *ws, size_t ws_bytes,
                         void *stream)
{
    if (A_idx == nullptr || W_idx == nullptr || M <= 0 || N <= 0 || K <= 0) return CDL_ERR_ARG;
    if (acc_out == nullptr && y_out == nullptr && idx_next == nullptr) return CDL_ERR_ARG;
    NextQuant nq;
    {
        const int rcn = next_quant(next, idx_next, &nq);
        if (rcn != CDL_OK) return rcn;
    }
    if (lda < K || ldw < N) return CDL_ERR_ARG;
    IndexRange ra, rw;
    int rc;
    if ((rc = index_range(a, &ra)) != CDL_OK) return rc;
    if ((rc = index_range(w, &rw)) != CDL_OK) return rc;
    if (rw.is_unsigned && w->hi > 127) return CDL_ERR_RANGE;
    if ((lda & 15) || (ldw & 15) || (reinterpret_cast<uintptr_t>(A_idx) & 15u) || (reinterpret_cast<uintptr_t>(W_idx) & 15u))
        return CDL_ERR_ALIGN;
    if (bad_f32_ptr(acc_out) || bad_f32_ptr(y_out) || bad_f32_ptr(bias)) return CDL_ERR_ALIGN;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_workspace_bytes(CDL_OP_QLINEAR_FWD, M, N, K))
        return CDL_ERR_WORKSPACE;
    if (acc_out != nullptr && overflow_risk(K, ra, rw)) return CDL_ERR_OVERFLOW_RISK;
    if ((rc = check_device()) != CDL_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float scale = (a->q * w->q);
    // few output channels: an HBM-bound streaming product, served by the dp4a kernels
    if (nq.idx_out == nullptr && skinny_fwd_ok(M, N, K) && !overflow_risk(K, ra, rw) &&
        (reinterpret_cast<uintptr_t>(acc_out) & 15u) == 0 && (reinterpret_cast<uintptr_t>(y_out) & 15u) == 0)
        return launch_skinny_fwd(A_idx, lda, ra.is_unsigned, W_idx, ldw, M, N, K, acc_out, y_out, scale, bias, st);
    GemmOperand X{A_idx, lda, 1, ra.is_unsigned, (int)ra.absmax};
    GemmOperand Y{W_idx, 1, ldw, false, (int)rw.absmax};
    return launch_index_gemm_tc(X, Y, M, N, K, acc_out, y_out, scale, bias, static_cast<char *>(ws) + kStatusBytes,
                                static_cast<int *>(ws), st, nullptr, &nq);
}

int cdl_qlinear_fwd(const void *A_idx, int64_t lda, const cdl_index_desc *a, const void *W_idx, int64_t ldw,
                    const cdl_index_desc *w, int32_t M, int32_t N, int32_t K, int32_t *acc_out, float *y_out,
                    const float *bias, void *ws, size_t ws_bytes, void *stream)
{
    return cdl_qlinear_fwd_next(A_idx, lda, a, W_idx, ldw, w, M, N, K, acc_out, y_out, bias, nullptr, nullptr, ws,
                                ws_bytes, stream);
}

int cdl_qlinear_bwd(const void *G_idx, int64_t ldg, const cdl_index_desc *g, const void *A_idx, int64_t lda,
                    const cdl_index_desc *a, const void *W_idx, int64_t ldw, const cdl_index_desc *w, int32_t M,
                    int32_t N, int32_t K, int32_t *dXacc, float *dX, int32_t *dWacc, float *dW, void *ws,
                    size_t ws_bytes, void *stream)
{
    const bool want_dx = dXacc != nullptr || dX != nullptr;
    const bool want_dw = dWacc != nullptr || dW != nullptr;
    if (G_idx == nullptr || M <= 0 || N <= 0 || K <= 0) return CDL_ERR_ARG;
    if (!want_dx && !want_dw) return CDL_ERR_ARG;
    if ((want_dx && W_idx == nullptr) || (want_dw && A_idx == nullptr)) return CDL_ERR_ARG;
    if (ldg < N || (want_dw && lda < K) || (want_dx && ldw < N)) return CDL_ERR_ARG;
    IndexRange rg, ra{false, 0}, rw{false, 0};
    int rc;
    if ((rc = index_range(g, &rg)) != CDL_OK) return rc;
    if (rg.is_unsigned && g->hi > 127) return CDL_ERR_RANGE;
    if (want_dw && (rc = index_range(a, &ra)) != CDL_OK) return rc;
    if (want_dx) {
        if ((rc = index_range(w, &rw)) != CDL_OK) return rc;
        if (rw.is_unsigned && w->hi > 127) return CDL_ERR_RANGE;
    }
    if ((ldg & 15) || (reinterpret_cast<uintptr_t>(G_idx) & 15u)) return CDL_ERR_ALIGN;
    if (want_dw && ((lda & 15) || (reinterpret_cast<uintptr_t>(A_idx) & 15u))) return CDL_ERR_ALIGN;
    if (want_dx && ((ldw & 15) || (reinterpret_cast<uintptr_t>(W_idx) & 15u))) return CDL_ERR_ALIGN;
    if (bad_f32_ptr(dXacc) || bad_f32_ptr(dX) || bad_f32_ptr(dWacc) || bad_f32_ptr(dW)) return CDL_ERR_ALIGN;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_workspace_bytes(CDL_OP_QLINEAR_BWD, M, N, K))
        return CDL_ERR_WORKSPACE;
    if (dXacc != nullptr && overflow_risk(N, rg, rw)) return CDL_ERR_OVERFLOW_RISK;
    if (dWacc != nullptr && overflow_risk(M, ra, rg)) return CDL_ERR_OVERFLOW_RISK;
    if ((rc = check_device()) != CDL_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (want_dx && skinny_dx_ok(M, N, K) && !overflow_risk(N, rg, rw)) {
        // few reduced channels: HBM-bound, streamed by the dp4a kernel
        rc = launch_skinny_dx(G_idx, ldg, W_idx, ldw, M, N, K, dXacc, dX, (g->q * w->q), false, st);
        if (rc != CDL_OK) return rc;
    } else if (want_dx) {
        // dX[m,k] = sum_n G[m,n] W[k,n]
        GemmOperand X{G_idx, ldg, 1, false, (int)rg.absmax};
        GemmOperand Y{W_idx, ldw, 1, false, (int)rw.absmax};
        rc = launch_index_gemm_tc(X, Y, M, K, N, dXacc, dX, (g->q * w->q), nullptr,
                                  static_cast<char *>(ws) + kStatusBytes, static_cast<int *>(ws), st);
        if (rc != CDL_OK) return rc;
    }
    if (want_dw && skinny_dw_ok(M, N, K) && !overflow_risk(M, ra, rg)) {
        rc = launch_skinny_dw(A_idx, lda, ra.is_unsigned, G_idx, ldg, M, N, K, dWacc, dW, (g->q * a->q), false,
                              static_cast<char *>(ws) + kStatusBytes, st);
        if (rc != CDL_OK) return rc;
    } else if (want_dw) {
        // dW[k,n] = sum_m A[m,k] G[m,n]
        GemmOperand X{A_idx, 1, lda, ra.is_unsigned, (int)ra.absmax};
        GemmOperand Y{G_idx, 1, ldg, false, (int)rg.absmax};
        rc = launch_index_gemm_tc(X, Y, K, N, M, dWacc, dW, (g->q * a->q), nullptr,
                                  static_cast<char *>(ws) + kStatusBytes, static_cast<int *>(ws), st);
        if (rc != CDL_OK) return rc;
    }
    return CDL_OK;
}

namespace {
// Geometry of a supported convolution shape: output grid, pixel counts, taps.
struct ConvGeo {
    int stride, pad_h, pad_w;
    int P, Q;               // output pixels per image column / row
    int64_t M_out, M_in;    // N * P * Q, N * H * W
    int taps;
};

// false when the shape is not supported
bool conv_geo(const cdl_conv_shape *s, int32_t C_out, ConvGeo *g)
{
    if (s == nullptr || s->N <= 0 || s->H <= 0 || s->W <= 0 || s->C <= 0 || C_out <= 0) return false;
    if (s->R <= 0 || s->S <= 0 || s->R > 7 || s->S > 7) return false;
    if ((s->C % 64) != 0 || (C_out % 64) != 0) return false;
    g->stride = s->stride == 0 ? 1 : s->stride;                   // 0 and a negative padding: the defaults
    g->pad_h = s->pad_h < 0 ? (s->R - 1) / 2 : s->pad_h;
    g->pad_w = s->pad_w < 0 ? (s->S - 1) / 2 : s->pad_w;
    if (g->stride < 1 || g->stride > 4 || g->pad_h >= s->R || g->pad_w >= s->S) return false;
    if (s->H + 2 * g->pad_h < s->R || s->W + 2 * g->pad_w < s->S) return false;
    g->P = (s->H + 2 * g->pad_h - s->R) / g->stride + 1;
    g->Q = (s->W + 2 * g->pad_w - s->S) / g->stride + 1;
    g->M_out = (int64_t)s->N * g->P * g->Q;
    g->M_in = (int64_t)s->N * s->H * s->W;
    g->taps = s->R * s->S;
    if (g->M_out > 0x7fffff00ll || g->M_in > 0x7fffff00ll || (int64_t)g->taps * (s->C + 64) > 0x7fffff00ll ||
        (int64_t)g->taps * (C_out + 64) > 0x7fffff00ll)
        return false;
    return true;
}

// the patch matrix of the layer's input: rows = output pixels, taps in filter order
cdl::ConvGather input_gather(const cdl_conv_shape *s, const ConvGeo &g, int transposed)
{
    cdl::ConvGather cg;
    memset(&cg, 0, sizeof cg);
    cg.N = s->N;
    cg.H = s->H;
    cg.W = s->W;
    cg.C = s->C;
    cg.P = g.P;
    cg.Q = g.Q;
    cg.lower_h = -g.pad_h;
    cg.lower_w = -g.pad_w;
    cg.stride = g.stride;
    cg.taps = g.taps;
    for (int t = 0; t < g.taps; ++t) {
        cg.oh[t] = (signed char)(t / s->S);
        cg.ow[t] = (signed char)(t % s->S);
    }
    cg.transposed = transposed;
    return cg;
}

// The patch matrix of the gradient tensor [N,P,Q,C_out] for the data gradient of the input pixels h = st i + a,
// w = st j + b (st = the layer's stride; st = 1: all pixels, a = b = 0): only the filter taps r = a + pad_h (mod st),
// s = b + pad_w (mod st) reach such a pixel, tap r from gradient row i + (a + pad_h - r) / st.  Returns the number of
// taps (0: these pixels receive nothing).
int gradient_gather(const cdl_conv_shape *s, const ConvGeo &g, int32_t C_out, int a, int b, cdl::ConvGather *out)
{
    cdl::ConvGather cg;
    memset(&cg, 0, sizeof cg);
    const int st = g.stride;
    int rs[8], dr[8], nr = 0, ss[8], ds[8], ns = 0;
    for (int r = 0; r < s->R; ++r)
        if ((a + g.pad_h - r) % st == 0) {
            rs[nr] = r;
            dr[nr++] = (a + g.pad_h - r) / st;
        }
    for (int c = 0; c < s->S; ++c)
        if ((b + g.pad_w - c) % st == 0) {
            ss[ns] = c;
            ds[ns++] = (b + g.pad_w - c) / st;
        }
    if (nr == 0 || ns == 0) return 0;
    int dmin_h = dr[0], dmin_w = ds[0];
    for (int i = 1; i < nr; ++i) dmin_h = dr[i] < dmin_h ? dr[i] : dmin_h;
    for (int i = 1; i < ns; ++i) dmin_w = ds[i] < dmin_w ? ds[i] : dmin_w;
    cg.N = s->N;
    cg.H = g.P;
    cg.W = g.Q;
    cg.C = C_out;
    cg.P = (s->H - a + st - 1) / st;          // pixels h = st i + a < H
    cg.Q = (s->W - b + st - 1) / st;
    cg.lower_h = dmin_h;
    cg.lower_w = dmin_w;
    cg.stride = 1;
    cg.taps = nr * ns;
    for (int i = 0; i < nr; ++i)
        for (int j = 0; j < ns; ++j) {
            const int t = i * ns + j;
            cg.oh[t] = (signed char)(dr[i] - dmin_h);
            cg.ow[t] = (signed char)(ds[j] - dmin_w);
            cg.ytap[t] = (unsigned char)(rs[i] * s->S + ss[j]);
        }
    cg.transposed = 0;
    cg.y_tap_rows = s->C;
    cg.y_rows = g.taps * s->C;
    if (st > 1) {
        cg.sc_on = 1;
        cg.sc_H = s->H;
        cg.sc_W = s->W;
        cg.sc_s = st;
        cg.sc_a = a;
        cg.sc_b = b;
    }
    *out = cg;
    return cg.taps;
}
}  // namespace

size_t cdl_qconv_workspace_bytes(const cdl_conv_shape *shape, int32_t C_out)
{
    ConvGeo g;
    if (!conv_geo(shape, C_out, &g)) return 0;
    // the tiling pads every tap to whole 128-channel blocks (except the transposed gather of 64-channel taps)
    const int cp = (shape->C + 127) / 128 * 128, cop = (C_out + 127) / 128 * 128;
    const size_t f = tc_gemm_scratch_bytes((int)g.M_out, C_out, g.taps * cp);
    const size_t dx = g.stride == 1 ? tc_gemm_scratch_bytes((int)g.M_in, shape->C, g.taps * cop) : 0;   // (strided: no split)
    const size_t dw = tc_gemm_scratch_bytes(g.taps * (shape->C == 64 ? 64 : cp), C_out, (int)g.M_out);     // (64-channel taps: no padding)
    size_t m = f > dx ? f : dx;
    if (dw > m) m = dw;
    return kStatusBytes + m;
}

int cdl_qconv_fwd_next(const void *X_idx, const cdl_index_desc *x, const void *W_idx, int64_t ldw,
                       const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out, int32_t *acc_out, float *y_out,
                       const float *bias, const cdl_index_desc *next, void *idx_next, void *ws, size_t ws_bytes,
                       void *stream)
{
    ConvGeo geo;
    if (X_idx == nullptr || W_idx == nullptr || !conv_geo(shape, C_out, &geo)) return CDL_ERR_ARG;
    if (acc_out == nullptr && y_out == nullptr && idx_next == nullptr) return CDL_ERR_ARG;
    NextQuant nq;
    {
        const int rcn = next_quant(next, idx_next, &nq);
        if (rcn != CDL_OK) return rcn;
    }
    if (ldw < C_out) return CDL_ERR_ARG;
    IndexRange rx, rw;
    int rc;
    if ((rc = index_range(x, &rx)) != CDL_OK) return rc;
    if ((rc = index_range(w, &rw)) != CDL_OK) return rc;
    if (rw.is_unsigned && w->hi > 127) return CDL_ERR_RANGE;
    if ((ldw & 15) || (reinterpret_cast<uintptr_t>(X_idx) & 15u) || (reinterpret_cast<uintptr_t>(W_idx) & 15u)) return CDL_ERR_ALIGN;
    if (bad_f32_ptr(acc_out) || bad_f32_ptr(y_out) || bad_f32_ptr(bias)) return CDL_ERR_ALIGN;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_qconv_workspace_bytes(shape, C_out))
        return CDL_ERR_WORKSPACE;
    const int K = geo.taps * shape->C;
    if (acc_out != nullptr && overflow_risk(K, rx, rw)) return CDL_ERR_OVERFLOW_RISK;
    if ((rc = check_device()) != CDL_OK) return rc;
    // Y[pixel, co] = sum_{tap, c} patch(pixel; tap, c) * W[tap * C + c, co]
    const ConvGather cg = input_gather(shape, geo, 0);
    GemmOperand X{X_idx, 0, 0, rx.is_unsigned, (int)rx.absmax};
    GemmOperand Y{W_idx, 1, ldw, false, (int)rw.absmax};
    return launch_index_gemm_tc(X, Y, (int)geo.M_out, C_out, K, acc_out, y_out, (x->q * w->q), bias,
                                static_cast<char *>(ws) + kStatusBytes, static_cast<int *>(ws),
                                static_cast<cudaStream_t>(stream), &cg, &nq);
}

int cdl_qconv_fwd(const void *X_idx, const cdl_index_desc *x, const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                  const cdl_conv_shape *shape, int32_t C_out, int32_t *acc_out, float *y_out, const float *bias,
                  void *ws, size_t ws_bytes, void *stream)
{
    return cdl_qconv_fwd_next(X_idx, x, W_idx, ldw, w, shape, C_out, acc_out, y_out, bias, nullptr, nullptr, ws, ws_bytes,
                              stream);
}

namespace {
// Argument checks of the backward convolution products (everything but the workspace): CDL_OK, or the status the
// entry point returns before anything is enqueued.
int check_qconv_bwd(const void *G_idx, const cdl_index_desc *g, const void *X_idx, const cdl_index_desc *x,
                    const void *W_idx, int64_t ldw, const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out,
                    const int32_t *dXacc, const float *dX, const int32_t *dWacc, const float *dW, ConvGeo *geo,
                    cdl::IndexRange *rg, cdl::IndexRange *rx, cdl::IndexRange *rw)
{
    using namespace cdl;
    const bool want_dx = dXacc != nullptr || dX != nullptr;
    const bool want_dw = dWacc != nullptr || dW != nullptr;
    if (G_idx == nullptr || !conv_geo(shape, C_out, geo)) return CDL_ERR_ARG;
    if (!want_dx && !want_dw) return CDL_ERR_ARG;
    if ((want_dx && W_idx == nullptr) || (want_dw && X_idx == nullptr)) return CDL_ERR_ARG;
    if (want_dx && ldw < C_out) return CDL_ERR_ARG;
    int rc;
    if ((rc = index_range(g, rg)) != CDL_OK) return rc;
    if (rg->is_unsigned && g->hi > 127) return CDL_ERR_RANGE;
    if (want_dw && (rc = index_range(x, rx)) != CDL_OK) return rc;
    if (want_dx) {
        if ((rc = index_range(w, rw)) != CDL_OK) return rc;
        if (rw->is_unsigned && w->hi > 127) return CDL_ERR_RANGE;
    }
    if (reinterpret_cast<uintptr_t>(G_idx) & 15u) return CDL_ERR_ALIGN;
    if (want_dw && (reinterpret_cast<uintptr_t>(X_idx) & 15u)) return CDL_ERR_ALIGN;
    if (want_dx && ((ldw & 15) || (reinterpret_cast<uintptr_t>(W_idx) & 15u))) return CDL_ERR_ALIGN;
    if (bad_f32_ptr(dXacc) || bad_f32_ptr(dX) || bad_f32_ptr(dWacc) || bad_f32_ptr(dW)) return CDL_ERR_ALIGN;
    if (dXacc != nullptr && overflow_risk((int64_t)geo->taps * C_out, *rg, *rw)) return CDL_ERR_OVERFLOW_RISK;
    if (dWacc != nullptr && overflow_risk(geo->M_out, *rx, *rg)) return CDL_ERR_OVERFLOW_RISK;
    return CDL_OK;
}

// The two backward products of a convolutional layer for one gradient index tensor (already validated arguments).
// accumulate: the float outputs are added to (second digit plane of a real-valued gradient).
int run_qconv_bwd(const void *G_idx, float q_g, const cdl::IndexRange &rg, const void *X_idx, const cdl_index_desc *x,
                  const cdl::IndexRange &rx, const void *W_idx, int64_t ldw, const cdl_index_desc *w, const cdl::IndexRange &rw,
                  const cdl_conv_shape *shape, const ConvGeo &geo, int32_t C_out, int32_t *dXacc, float *dX, int32_t *dWacc,
                  float *dW, bool accumulate, void *ws, cudaStream_t st)
{
    using namespace cdl;
    char *scratch = static_cast<char *>(ws) + kStatusBytes;
    int *status = static_cast<int *>(ws);
    int rc;
    if (dXacc != nullptr || dX != nullptr) {
        // dX[pixel, c] = sum over the filter taps that reach the pixel and over co of G[..] * W[tap * C + c, co]: the
        // patches of the gradient tensor against the filter taps.  With a stride st > 1 the input pixels fall into
        // st x st residue classes (h mod st, w mod st), each reached by its own subset of taps: one product per class,
        // its rows written to the pixels of the class; a class no tap reaches receives zeros.
        GemmOperand X{G_idx, 0, 0, false, (int)rg.absmax};
        GemmOperand Y{W_idx, ldw, 1, false, (int)rw.absmax};
        const int st_ = geo.stride;
        bool cleared = false;
        for (int a = 0; a < st_; ++a)
            for (int b = 0; b < st_; ++b) {
                ConvGather cg;
                const int ntaps = gradient_gather(shape, geo, C_out, a, b, &cg);
                if (ntaps == 0) {
                    if (!cleared && !accumulate) {       // (cleared before any class is written: the stream keeps the order)
                        const size_t n = (size_t)geo.M_in * shape->C;
                        if ((dX != nullptr && cudaMemsetAsync(dX, 0, n * sizeof(float), st) != cudaSuccess) ||
                            (dXacc != nullptr && cudaMemsetAsync(dXacc, 0, n * sizeof(int32_t), st) != cudaSuccess)) {
                            (void)cudaGetLastError();
                            return CDL_ERR_LAUNCH;
                        }
                        cleared = true;
                    }
                    continue;
                }
                (void)ntaps;
            }
        for (int a = 0; a < st_; ++a)
            for (int b = 0; b < st_; ++b) {
                ConvGather cg;
                const int ntaps = gradient_gather(shape, geo, C_out, a, b, &cg);
                if (ntaps == 0 || cg.P <= 0 || cg.Q <= 0) continue;
                const long long rows = (long long)shape->N * cg.P * cg.Q;
                rc = launch_index_gemm_tc(X, Y, (int)rows, shape->C, ntaps * C_out, dXacc, dX, (q_g * w->q), nullptr, scratch,
                                          status, st, &cg, nullptr, accumulate);
                if (rc != CDL_OK) return rc;
            }
    }
    if (dWacc != nullptr || dW != nullptr) {
        // dW[tap * C + c, co] = sum_pixel patch(pixel; tap, c) * G[pixel, co]
        const ConvGather cg = input_gather(shape, geo, 1);
        GemmOperand X{X_idx, 0, 0, rx.is_unsigned, (int)rx.absmax};
        GemmOperand Y{G_idx, 1, C_out, false, (int)rg.absmax};
        rc = launch_index_gemm_tc(X, Y, geo.taps * shape->C, C_out, (int)geo.M_out, dWacc, dW, (q_g * x->q), nullptr, scratch,
                                  status, st, &cg, nullptr, accumulate);
        if (rc != CDL_OK) return rc;
    }
    return CDL_OK;
}
}  // namespace

int cdl_qconv_bwd(const void *G_idx, const cdl_index_desc *g, const void *X_idx, const cdl_index_desc *x,
                  const void *W_idx, int64_t ldw, const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out,
                  int32_t *dXacc, float *dX, int32_t *dWacc, float *dW, void *ws, size_t ws_bytes, void *stream)
{
    ConvGeo geo;
    IndexRange rg, rx{false, 0}, rw{false, 0};
    int rc = check_qconv_bwd(G_idx, g, X_idx, x, W_idx, ldw, w, shape, C_out, dXacc, dX, dWacc, dW, &geo, &rg, &rx, &rw);
    if (rc != CDL_OK) return rc;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_qconv_workspace_bytes(shape, C_out))
        return CDL_ERR_WORKSPACE;
    if ((rc = check_device()) != CDL_OK) return rc;
    return run_qconv_bwd(G_idx, g->q, rg, X_idx, x, rx, W_idx, ldw, w, rw, shape, geo, C_out, dXacc, dX, dWacc, dW, false, ws,
                         static_cast<cudaStream_t>(stream));
}

int cdl_rescale_acc(const void *acc, int32_t acc_bits, int64_t n, float q_x, float q_y, float *out, void *stream)
{
    const float scale = q_x * q_y;      // formed once in binary32, as in the products' epilogue
    if (n < 0 || (n > 0 && (acc == nullptr || out == nullptr))) return CDL_ERR_ARG;
    if (acc_bits != 32 && acc_bits != 64) return CDL_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(acc) & (uintptr_t)(acc_bits / 8 - 1)) || bad_f32_ptr(out)) return CDL_ERR_ALIGN;
    if (!(q_x > 0.0f) || !(q_y > 0.0f) || !isfinite(scale)) return CDL_ERR_RANGE;
    int rc = check_device();
    if (rc != CDL_OK) return rc;
    if (n == 0) return CDL_OK;
    const int sms = sm_count();
    long long blocks = (n + 255) / 256;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (acc_bits == 64) rescale_acc_kernel<long long><<<(unsigned int)blocks, 256, 0, st>>>(static_cast<const long long *>(acc), n, scale, out);
    else rescale_acc_kernel<int><<<(unsigned int)blocks, 256, 0, st>>>(static_cast<const int *>(acc), n, scale, out);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

namespace {
size_t align256(size_t v) { return (v + 255u) & ~(size_t)255u; }
int64_t ld16(int64_t n) { return (n + 15) / 16 * 16; }
}  // namespace

size_t cdl_qlinear_bwd_fp_workspace_bytes(int32_t M, int32_t N, int32_t K)
{
    const size_t base = cdl_workspace_bytes(CDL_OP_QLINEAR_BWD, M, N, K);
    if (base == 0) return 0;
    return align256(base) + 2 * align256((size_t)M * (size_t)ld16(N));
}

int cdl_qlinear_bwd_fp(const float *G, float g_absmax, const void *A_idx, int64_t lda, const cdl_index_desc *a,
                       const void *W_idx, int64_t ldw, const cdl_index_desc *w, int32_t M, int32_t N, int32_t K,
                       float *dX, float *dW, void *ws, size_t ws_bytes, void *stream)
{
    if (G == nullptr || M <= 0 || N <= 0 || K <= 0 || (dX == nullptr && dW == nullptr)) return CDL_ERR_ARG;
    if (!(g_absmax > 0.0f) || !(g_absmax < 1e30f)) return CDL_ERR_RANGE;
    if ((dX != nullptr && W_idx == nullptr) || (dW != nullptr && A_idx == nullptr)) return CDL_ERR_ARG;
    if (bad_f32_ptr(G)) return CDL_ERR_ALIGN;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_qlinear_bwd_fp_workspace_bytes(M, N, K))
        return CDL_ERR_WORKSPACE;
    // every argument is checked before the first operation is enqueued
    IndexRange rg{false, 127}, ra{false, 0}, rw{false, 0};
    int rc;
    if (dW != nullptr && (rc = index_range(a, &ra)) != CDL_OK) return rc;
    if (dX != nullptr) {
        if ((rc = index_range(w, &rw)) != CDL_OK) return rc;
        if (rw.is_unsigned && w->hi > 127) return CDL_ERR_RANGE;
        if (ldw < N) return CDL_ERR_ARG;
        if ((ldw & 15) || (reinterpret_cast<uintptr_t>(W_idx) & 15u)) return CDL_ERR_ALIGN;
    }
    if (dW != nullptr) {
        if (lda < K) return CDL_ERR_ARG;
        if ((lda & 15) || (reinterpret_cast<uintptr_t>(A_idx) & 15u)) return CDL_ERR_ALIGN;
    }
    if (bad_f32_ptr(dX) || bad_f32_ptr(dW)) return CDL_ERR_ALIGN;
    if ((rc = check_device()) != CDL_OK) return rc;
    const float q1 = g_absmax / 127.0f, q2 = q1 / 254.0f;
    const int64_t ldg = ld16(N);
    const size_t base = align256(cdl_workspace_bytes(CDL_OP_QLINEAR_BWD, M, N, K));
    const size_t plane = align256((size_t)M * (size_t)ldg);
    char *d1 = static_cast<char *>(ws) + base, *d2 = d1 + plane;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ldg != N) {      // the pad columns are operands of the TMA loads: keep them defined
        if (cudaMemsetAsync(d1, 0, 2 * plane, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }
    if ((rc = launch_gradient_digits(G, M, N, (int)ldg, q1, q2, d1, d2, st)) != CDL_OK) return rc;
    const cdl_index_desc g1{q1, -127, 127}, g2{q2, -127, 127};
    // first digit stores, second digit adds: dX = RN(RN(acc1 s1) + RN(acc2 s2))
    char *scratch = static_cast<char *>(ws) + kStatusBytes;
    for (int pass = 0; pass < 2; ++pass) {
        const char *dig = pass == 0 ? d1 : d2;
        const float qg = pass == 0 ? g1.q : g2.q;
        if (dX != nullptr) {
            GemmOperand X{dig, ldg, 1, false, (int)rg.absmax};
            GemmOperand Y{W_idx, ldw, 1, false, (int)rw.absmax};
            rc = launch_index_gemm_tc(X, Y, M, K, N, nullptr, dX, (qg * w->q), nullptr, scratch, static_cast<int *>(ws), st,
                                      nullptr, nullptr, pass == 1);
            if (rc != CDL_OK) return rc;
        }
        if (dW != nullptr) {
            GemmOperand X{A_idx, 1, lda, ra.is_unsigned, (int)ra.absmax};
            GemmOperand Y{dig, 1, ldg, false, (int)rg.absmax};
            rc = launch_index_gemm_tc(X, Y, K, N, M, nullptr, dW, (qg * a->q), nullptr, scratch, static_cast<int *>(ws), st,
                                      nullptr, nullptr, pass == 1);
            if (rc != CDL_OK) return rc;
        }
    }
    return CDL_OK;
}

size_t cdl_qconv_bwd_fp_workspace_bytes(const cdl_conv_shape *shape, int32_t C_out)
{
    const size_t base = cdl_qconv_workspace_bytes(shape, C_out);
    ConvGeo geo;
    if (base == 0 || !conv_geo(shape, C_out, &geo)) return 0;
    return align256(base) + 2 * align256((size_t)geo.M_out * (size_t)C_out);
}

int cdl_qconv_bwd_fp(const float *G, float g_absmax, const void *X_idx, const cdl_index_desc *x, const void *W_idx,
                     int64_t ldw, const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out, float *dX, float *dW,
                     void *ws, size_t ws_bytes, void *stream)
{
    ConvGeo geo;
    if (G == nullptr || !conv_geo(shape, C_out, &geo) || (dX == nullptr && dW == nullptr)) return CDL_ERR_ARG;
    if (!(g_absmax > 0.0f) || !(g_absmax < 1e30f)) return CDL_ERR_RANGE;
    if (bad_f32_ptr(G)) return CDL_ERR_ALIGN;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < cdl_qconv_bwd_fp_workspace_bytes(shape, C_out))
        return CDL_ERR_WORKSPACE;
    const float q1 = g_absmax / 127.0f, q2 = q1 / 254.0f;
    if (!(q1 > 0.0f) || !(q2 > 0.0f)) return CDL_ERR_RANGE;
    const size_t base = align256(cdl_qconv_workspace_bytes(shape, C_out));
    const size_t plane = align256((size_t)geo.M_out * (size_t)C_out);
    char *d1 = static_cast<char *>(ws) + base, *d2 = d1 + plane;
    // every argument is checked before the first operation is enqueued (the digit planes stand in for G_idx)
    const cdl_index_desc gd{q1, -127, 127};
    IndexRange rg, rx{false, 0}, rw{false, 0};
    int rc = check_qconv_bwd(d1, &gd, X_idx, x, W_idx, ldw, w, shape, C_out, nullptr, dX, nullptr, dW, &geo, &rg, &rx, &rw);
    if (rc != CDL_OK) return rc;
    if ((rc = check_device()) != CDL_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = launch_gradient_digits(G, geo.M_out, C_out, C_out, q1, q2, d1, d2, st)) != CDL_OK) return rc;
    // each digit plane is a gradient index tensor of its own step: the first pass stores, the second adds.  The
    // products share the front of the workspace (status block, split slabs); calls on one stream run in order.
    for (int pass = 0; pass < 2; ++pass) {
        rc = run_qconv_bwd(pass == 0 ? d1 : d2, pass == 0 ? q1 : q2, rg, X_idx, x, rx, W_idx, ldw, w, rw, shape, geo, C_out,
                           nullptr, dX, nullptr, dW, pass == 1, ws, st);
        if (rc != CDL_OK) return rc;
    }
    return CDL_OK;
}

}  // extern "C"
