// Internal declarations shared by the translation units of libcdl.so (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "cdl.h"

namespace cdl {

// Quantizer parameters in the form the kernels consume; derived on the host in double
// precision from (q, lo, hi, alpha, rate weight) and rounded once to binary32.
struct QuantDev {
    float q;          // step size
    float half_q;     // q / 2 (exact)
    float rq;         // RN(1/q)
    int fast_div;     // q and 1/q are normal numbers well inside the exponent range: x * rq may stand in for x / q
    float flo, fhi;   // index range as floats
    int lo, hi, nlev;
    float c1;         // alpha * q * log2(e): the logit of level kn+j relative to level kn is -c1 * j * (j q - 2 d)
    float A;          // alpha * q^2 * log2(e) = c1 * q
    float c1x2;       // 2 * c1
    int near3;        // alpha q^2 > 12: only the nearest level and its two neighbours carry weight (> 2^-34 relative)
    int res1;         // alpha q^2 <= 64: theta - k q from one fused multiply-add is accurate enough for the logits
    float a2;         // 2 alpha q^2: dQ_d/dtheta = a2 * Var{J}
    float two_aq;     // 2 alpha q
    float q2;         // q^2
    float rate_c;     // rate_weight * (-2 alpha q)
    int window;       // 0 = whole index set, else an odd window smaller than nlev
    int jmax;         // levels further than jmax from the nearest one carry < 2^-40 of its weight
    const float *level_prob;  // nullptr: no rate term
    unsigned long long seed;         // MODE_SAMPLE: generator key
    unsigned long long first_index;  // MODE_SAMPLE: counter-space index of element 0
};

enum QuantMode { MODE_HARD = 0, MODE_SOFT = 1, MODE_BWD = 2, MODE_SAMPLE = 3 };

// A status block (first 16 bytes of a workspace, or of the built-in scratch) holds a timeout record when its first
// word is CDL_ERR_TIMEOUT and the next two are these tags.
constexpr unsigned int kStatusTag1 = 0x43444C54u, kStatusTag2 = 0x6F757421u;
// Synchronises the stream, reads the block, clears a record if there is one; CDL_OK, CDL_ERR_TIMEOUT or CDL_ERR_LAUNCH.
int read_status_block(void *block, cudaStream_t stream);

int check_device();   // CDL_OK, CDL_ERR_UNSUPPORTED or CDL_ERR_LAUNCH
int sm_count();       // multiprocessors of the current device (0 on error)
int make_quant_dev(const cdl_quant_params *p, bool need_alpha, QuantDev *out);

int launch_quantize(int mode, const float *x, const float *grad_out, int64_t n, const QuantDev &qd,
                    float *y, void *idx, unsigned long long *hist, bool hist_accumulate,
                    float *grad_x, double *grad_q, double *grad_alpha, unsigned long long *soft_hist,
                    cudaStream_t stream);
int launch_entropy(const unsigned long long *hist, int nlev, double *H, float *prob,
                   unsigned long long *n_out, cudaStream_t stream);

// Operand of an index GEMM D[i,j] = sum_r X(i,r) * Y(r,j): index bytes with arbitrary strides.
struct GemmOperand {
    const void *ptr;
    int64_t stride_outer;   // stride of the non-reduced dimension (i for X, j for Y)
    int64_t stride_red;     // stride of the reduced dimension r
    bool is_unsigned;
    int absmax;             // bound on |entry| (from the operand's declared index range)
};

// Streaming dp4a kernels for products with few output channels (N in {4, 8, 16, 32}); see cdl_gemm_skinny.cu.
bool skinny_fwd_ok(int M, int N, int K);
bool skinny_dx_ok(int M, int N, int K);
bool skinny_dw_ok(int M, int N, int K);
size_t skinny_dw_scratch_bytes(int N, int K);
int launch_skinny_dw(const void *A, long long lda, bool a_unsigned, const void *G, long long ldg, int M, int N, int K,
                     int32_t *acc_out, float *f_out, float scale, bool accumulate, void *scratch, cudaStream_t stream);
int launch_skinny_fwd(const void *A, long long lda, bool a_unsigned, const void *W, long long ldw, int M, int N, int K,
                      int32_t *acc_out, float *y_out, float scale, const float *bias, cudaStream_t stream);
int launch_skinny_dx(const void *G, long long ldg, const void *W, long long ldw, int M, int N, int K, int32_t *acc_out,
                     float *f_out, float scale, bool accumulate, cudaStream_t stream);

int launch_gradient_digits(const float *g, long long rows, int cols, int ld, float q1, float q2, void *d1, void *d2,
                           cudaStream_t stream);
int launch_huffman(const unsigned long long *hist, int nlev, unsigned char *lengths, unsigned long long *total_bits,
                   double *avg_bits, cudaStream_t stream);

// The X operand as an implicit patch matrix of a convolution: X.ptr then is an [N,H,W,C] tensor of index bytes and
// the rows / columns of the patch matrix are gathered by TMA im2col loads, never stored.  The gather is described by
// a grid of P x Q base pixels per image - base pixel (p, q) sits at (lower_h + p * stride, lower_w + q * stride), which
// may lie outside the tensor (padding reads as zero) - and by `taps` filter taps, tap t reading the pixel at offset
// (oh[t], ow[t]) >= 0 from the base pixel.
constexpr int kConvMaxTaps = 64;
struct ConvGather {
    int N, H, W, C;         // the gathered tensor
    int P, Q;               // base pixels per image (rows of the patch matrix = N * P * Q)
    int lower_h, lower_w, stride;
    int taps;
    signed char oh[kConvMaxTaps], ow[kConvMaxTaps];
    int transposed;         // 0: X(i = pixel, r = tap * C + c);  1: X(i = tap * C + c, r = pixel)
    int y_tap_rows;         // > 0: Y is stored as [.. * y_tap_rows][C] (r contiguous) and the block of tap t starts at row
    unsigned char ytap[kConvMaxTaps];   //  ytap[t] * y_tap_rows  (backward-data products: the filter's own tap of gather tap t)
    int y_rows;             //  ... and y_rows rows in all
    // output rows scattered over a larger image (see TcParams): row (n, p, q) -> pixel (n, sc_s p + sc_a, sc_s q + sc_b)
    int sc_on, sc_H, sc_W, sc_s, sc_a, sc_b;
};

// Hard index of the next layer's quantizer, computed in the forward product's epilogue from the float output:
// idx = clamp(rint(y / q), lo, hi) with the arithmetic of the quantizer kernels (bit-identical to quantizing Y).
struct NextQuant {
    void *idx_out;      // I x J index bytes, row pitch J
    float q, rq;        // step and RN(1/q)
    float flo, fhi;     // index range as floats
    int fast_div;       // as QuantDev::fast_div
};

// Tensor-core index GEMM (TMA + tcgen05 + TMEM); operands need 16-byte aligned bases and pitches.
size_t tc_gemm_scratch_bytes(int I, int J, int R);
int launch_index_gemm_tc(const GemmOperand &X, const GemmOperand &Y, int I, int J, int R, int32_t *acc_out,
                         float *f_out, float scale, const float *bias, void *scratch, int *status,
                         cudaStream_t stream, const ConvGather *conv = nullptr, const NextQuant *next = nullptr,
                         bool accumulate_f = false,    // f_out += result instead of f_out = result
                         bool compact_scratch = false); // split runs add into one I x J buffer (scratch of I * J * 4 bytes)

}  // namespace cdl
