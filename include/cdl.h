/*
 * cdl.h - C ABI of the CDL quantized layer for NVIDIA B200 (sm_100a).
 *
 * Method: "Coded Deep Learning: Framework and Algorithm" (arXiv 2501.09849).
 * The library computes, on the GPU, the per-element probabilistic quantizer of
 * Sec. IV (CPMF, hard index, soft value Q_d, analytic partial derivatives of
 * Lemma 1), the per-tensor level histogram and its entropy (Sec. V-C), and the
 * forward / backward layer products over the integer indices (Sec. V-A,
 * Algorithm 1, forward pass and backward pass).
 *
 * Conventions common to every entry point
 *  - Pointers marked [dev] are device memory owned by the caller; [host] are
 *    host memory read during the call only.  The library allocates no device
 *    memory and never synchronises the device (cdl_workspace_status and
 *    cdl_noalloc_status excepted).  What it keeps between calls is per-device
 *    bookkeeping only (device properties, kernel attributes set once, the
 *    address and contents of the built-in scratch of
 *    cdl_qlinear_bwd_dw_noalloc): no result depends on earlier calls.
 *    Work is enqueued on `stream` (a
 *    cudaStream_t passed as void*; NULL is the legacy default stream) and
 *    outputs are valid once the stream reaches it.
 *  - All matrices are row-major; leading dimensions are in elements.
 *  - Return value: CDL_OK (0) or a negative cdl_status.  On an argument error
 *    nothing has been launched.  No call aborts, throws or traps.
 *  - Notation follows the paper: theta = a weight or an activation, q = step
 *    size (q_l for weights, s_l for activations), index set {lo..hi}
 *    (weights: -2^(b-1)..2^(b-1)-1, activations: 0..2^b-1, Sec. V-A; a
 *    symmetric set -L..L is lo=-L, hi=L), alpha = CPMF parameter (alpha_l for
 *    weights, beta_l for activations), rate weight = lambda or gamma (Sec. V-D).
 */
#ifndef CDL_H_
#define CDL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CDL_VERSION 100 /* 0.1.0 */
#define CDL_MAX_LEVELS 256

typedef enum cdl_status {
    CDL_OK = 0,
    CDL_ERR_ARG = -1,           /* NULL where a pointer is required, negative size, even window, bad flag */
    CDL_ERR_ALIGN = -2,         /* pointer or leading dimension not aligned as documented */
    CDL_ERR_RANGE = -3,         /* q <= 0, alpha <= 0, non-finite parameter, more than 256 levels,
                                   index set not representable in the index byte */
    CDL_ERR_WORKSPACE = -4,     /* workspace NULL, misaligned or smaller than cdl_workspace_bytes() */
    CDL_ERR_OVERFLOW_RISK = -5, /* an int32 accumulator could overflow for these sizes and index ranges */
    CDL_ERR_LAUNCH = -6,        /* the CUDA runtime refused a launch or a driver call */
    CDL_ERR_TIMEOUT = -7,       /* a bounded device-side wait expired (reported by cdl_workspace_status) */
    CDL_ERR_UNSUPPORTED = -8,   /* the current device is not compute capability 10.x */
    CDL_ERR_TOO_LARGE = -9      /* problem exceeds the built-in scratch of cdl_qlinear_bwd_dw_noalloc */
} cdl_status;

/* Flags of cdl_quant_params.flags */
#define CDL_HIST_ACCUMULATE 0x1u /* add to the histogram instead of clearing it first */

/*
 * One trainable quantizer (Sec. IV-A, Sec. V-A): step size, index set, CPMF parameter.
 *   q           step size, finite, > 0.
 *   lo, hi      index set {lo..hi}, 1 <= hi-lo+1 <= 256.  Index bytes are int8 when lo < 0
 *               (requires -128 <= lo, hi <= 127) and uint8 otherwise (requires hi <= 255).
 *   alpha       CPMF parameter of Eq. (4), finite, > 0.
 *   rate_weight lambda (weights) or gamma (activations) of the objective of Sec. V-D, finite, >= 0.
 *               Only cdl_quantize_backward reads it.
 *   level_prob  [dev] nlev floats, the level probabilities the rate term differentiates through
 *               (normally written by cdl_index_entropy), or NULL for "no rate term".  The paper's CPMF
 *               has no rate term in its logits: the rate acts through the gradient only.
 *   window      0 = the CPMF over the whole index set (the definition).  An odd k > 0 keeps the k most
 *               probable levels, i.e. the k in-range levels nearest theta, and renormalises
 *               (Sec. VI-B.1 uses 5 for activations); of two equally distant levels the lower one is
 *               kept.  k >= nlev is the same as 0.
 */
typedef struct cdl_quant_params {
    float q;
    int32_t lo, hi;
    float alpha;
    float rate_weight;
    const float *level_prob;
    int32_t window;
    uint32_t flags;
} cdl_quant_params;

/* An index tensor as a GEMM operand: its step size and the range its entries lie in
 * (bytes are int8 when lo < 0, uint8 otherwise).  The range only serves the overflow check. */
typedef struct cdl_index_desc {
    float q;
    int32_t lo, hi;
} cdl_index_desc;

/*
 * Hard index = uniform quantizer Q_u, the limit of Q_p and Q_d for large alpha (Remark of
 * Sec. IV-A; end of Sec. IV-B), with the per-tensor level histogram fused in (the empirical
 * distribution over levels whose entropy Sec. V-C constrains).
 *   idx = clamp(round_half_even(x / q), lo, hi), quotient in IEEE binary32; a NaN input gives lo.
 *   x        [dev] n floats (4-byte aligned; 16-byte alignment takes the vector path).
 *   p        [host].
 *   idx_out  [dev] n bytes (int8 or uint8, see cdl_quant_params), nullable.
 *   hist     [dev] nlev uint64 counters, nullable; cleared first unless CDL_HIST_ACCUMULATE.
 * n = 0 is valid (clears hist).  p->alpha, rate_weight, level_prob and window are not read.
 */
int cdl_quantize_hard(const float *x, int64_t n, const cdl_quant_params *p,
                      void *idx_out, uint64_t *hist, void *stream);

/*
 * Soft deterministic quantizer Q_d(x) = sum_i P_alpha(iq | x) iq of Sec. IV-B, Eq. (8), with the
 * CPMF of Eq. (4) (optionally truncated to p->window levels), and, in the same pass over x,
 * optionally the hard index and the histogram exactly as cdl_quantize_hard writes them, and the soft
 * histogram of Sec. V-C, Eq. (25): the marginal PMF of the randomly quantized tensor is
 * (1/n) sum_i P_alpha(. | x[i]), whose entropy is the bits-per-entry the objective constrains.
 *   y_soft    [dev] n floats, required.   idx_out, hist: nullable.
 *   soft_hist [dev] nlev uint64, nullable: sum_i P_alpha(kq | x[i]) per level k in fixed point, units of 2^-32
 *             (integer sums: exact and independent of the order of accumulation).  Cleared first unless
 *             CDL_HIST_ACCUMULATE.  cdl_index_entropy accepts it in place of a count histogram (it only uses
 *             ratios): H_bits is then the entropy of the marginal PMF and level_prob that PMF.
 * x must be finite for y_soft to be meaningful (NaN and infinities give NaN).
 */
int cdl_quantize_soft(const float *x, int64_t n, const cdl_quant_params *p,
                      float *y_soft, void *idx_out, uint64_t *hist, uint64_t *soft_hist, void *stream);

/*
 * Probabilistic quantizer Q_p of Sec. IV-A, Eq. (7) - what CDL's forward pass applies to weights and activations
 * (Algorithm 1): element i is mapped to level k with probability P_alpha(kq | x[i]) (CPMF of Eq. (4), optionally
 * truncated to p->window levels).  Sampling is by inversion in increasing level order: with u_i in [0,1) the
 * element's uniform number, the index is the first level whose cumulative probability exceeds u_i.  u_i is the
 * top 24 bits, times 2^-24, of word (e mod 4) of the Philox4x32-10 block with counter (e div 4, 0) and key `seed`,
 * where e = first_index + i: the draw depends only on (seed, e), so any partition of a tensor into calls or
 * ranks (each passing its own first_index) reproduces the same sample.  The cumulative sums are binary32; next to
 * a cumulative-probability boundary (within ~1e-6) the neighbouring level may be chosen.
 *   idx_out [dev] n index bytes, nullable;  y_out [dev] n floats idx * q, nullable;  hist: as cdl_quantize_hard.
 */
int cdl_quantize_sample(const float *x, int64_t n, const cdl_quant_params *p, uint64_t seed,
                        uint64_t first_index, void *idx_out, float *y_out, uint64_t *hist, void *stream);

/*
 * Backward of the quantizer with Q_d as the gradient proxy (Sec. V-B, Eqs. (18), (20)-(24)):
 *   grad_x[i]  = grad_out[i] * dQ_d/dtheta(x[i])                     Lemma 1, Eq. (9a): 2 alpha Var
 *                + rate_weight * d(n H)/dtheta_i                      (only if level_prob != NULL)
 *   grad_q     = sum_i grad_out[i] * dQ_d/dq(x[i])                   Lemma 1, Eq. (9b)
 *   grad_alpha = sum_i grad_out[i] * dQ_d/dalpha(x[i])               = 2 theta Var - Skew_u (derived
 *                                                                      with the steps of Appendix B)
 * The rate term is the derivative of the total bits n*H of Sec. V-C w.r.t. theta_i with the level
 * probabilities pbar held as passed in:  -2 alpha sum_k P_k log2(pbar_k) (k q - Q_d(theta_i));
 * log2 of a probability below 2^-30 counts as -30.  The CPMF is recomputed from x; nothing is
 * kept from the forward pass.
 *   grad_out [dev] n floats: dL/dQ_p(x), the gradient arriving at the quantized tensor.
 *   grad_x   [dev] n floats, nullable.
 *   grad_q, grad_alpha [dev] one double each, nullable, overwritten (not accumulated).  Partial sums
 *            are combined with floating-point atomics: the last bits can differ from run to run.
 */
int cdl_quantize_backward(const float *x, const float *grad_out, int64_t n,
                          const cdl_quant_params *p, float *grad_x,
                          double *grad_q, double *grad_alpha, void *stream);

/*
 * Entropy in bits of the level distribution given by a histogram (Sec. III-A definition of H,
 * base 2; Sec. V-C: bits per weight / activation), and the level probabilities themselves.
 *   hist        [dev] nlev uint64 counters.
 *   H_bits      [dev] one double: -sum_k p_k log2 p_k, p_k = hist[k]/n, 0 log 0 = 0; 0 when n = 0.
 *   level_prob  [dev] nlev floats p_k, nullable.      n_out [dev] one uint64 (= sum of hist), nullable.
 */
int cdl_index_entropy(const uint64_t *hist, int32_t nlev, double *H_bits,
                      float *level_prob, uint64_t *n_out, void *stream);

/*
 * Huffman code lengths for the levels of a tensor, from its histogram (Sec. VI-B: the average numbers of bits per
 * weight and per activation that the paper reports are those of a Huffman code of the quantized tensor).
 *   hist       [dev] nlev uint64 counters (a count histogram of cdl_quantize_hard / _soft / _sample).
 *   lengths    [dev] nlev bytes, nullable: code length of each level; 0 for a level that does not occur; when only one
 *              level occurs its length is 1 (a reading: the paper does not treat the one-symbol case).
 *   total_bits [dev] one uint64, nullable: sum_k hist[k] * lengths[k], the size of the coded tensor without the table.
 *   avg_bits   [dev] one double, nullable: total_bits / n, 0 when the histogram is empty.
 * The individual lengths depend on how equal weights are paired (any optimal prefix code is a valid answer); the
 * total does not.  At least one output is required.
 */
int cdl_huffman_lengths(const uint64_t *hist, int32_t nlev, uint8_t *lengths, uint64_t *total_bits, double *avg_bits,
                        void *stream);

/*
 * Forward layer product over the indices (Sec. V-A; Algorithm 1, forward pass) with the
 * q_a * q_w rescale in the epilogue:
 *   ACC[m,n] = sum_k A_idx[m,k] * W_idx[k,n]   (int32, exact)
 *   Y[m,n]   = (float)ACC[m,n] * (a->q * w->q) + bias[n]   (a->q * w->q formed once in binary32;
 *              multiply and add each rounded to binary32)
 *   A_idx [dev] M x K bytes, leading dimension lda;  W_idx [dev] K x N int8, leading dimension ldw.
 *   lda, ldw multiples of 16; A_idx, W_idx 16-byte aligned (TMA requirements).
 *   acc_out [dev] M x N int32 (ld N), nullable.  y_out [dev] M x N floats (ld N), nullable.
 *   bias [dev] N floats, nullable.  At least one of acc_out, y_out.
 *   ws [dev]: cdl_workspace_bytes(CDL_OP_QLINEAR_FWD, M, N, K) bytes, 256-byte aligned.
 * CDL_ERR_OVERFLOW_RISK when acc_out is requested and K * max|a| * max|w| >= 2^31 for the declared index ranges
 * (the float output alone is always available: long reductions are then cut into exact int32 parts that are
 * summed in int64 before the single conversion to float).
 */
int cdl_qlinear_fwd(const void *A_idx, int64_t lda, const cdl_index_desc *a,
                    const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                    int32_t M, int32_t N, int32_t K,
                    int32_t *acc_out, float *y_out, const float *bias,
                    void *ws, size_t ws_bytes, void *stream);

/*
 * Forward products that also emit the hard index of the NEXT layer's activation quantizer (Sec. IV-A Remark /
 * end of Sec. IV-B: Q_u; Algorithm 1 feeds each layer's output to the next layer's quantizer), taken in the
 * epilogue from the finished float output, so that a forward-only (inference) pass never writes or re-reads the
 * fp32 activations:
 *   idx_next[m,n] = clamp(rint(Y[m,n] / next->q), next->lo, next->hi)        -- the bytes cdl_quantize_hard(Y) writes
 *   next     index set and step of the next layer's quantizer (with lo = 0 the clamp doubles as the ReLU).
 *   idx_next [dev] M x N (resp. N x H x W x C_out) index bytes, row pitch N (C_out); nullable = plain forward.
 *   acc_out, y_out may then both be NULL.  Everything else as cdl_qlinear_fwd / cdl_qconv_fwd.
 * The reduced dimension is not split across CTAs for these calls; CDL_ERR_OVERFLOW_RISK when it is so long that
 * its int32 sum could overflow for the declared index ranges.
 */
int cdl_qlinear_fwd_next(const void *A_idx, int64_t lda, const cdl_index_desc *a,
                         const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                         int32_t M, int32_t N, int32_t K,
                         int32_t *acc_out, float *y_out, const float *bias,
                         const cdl_index_desc *next, void *idx_next,
                         void *ws, size_t ws_bytes, void *stream);

/*
 * Backward layer products over the indices (Algorithm 1, backward pass over the quantized weights
 * and activations).  The gradient operand is an index tensor as well: the caller quantizes
 * dL/dY with cdl_quantize_hard (for example lo=-127, hi=127 and a step g->q of its choice) - a
 * reading of the paper, which does not say how the arriving gradient is represented.
 *   dXACC[m,k] = sum_n G_idx[m,n] * W_idx[k,n]     dX[m,k] = (float)dXACC * (g->q * w->q)
 *   dWACC[k,n] = sum_m A_idx[m,k] * G_idx[m,n]     dW[k,n] = (float)dWACC * (g->q * a->q)
 *   G_idx [dev] M x N int8 (ld ldg);  A_idx M x K (ld lda);  W_idx K x N (ld ldw); all ld % 16 == 0,
 *   all base pointers 16-byte aligned.
 *   dXacc, dWacc [dev] int32 (ld K, ld N), dX, dW [dev] floats; each nullable.  A_idx may be NULL
 *   when neither dWacc nor dW is wanted, W_idx when neither dXacc nor dX is.
 *   ws [dev]: cdl_workspace_bytes(CDL_OP_QLINEAR_BWD, M, N, K) bytes, 256-byte aligned.
 * CDL_ERR_OVERFLOW_RISK when dXacc (dWacc) is requested and N*max|g|*max|w| (M*max|a|*max|g|) reaches 2^31; the
 * float outputs alone are always available (exact int32 parts summed in int64, as for cdl_qlinear_fwd), which is
 * what lets dW reduce over millions of rows.
 */
int cdl_qlinear_bwd(const void *G_idx, int64_t ldg, const cdl_index_desc *g,
                    const void *A_idx, int64_t lda, const cdl_index_desc *a,
                    const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                    int32_t M, int32_t N, int32_t K,
                    int32_t *dXacc, float *dX, int32_t *dWacc, float *dW,
                    void *ws, size_t ws_bytes, void *stream);

/*
 * The rescale of the products' epilogue on its own (Sec. V-A: the integer sums times the two step sizes), for
 * accumulators that were summed outside a product call - data-parallel ranks all-reduce the int32 dWacc of
 * cdl_qlinear_bwd / cdl_qconv_bwd (integers: the sum does not depend on the number of ranks or their order) and
 * convert once afterwards:   out[i] = (float)acc[i] * (q_x * q_y),   the two step sizes of the product's operands
 * multiplied once in binary32, the conversion and the multiply each rounded to binary32 - the bits a single product
 * over the whole batch gives.
 *   acc [dev] n integers of acc_bits (32 or 64; 64 when the sum over all ranks could leave int32), naturally aligned;
 *   out [dev] n floats.  n = 0 is valid.
 */
int cdl_rescale_acc(const void *acc, int32_t acc_bits, int64_t n, float q_x, float q_y, float *out, void *stream);

/*
 * Backward layer products for a real-valued incoming gradient (Algorithm 1's backward pass as printed: dL/dY is
 * not quantized there; cdl_qlinear_bwd is the int8-gradient reading).  The gradient is expanded in two int8 digits,
 *   g ~ q1 i1 + q2 i2,  q1 = g_absmax / 127,  q2 = q1 / 254,
 *   i1 = clamp(rint(g / q1), -127, 127),  i2 = clamp(rint(RN(g - i1 q1) / q2), -127, 127)      (binary32),
 * so |g - (q1 i1 + q2 i2)| <= q1 / 508 = g_absmax / 64516 for |g| <= g_absmax (larger entries saturate), and each
 * digit plane goes through the exact integer product of cdl_qlinear_bwd:
 *   dX[m,k] = RN(RN((float)(I1 W^T)[m,k] * (q1 w->q)) + RN((float)(I2 W^T)[m,k] * (q2 w->q)))      and dW likewise with a->q.
 * Against the products with the real gradient the error is at most (g_absmax / 64516) * sum_n |w->q W_idx[k,n]| per
 * entry of dX (sum_m |a->q A_idx[m,k]| for dW) plus binary32 rounding of the result.
 *   G [dev] M x N floats (row pitch N); g_absmax > 0: the caller's bound on |G|.
 *   dX [dev] M x K floats, dW [dev] K x N floats, each nullable; A_idx / W_idx as in cdl_qlinear_bwd.
 *   ws [dev]: cdl_qlinear_bwd_fp_workspace_bytes(M, N, K) bytes (holds the two digit planes), 256-byte aligned.
 */
int cdl_qlinear_bwd_fp(const float *G, float g_absmax,
                       const void *A_idx, int64_t lda, const cdl_index_desc *a,
                       const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                       int32_t M, int32_t N, int32_t K, float *dX, float *dW,
                       void *ws, size_t ws_bytes, void *stream);
size_t cdl_qlinear_bwd_fp_workspace_bytes(int32_t M, int32_t N, int32_t K);


/*
 * Weight-gradient product for callers that cannot allocate device memory.  (The paper has no counterpart
 * of this entry point; it is a packaging variant of the dW half of cdl_qlinear_bwd.)
 *
 * Who needs it: code that runs where a cudaMalloc is off the table - for example inside a training process
 * whose framework allocator has already reserved nearly all device memory, so that a raw allocation fails
 * or fragments the pool, or inside a latency-bound step loop that must not hit the implicit device
 * synchronisation of cudaMalloc / cudaFree.  Such a caller has nowhere to get the workspace that
 * cdl_qlinear_bwd asks for.  Here the split-reduction scratch (int32 accumulators) and the status word sit in
 * a static device array inside the library instead; every GPU that loads the library holds that array
 * (256 bytes + 4 * CDL_NOALLOC_MAX_DW_ELEMS bytes = 4 MiB + 256 B) until the process exits.
 *
 *   dW[k,n] = (float)(sum_m A_idx[m,k] * G_idx[m,n]) * (g->q * a->q)      -- same values as cdl_qlinear_bwd
 *   G_idx [dev] M x N int8 (ld ldg), A_idx [dev] M x K bytes (ld lda), dW [dev] K x N floats; alignment and
 *   leading-dimension rules as for cdl_qlinear_bwd.  The caller still owns inputs and output.
 *
 * Limits: K * N <= CDL_NOALLOC_MAX_DW_ELEMS, otherwise CDL_ERR_TOO_LARGE; and M * max|a| * max|g| < 2^31 for the
 * declared index ranges (the sum over M must fit the int32 accumulators: there is no room here for the per-part
 * slabs with which cdl_qlinear_bwd sums longer reductions in int64), otherwise CDL_ERR_OVERFLOW_RISK - for
 * indices 0..15 against -127..127 that is M <= 1,127,288 rows.  In both cases nothing is launched.  Within the
 * limits the values are those of cdl_qlinear_bwd, bit for bit.
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 * Set-up: the first call on each device (with that device current) looks up the array's device address;
 * make that first call before any stream capture begins.
 * Sharing: all calls on a device use the same array, which still holds the previous call's contents; the
 * call clears what it needs before use.  Two calls whose GPU work can overlap (different streams, no
 * dependency) race on it: serialise them.  A bounded device-side wait that expires is recorded in the array's
 * status block; cdl_noalloc_status reads it.
 */
#define CDL_NOALLOC_MAX_DW_ELEMS (1 << 20)
int cdl_qlinear_bwd_dw_noalloc(const void *G_idx, int64_t ldg, const cdl_index_desc *g,
                               const void *A_idx, int64_t lda, const cdl_index_desc *a,
                               int32_t M, int32_t N, int32_t K, float *dW, void *stream);

/* cdl_workspace_status for the built-in scratch of cdl_qlinear_bwd_dw_noalloc on the current device: synchronises
 * `stream`, returns CDL_ERR_TIMEOUT (and clears the record) when a wait of such a call gave up, else CDL_OK.
 * Allocates nothing.  (No counterpart in the paper.) */
int cdl_noalloc_status(void *stream);

/*
 * The same three layer products for a convolutional layer (the layers of the paper's networks, Sec. VI-C and
 * VI-D, are convolutions, the first of every ResNet stage with stride 2; Algorithm 1, forward and backward pass),
 * computed straight from the NHWC index tensors: the patch matrix whose rows cdl_qlinear_* takes as A_idx is never
 * written to memory, its tiles are gathered by the loads of the kernel, with zero (= index 0 = level 0) outside the
 * image.
 * Cross-correlation with filter R x S (1 <= R, S <= 7), stride 1..4 (the same in both directions) and zero padding
 * pad_h < R, pad_w < S; output P x Q per image, P = (H + 2 pad_h - R) / stride + 1, Q likewise (integer division).
 * C and C_out multiples of 64 (else CDL_ERR_ARG: form the patch matrix and call cdl_qlinear_*).
 *   X_idx [dev] N x H x W x C index bytes (signedness from x);  G_idx [dev] N x P x Q x C_out int8;
 *   W_idx [dev] (R*S*C) x C_out int8, row (r*S + s)*C + c, leading dimension ldw (multiple of 16);
 *   all three 16-byte aligned.
 *   forward   ACC[n,p,q,co] = sum_{r,s,c} X_idx[n, p*stride-pad_h+r, q*stride-pad_w+s, c] * W_idx[(r*S+s)*C+c, co]
 *             Y = (float)ACC * (x->q * w->q) + bias[co]            acc_out, y_out: N x P x Q x C_out, nullable
 *   backward  dXACC[n,h,w,c] = sum of G_idx[n,p,q,co] * W_idx[(r*S+s)*C+c, co] over co and the (r,s,p,q) with
 *             p*stride-pad_h+r = h, q*stride-pad_w+s = w (the adjoint of the forward map in X)
 *             dX = (float)dXACC * (g->q * w->q)                     dXacc, dX: N x H x W x C, nullable
 *             dWACC[(r*S+s)*C+c, co] = sum_{n,p,q} X_idx[n, p*stride-pad_h+r, q*stride-pad_w+s, c] * G_idx[n,p,q,co]
 *             dW = (float)dWACC * (g->q * x->q)                     dWacc, dW: (R*S*C) x C_out (ld C_out), nullable
 *   X_idx may be NULL when no dW output is wanted, W_idx when no dX output is.
 *   ws [dev]: cdl_qconv_workspace_bytes(shape, C_out) bytes, 256-byte aligned.
 * Overflow rule and the int64 summation of long reductions as for cdl_qlinear_* (with a stride above 1 the data
 * gradient is one product per residue class of pixels and has no such long-reduction path: CDL_ERR_OVERFLOW_RISK).
 */
typedef struct {
    int32_t N, H, W, C;   /* the layer's input tensor */
    int32_t R, S;         /* filter height and width */
    int32_t stride;       /* 1..4; 0 means 1 */
    int32_t pad_h, pad_w; /* zero padding on each side; a negative value means (R-1)/2 resp. (S-1)/2 */
} cdl_conv_shape;

int cdl_qconv_fwd(const void *X_idx, const cdl_index_desc *x, const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                  const cdl_conv_shape *shape, int32_t C_out, int32_t *acc_out, float *y_out, const float *bias,
                  void *ws, size_t ws_bytes, void *stream);

int cdl_qconv_fwd_next(const void *X_idx, const cdl_index_desc *x, const void *W_idx, int64_t ldw,
                       const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out,
                       int32_t *acc_out, float *y_out, const float *bias,
                       const cdl_index_desc *next, void *idx_next, void *ws, size_t ws_bytes, void *stream);

int cdl_qconv_bwd(const void *G_idx, const cdl_index_desc *g, const void *X_idx, const cdl_index_desc *x,
                  const void *W_idx, int64_t ldw, const cdl_index_desc *w, const cdl_conv_shape *shape, int32_t C_out,
                  int32_t *dXacc, float *dX, int32_t *dWacc, float *dW, void *ws, size_t ws_bytes, void *stream);

/* Bytes of device workspace cdl_qconv_fwd / cdl_qconv_bwd need; 0 for an unsupported shape. */
size_t cdl_qconv_workspace_bytes(const cdl_conv_shape *shape, int32_t C_out);

/* cdl_qlinear_bwd_fp for a convolutional layer (shapes, layouts and limits of cdl_qconv_bwd): G [dev] N x H x W x C_out floats;
 * dX [dev] N x H x W x C floats, dW [dev] (R*S*C) x C_out floats, each nullable;
 * ws [dev]: cdl_qconv_bwd_fp_workspace_bytes(shape, C_out) bytes, 256-byte aligned. */
int cdl_qconv_bwd_fp(const float *G, float g_absmax, const void *X_idx, const cdl_index_desc *x,
                     const void *W_idx, int64_t ldw, const cdl_index_desc *w,
                     const cdl_conv_shape *shape, int32_t C_out, float *dX, float *dW,
                     void *ws, size_t ws_bytes, void *stream);
size_t cdl_qconv_bwd_fp_workspace_bytes(const cdl_conv_shape *shape, int32_t C_out);

#define CDL_OP_QLINEAR_FWD 1
#define CDL_OP_QLINEAR_BWD 2

/* Bytes of device workspace the GEMM entry points need for these sizes; never less than the
 * 256-byte status block at its start.  0 for an unknown op or non-positive sizes. */
size_t cdl_workspace_bytes(int32_t op, int32_t M, int32_t N, int32_t K);

/* Synchronises `stream` and reports whether a bounded device-side wait of a GEMM call that used this workspace
 * gave up: CDL_ERR_TIMEOUT (the outputs of that call are then undefined; the record is cleared by this call) or
 * CDL_OK.  The GEMM calls never touch the status block (the first 16 bytes of a workspace) unless a wait expires, in
 * which case they store a record there - CDL_ERR_TIMEOUT followed by two tag words - that stays until read here;
 * any other content, such as whatever a fresh or recycled allocation holds, reads as OK. */
int cdl_workspace_status(void *ws, void *stream);

/* Static, NUL-terminated description of a status code. */
const char *cdl_strerror(int status);

/* CDL_VERSION of the built library. */
int cdl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CDL_H_ */
