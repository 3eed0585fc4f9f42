// Two-digit integer expansion of a real-valued gradient tensor (backward products with an unquantized dL/dY):
//   g ~ q1 * i1 + q2 * i2,   i1 = clamp(rint(g / q1), -127, 127),  r = RN(g - i1 q1),  i2 = clamp(rint(r / q2), -127, 127)
// with q2 = q1 / 254, so that |g - (q1 i1 + q2 i2)| <= q2 / 2 = q1 / 508 wherever |g| <= 127.5 q1.  Both digit planes
// then go through the exact integer products.  Element-wise, one pass: 4 bytes read, 2 written per element (HBM-bound).
#include "cdl_internal.h"

namespace cdl {
namespace {

__device__ __forceinline__ int digit(float v, float q)
{
    return __float2int_rn(fminf(fmaxf(__fdiv_rn(v, q), -127.0f), 127.0f));     // NaN clamps to -127
}

// the two digits of four consecutive gradients, packed as the bytes of two words
__device__ __forceinline__ void digits4(float4 v, float q1, float q2, unsigned int &w1, unsigned int &w2)
{
    const float in[4] = {v.x, v.y, v.z, v.w};
    w1 = 0u;
    w2 = 0u;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int i1 = digit(in[c], q1);
        const int i2 = digit(__fmaf_rn(-(float)i1, q1, in[c]), q2);
        w1 |= ((unsigned int)i1 & 0xffu) << (8 * c);
        w2 |= ((unsigned int)i2 & 0xffu) << (8 * c);
    }
}

// Rows of `cols` floats (pitch cols) -> two planes of digit bytes (pitch ld >= cols, a multiple of 16).  VEC: cols is
// a multiple of 4 and g is 16-byte aligned, so every row starts on a 16-byte boundary of g and on a 4-byte boundary
// of the planes: 128-bit loads, packed 4-byte stores.  With ld == cols the tensor is one long row (no division at
// all); otherwise a block walks whole rows.
template <bool VEC>
__global__ void __launch_bounds__(256)
gradient_digits_kernel(const float *__restrict__ g, long long rows, int cols, int ld, float q1, float q2,
                       signed char *__restrict__ d1, signed char *__restrict__ d2)
{
    for (long long r = blockIdx.y; r < rows; r += gridDim.y) {
        const float *gr = g + r * cols;
        signed char *o1 = d1 + r * ld, *o2 = d2 + r * ld;
        const long long stride = (long long)gridDim.x * blockDim.x;
        const long long first = (long long)blockIdx.x * blockDim.x + threadIdx.x;
        if (VEC) {
            const float4 *g4 = reinterpret_cast<const float4 *>(gr);
            unsigned int *p1 = reinterpret_cast<unsigned int *>(o1), *p2 = reinterpret_cast<unsigned int *>(o2);
            for (long long i = first; i < cols / 4; i += stride) {
                unsigned int w1, w2;
                digits4(__ldcs(g4 + i), q1, q2, w1, w2);
                p1[i] = w1;
                p2[i] = w2;
            }
        } else {
            for (long long i = first; i < cols; i += stride) {
                const float v = gr[i];
                const int i1 = digit(v, q1);
                o1[i] = (signed char)i1;
                o2[i] = (signed char)digit(__fmaf_rn(-(float)i1, q1, v), q2);
            }
        }
    }
}

}  // namespace

int launch_gradient_digits(const float *g, long long rows, int cols, int ld, float q1, float q2, void *d1, void *d2,
                           cudaStream_t stream)
{
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    // an unpadded tensor is one row of rows * cols elements
    long long nrows = rows, ncols = cols;
    if (ld == cols && rows * (long long)cols < (1ll << 31)) {
        ncols = rows * cols;
        nrows = 1;
    }
    const bool vec = (ncols % 4 == 0) && (reinterpret_cast<uintptr_t>(g) % 16 == 0) && (ld % 4 == 0) &&
                     (reinterpret_cast<uintptr_t>(d1) % 4 == 0) && (reinterpret_cast<uintptr_t>(d2) % 4 == 0);
    const long long per_row = vec ? ncols / 4 : ncols;
    long long bx = (per_row + 255) / 256;
    const long long cap = (long long)sms * 8;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    long long by = cap / bx;
    if (by > nrows) by = nrows;
    if (by < 1) by = 1;
    if (by > 65535) by = 65535;
    const dim3 grid((unsigned int)bx, (unsigned int)by);
    signed char *p1 = static_cast<signed char *>(d1), *p2 = static_cast<signed char *>(d2);
    if (vec) gradient_digits_kernel<true><<<grid, 256, 0, stream>>>(g, nrows, (int)ncols, nrows == 1 ? (int)ncols : ld, q1, q2, p1, p2);
    else gradient_digits_kernel<false><<<grid, 256, 0, stream>>>(g, nrows, (int)ncols, nrows == 1 ? (int)ncols : ld, q1, q2, p1, p2);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace cdl
