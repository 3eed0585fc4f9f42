// Two-digit integer expansion of a real-valued gradient tensor (backward products with an unquantized dL/dY):
//   g ~ q1 * i1 + q2 * i2,   i1 = clamp(rint(g / q1), -127, 127),  r = RN(g - i1 q1),  i2 = clamp(rint(r / q2), -127, 127)
// with q2 = q1 / 254, so that |g - (q1 i1 + q2 i2)| <= q2 / 2 = q1 / 508 wherever |g| <= 127.5 q1.  Both digit planes
// then go through the exact integer products.  Element-wise, one pass: 4 bytes read, 2 written per element.
#include "cdl_internal.h"

namespace cdl {
namespace {

__device__ __forceinline__ int digit(float v, float q)
{
    return __float2int_rn(fminf(fmaxf(__fdiv_rn(v, q), -127.0f), 127.0f));     // NaN clamps to -127
}

__global__ void __launch_bounds__(256)
gradient_digits_kernel(const float *__restrict__ g, long long rows, int cols, int ld, float q1, float q2,
                       signed char *__restrict__ d1, signed char *__restrict__ d2)
{
    const long long n = rows * cols;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float v = g[i];
        const int i1 = digit(v, q1);
        const float r = __fmaf_rn(-(float)i1, q1, v);
        const int i2 = digit(r, q2);
        const long long o = (i / cols) * ld + (i % cols);
        d1[o] = (signed char)i1;
        d2[o] = (signed char)i2;
    }
}

}  // namespace

int launch_gradient_digits(const float *g, long long rows, int cols, int ld, float q1, float q2, void *d1, void *d2,
                           cudaStream_t stream)
{
    const long long n = rows * cols;
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    long long blocks = (n + 255) / 256;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    if (blocks < 1) blocks = 1;
    gradient_digits_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(g, rows, cols, ld, q1, q2, static_cast<signed char *>(d1),
                                                                     static_cast<signed char *>(d2));
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace cdl
