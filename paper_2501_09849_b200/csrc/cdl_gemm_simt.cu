// Index GEMM on the integer dot-product units (dp4a): C[i,j] = sum_r X(i,r) Y(r,j) over int8/uint8
// index bytes with arbitrary strides, int32 accumulation, optional float epilogue.
// This is the plain path: it serves shapes and alignments the tensor-core path does not take and
// is bit-exact by construction (integer arithmetic only).
#include "cdl_internal.h"

namespace cdl {
namespace {

constexpr int TI = 64, TJ = 64, TR = 32, PAD = 36;

template <bool XU, bool YU>
__device__ __forceinline__ int dot4(unsigned int a, unsigned int b, int c)
{
    int d;
    if (XU && YU) asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    else if (XU) asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    else if (YU) asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    else asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ void load_tile(unsigned char (*dst)[PAD], const unsigned char *p, int64_t so, int64_t sr,
                                          int o0, int r0, int O, int R)
{
    // 64 x 32 bytes; walk the contiguous dimension fastest
    const bool outer_fast = (so == 1);
#pragma unroll
    for (int l = 0; l < (TI * TR) / 256; ++l) {
        const int e = threadIdx.x + 256 * l;
        const int row = outer_fast ? (e % TI) : (e / TR);
        const int rr = outer_fast ? (e / TI) : (e % TR);
        const int o = o0 + row, r = r0 + rr;
        unsigned char v = 0;
        if (o < O && r < R) v = p[(int64_t)o * so + (int64_t)r * sr];
        dst[row][rr] = v;
    }
}

template <bool XU, bool YU>
__global__ void __launch_bounds__(256)
index_gemm_kernel(const unsigned char *__restrict__ X, int64_t xso, int64_t xsr,
                  const unsigned char *__restrict__ Y, int64_t yso, int64_t ysr,
                  int I, int J, int R, int32_t *__restrict__ acc_out, float *__restrict__ f_out,
                  float scale, const float *__restrict__ bias)
{
    __shared__ __align__(16) unsigned char Xs[TI][PAD];
    __shared__ __align__(16) unsigned char Ys[TJ][PAD];
    const int i0 = blockIdx.x * TI, j0 = blockIdx.y * TJ;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    int acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0;

    for (int r0 = 0; r0 < R; r0 += TR) {
        load_tile(Xs, X, xso, xsr, i0, r0, I, R);
        load_tile(Ys, Y, yso, ysr, j0, r0, J, R);
        __syncthreads();
#pragma unroll
        for (int c = 0; c < TR / 4; ++c) {
            unsigned int xa[4], yb[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) xa[a] = *reinterpret_cast<const unsigned int *>(&Xs[ty * 4 + a][c * 4]);
#pragma unroll
            for (int b = 0; b < 4; ++b) yb[b] = *reinterpret_cast<const unsigned int *>(&Ys[tx * 4 + b][c * 4]);
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = dot4<XU, YU>(xa[a], yb[b], acc[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int i = i0 + ty * 4 + a;
        if (i >= I) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int j = j0 + tx * 4 + b;
            if (j >= J) continue;
            const int64_t off = (int64_t)i * J + j;
            if (acc_out) acc_out[off] = acc[a][b];
            if (f_out) {
                float v = __fmul_rn((float)acc[a][b], scale);
                if (bias) v = __fadd_rn(v, bias[j]);
                f_out[off] = v;
            }
        }
    }
}

}  // namespace

int launch_index_gemm(const GemmOperand &X, const GemmOperand &Y, int I, int J, int R,
                      int32_t *acc_out, float *f_out, float scale, const float *bias, cudaStream_t stream)
{
    dim3 grid((I + TI - 1) / TI, (J + TJ - 1) / TJ);
    if (grid.y > 65535u) return CDL_ERR_ARG;
    const unsigned char *xp = static_cast<const unsigned char *>(X.ptr);
    const unsigned char *yp = static_cast<const unsigned char *>(Y.ptr);
#define CDL_LAUNCH(XU, YU)                                                                             \
    index_gemm_kernel<XU, YU><<<grid, 256, 0, stream>>>(xp, X.stride_outer, X.stride_red, yp, Y.stride_outer, \
                                                        Y.stride_red, I, J, R, acc_out, f_out, scale, bias)
    if (X.is_unsigned && Y.is_unsigned) CDL_LAUNCH(true, true);
    else if (X.is_unsigned) CDL_LAUNCH(true, false);
    else if (Y.is_unsigned) CDL_LAUNCH(false, true);
    else CDL_LAUNCH(false, false);
#undef CDL_LAUNCH
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace cdl
