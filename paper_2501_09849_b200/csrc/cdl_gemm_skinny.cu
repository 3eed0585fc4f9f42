// Layer products whose weight matrix has few output channels (N <= 32: the 16-channel layers of CIFAR ResNets).
// With K * N of a few thousand there are only ~10 multiply-adds per byte moved, so these products are bound by
// HBM, not by arithmetic, and a 128-row tensor-core tile spends its time on hand-shakes: here they are streaming
// kernels on the integer dot-product instruction (dp4a, four byte products per lane and instruction), exact in
// int32 like the tensor-core path and with the same float epilogue.
//   forward  Y[m, :]  = A[m, :] W        one thread per row: its A row in registers, W packed four k per word in
//                                        shared memory and read as broadcasts
//   dX       dA[m, :] = G[m, :] W^T      one warp per 32 rows: lane = output column (coalesced 128-byte stores), its
//                                        W rows in registers, the G rows broadcast by shuffles
#include "cdl_internal.h"

namespace cdl {
namespace {

constexpr int kSkinnyThreads = 256;

template <bool A_UNSIGNED>
__device__ __forceinline__ int dot4(unsigned int a, unsigned int b, int c)
{
    int d;
    if (A_UNSIGNED) asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    else asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// ------------------------------------------------------------------------------------------------ forward
// Wp[k4 * N + n] = bytes W[4 k4 .. 4 k4 + 3][n]; K a multiple of 16, N a multiple of 4, N <= 32.
// STAGED: a warp first copies its 32 rows of A into shared memory with coalesced 16-byte loads and every lane then
// reads its own row from there; otherwise every lane reads its row straight from global memory (rows too long to
// stage for eight warps).
template <int N, bool A_UNSIGNED, bool STAGED>
__global__ void __launch_bounds__(kSkinnyThreads)
skinny_fwd_kernel(const unsigned char *__restrict__ A, long long lda, const signed char *__restrict__ W, long long ldw,
                  int M, int K, int32_t *__restrict__ acc_out, float *__restrict__ y_out, float scale,
                  const float *__restrict__ bias)
{
    extern __shared__ __align__(16) unsigned int Wp[];
    const int k4n = K / 4;
    for (int i = threadIdx.x; i < k4n * N; i += kSkinnyThreads) {
        const int k4 = i / N, n = i - k4 * N;
        unsigned int w = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) w |= (unsigned int)(unsigned char)W[(long long)(4 * k4 + b) * ldw + n] << (8 * b);
        Wp[i] = w;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp_in_cta = threadIdx.x >> 5;
    const int k16 = K / 16;
    uint4 *stage = reinterpret_cast<uint4 *>(Wp + k4n * N) + (size_t)warp_in_cta * 32 * k16;      // [32 rows][K / 16]
    const long long stride = (long long)gridDim.x * kSkinnyThreads;
    // whole warps iterate together (the staging copy is a warp's job); rows past M are skipped at the end
    for (long long m0 = (long long)blockIdx.x * kSkinnyThreads + warp_in_cta * 32; m0 < M; m0 += stride) {
        const long long m = m0 + lane;
        if (STAGED) {
            __syncwarp();
            for (int i = lane; i < 32 * k16; i += 32) {
                const int r = i / k16, c = i - r * k16;
                if (m0 + r < M) stage[i] = __ldcs(reinterpret_cast<const uint4 *>(A + (m0 + r) * lda) + c);
            }
            __syncwarp();
        }
        if (m >= M) continue;
        int acc[N];
#pragma unroll
        for (int n = 0; n < N; ++n) acc[n] = 0;
        const uint4 *arow = STAGED ? stage + (size_t)lane * k16 : reinterpret_cast<const uint4 *>(A + m * lda);
        for (int c = 0; c < k16; ++c) {
            const uint4 a = STAGED ? arow[c] : __ldcs(arow + c);
            const unsigned int aw[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 *wrow = reinterpret_cast<const uint4 *>(Wp + (4 * c + j) * N);
#pragma unroll
                for (int n4 = 0; n4 < N / 4; ++n4) {
                    const uint4 w = wrow[n4];                    // same address in every lane: a broadcast
                    acc[4 * n4 + 0] = dot4<A_UNSIGNED>(aw[j], w.x, acc[4 * n4 + 0]);
                    acc[4 * n4 + 1] = dot4<A_UNSIGNED>(aw[j], w.y, acc[4 * n4 + 1]);
                    acc[4 * n4 + 2] = dot4<A_UNSIGNED>(aw[j], w.z, acc[4 * n4 + 2]);
                    acc[4 * n4 + 3] = dot4<A_UNSIGNED>(aw[j], w.w, acc[4 * n4 + 3]);
                }
            }
        }
        if (acc_out != nullptr) {
            int4 *o = reinterpret_cast<int4 *>(acc_out + m * N);
#pragma unroll
            for (int n4 = 0; n4 < N / 4; ++n4) o[n4] = make_int4(acc[4 * n4], acc[4 * n4 + 1], acc[4 * n4 + 2], acc[4 * n4 + 3]);
        }
        if (y_out != nullptr) {
            float4 *o = reinterpret_cast<float4 *>(y_out + m * N);
#pragma unroll
            for (int n4 = 0; n4 < N / 4; ++n4) {
                float f[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    f[b] = __fmul_rn((float)acc[4 * n4 + b], scale);
                    if (bias != nullptr) f[b] = __fadd_rn(f[b], bias[4 * n4 + b]);
                }
                __stcs(o + n4, make_float4(f[0], f[1], f[2], f[3]));
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ dX
// NW = N / 4 words per row of G and of W; KPL output columns per lane and pass (a pass covers 32 * KPL columns).
template <int NW, int KPL>
__global__ void __launch_bounds__(kSkinnyThreads)
skinny_dx_kernel(const signed char *__restrict__ G, long long ldg, const signed char *__restrict__ W, long long ldw,
                 int M, int K, int32_t *__restrict__ acc_out, float *__restrict__ f_out, float scale, int accumulate)
{
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * kSkinnyThreads + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * kSkinnyThreads) >> 5;
    const long long nblocks = ((long long)M + 31) / 32;
    for (int kbase = 0; kbase < K; kbase += 32 * KPL) {
        // this lane's rows of W for the pass: columns kbase + j * 32 + lane
        unsigned int wreg[KPL][NW];
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const int k = kbase + j * 32 + lane;
#pragma unroll
            for (int w = 0; w < NW; ++w)
                wreg[j][w] = k < K ? *reinterpret_cast<const unsigned int *>(W + (long long)k * ldw + 4 * w) : 0u;
        }
        for (long long blk = warp; blk < nblocks; blk += nwarps) {
            const long long row0 = blk * 32;
            // lane r holds row row0 + r of G
            unsigned int g[NW];
            const long long myrow = row0 + lane;
#pragma unroll
            for (int w = 0; w < NW; ++w)
                g[w] = myrow < M ? *reinterpret_cast<const unsigned int *>(G + myrow * ldg + 4 * w) : 0u;
            const int nrows = (int)((M - row0) < 32 ? (M - row0) : 32);
            for (int r = 0; r < nrows; ++r) {
                unsigned int gr[NW];
#pragma unroll
                for (int w = 0; w < NW; ++w) gr[w] = __shfl_sync(0xffffffffu, g[w], r);
#pragma unroll
                for (int j = 0; j < KPL; ++j) {
                    const int k = kbase + j * 32 + lane;
                    int acc = 0;
#pragma unroll
                    for (int w = 0; w < NW; ++w) acc = dot4<false>(gr[w], wreg[j][w], acc);
                    if (k < K) {
                        const long long o = (row0 + r) * K + k;
                        if (acc_out != nullptr) acc_out[o] = acc;
                        if (f_out != nullptr) {
                            const float v = __fmul_rn((float)acc, scale);
                            if (accumulate) f_out[o] = __fadd_rn(f_out[o], v);
                            else __stcs(f_out + o, v);
                        }
                    }
                }
            }
        }
    }
}

int grid_for(long long work_items)
{
    const int sms = sm_count();
    if (sms <= 0) return 0;
    long long blocks = (work_items + kSkinnyThreads - 1) / kSkinnyThreads;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    return (int)(blocks < 1 ? 1 : blocks);
}

template <int N, bool A_UNSIGNED, bool STAGED>
int launch_fwd_t(const unsigned char *a, long long lda, const signed char *w, long long ldw, int M, int K, int32_t *acc_out,
                 float *y_out, float scale, const float *bias, cudaStream_t stream)
{
    const int grid = grid_for(M);
    if (grid == 0) return CDL_ERR_LAUNCH;
    const size_t smem = (size_t)K * N + (STAGED ? (size_t)(kSkinnyThreads / 32) * 32 * K : 0);
    auto kern = skinny_fwd_kernel<N, A_UNSIGNED, STAGED>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    kern<<<grid, kSkinnyThreads, smem, stream>>>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

template <int N>
int launch_fwd_n(const void *A, long long lda, bool a_unsigned, const void *W, long long ldw, int M, int K,
                 int32_t *acc_out, float *y_out, float scale, const float *bias, cudaStream_t stream)
{
    const unsigned char *a = static_cast<const unsigned char *>(A);
    const signed char *w = static_cast<const signed char *>(W);
    const bool staged = (size_t)K * N + (size_t)kSkinnyThreads * K <= 96 * 1024;
    if (a_unsigned)
        return staged ? launch_fwd_t<N, true, true>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream)
                      : launch_fwd_t<N, true, false>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream);
    return staged ? launch_fwd_t<N, false, true>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream)
                  : launch_fwd_t<N, false, false>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream);
}

template <int NW>
int launch_dx_nw(const void *G, long long ldg, const void *W, long long ldw, int M, int K, int32_t *acc_out, float *f_out,
                 float scale, bool accumulate, cudaStream_t stream)
{
    const int grid = grid_for((long long)((M + 31) / 32) * 32);
    if (grid == 0) return CDL_ERR_LAUNCH;
    const signed char *g = static_cast<const signed char *>(G);
    const signed char *w = static_cast<const signed char *>(W);
    const int acc = accumulate ? 1 : 0;
    const int kpl = (K + 31) / 32;
    if (kpl <= 2) skinny_dx_kernel<NW, 2><<<grid, kSkinnyThreads, 0, stream>>>(g, ldg, w, ldw, M, K, acc_out, f_out, scale, acc);
    else if (kpl <= 5) skinny_dx_kernel<NW, 5><<<grid, kSkinnyThreads, 0, stream>>>(g, ldg, w, ldw, M, K, acc_out, f_out, scale, acc);
    else skinny_dx_kernel<NW, 8><<<grid, kSkinnyThreads, 0, stream>>>(g, ldg, w, ldw, M, K, acc_out, f_out, scale, acc);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace

bool skinny_fwd_ok(int M, int N, int K)
{
    (void)M;
    return (N == 4 || N == 8 || N == 16 || N == 32) && (K % 16) == 0 && (long long)K * N <= 96 * 1024;
}

bool skinny_dx_ok(int M, int N, int K)
{
    (void)M;
    (void)K;
    return N == 4 || N == 8 || N == 16 || N == 32;
}

// Y (M x N, row pitch N) from A (M x K bytes, pitch lda, 16-byte aligned rows) and W (K x N int8, pitch ldw)
int launch_skinny_fwd(const void *A, long long lda, bool a_unsigned, const void *W, long long ldw, int M, int N, int K,
                      int32_t *acc_out, float *y_out, float scale, const float *bias, cudaStream_t stream)
{
    switch (N) {
        case 4: return launch_fwd_n<4>(A, lda, a_unsigned, W, ldw, M, K, acc_out, y_out, scale, bias, stream);
        case 8: return launch_fwd_n<8>(A, lda, a_unsigned, W, ldw, M, K, acc_out, y_out, scale, bias, stream);
        case 16: return launch_fwd_n<16>(A, lda, a_unsigned, W, ldw, M, K, acc_out, y_out, scale, bias, stream);
        case 32: return launch_fwd_n<32>(A, lda, a_unsigned, W, ldw, M, K, acc_out, y_out, scale, bias, stream);
        default: return CDL_ERR_ARG;
    }
}

// dA (M x K, row pitch K) from G (M x N int8, pitch ldg, 4-byte aligned rows) and W (K x N int8, pitch ldw)
int launch_skinny_dx(const void *G, long long ldg, const void *W, long long ldw, int M, int N, int K, int32_t *acc_out,
                     float *f_out, float scale, bool accumulate, cudaStream_t stream)
{
    switch (N) {
        case 4: return launch_dx_nw<1>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 8: return launch_dx_nw<2>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 16: return launch_dx_nw<4>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 32: return launch_dx_nw<8>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        default: return CDL_ERR_ARG;
    }
}

}  // namespace cdl
