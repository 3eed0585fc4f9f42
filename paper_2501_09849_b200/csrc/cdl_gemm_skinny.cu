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

// ------------------------------------------------------------------------------------------------ dW
// dW[k, n] = sum_m A[m, k] G[m, n]: the contraction runs over rows, so both operands are needed with four
// consecutive rows of one column in a word.  A warp works alone on jobs of 32 rows x (16 MT columns of A): it reads
// the rows with coalesced 4-byte loads, four rows at a time, transposes 4 x 4 byte blocks in registers (byte
// permutes), parks the words in its own shared-memory patch and multiplies from there with the warp-level int8
// matrix instruction (m16n8k32: 16 columns of A x 8 of G x 32 rows), sums in registers across its jobs.  The next
// job's loads are in flight during the multiplication.  At the end the warps of a CTA add their sums in shared
// memory and the CTA adds them to the int32 result with coalesced reductions; the last CTA to finish converts.
constexpr int kDwWarps = 12;

__device__ __forceinline__ void transpose4x4(unsigned int r0, unsigned int r1, unsigned int r2, unsigned int r3,
                                             unsigned int (&o)[4])
{
    const unsigned int t0 = __byte_perm(r0, r1, 0x5140), t1 = __byte_perm(r2, r3, 0x5140);
    const unsigned int t2 = __byte_perm(r0, r1, 0x7362), t3 = __byte_perm(r2, r3, 0x7362);
    o[0] = __byte_perm(t0, t1, 0x5410);
    o[1] = __byte_perm(t0, t1, 0x7632);
    o[2] = __byte_perm(t2, t3, 0x5410);
    o[3] = __byte_perm(t2, t3, 0x7632);
}

// D (16 x 8, int32) += A (16 x 32 bytes, row-major fragment) B (32 x 8 int8, column fragment)
template <bool A_UNSIGNED>
__device__ __forceinline__ void mma_k32(int (&d)[4], unsigned int a0, unsigned int a1, unsigned int a2, unsigned int a3,
                                        unsigned int b0, unsigned int b1)
{
    if (A_UNSIGNED)
        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DwTail {                 // what the last CTA to finish does with the sums
    float *f_out;
    float scale;
    int accumulate;
    unsigned int *counter;      // zeroed together with the sums
};

template <int N, int MT> struct DwGeom {
    static constexpr int NT = N >= 8 ? N / 8 : 1;           // 8-column tiles of G
    static constexpr int NP = NT * 8;
    static constexpr int KSL = 16 * MT;                     // columns of A per job
    static constexpr int KS = (KSL & 31) == 8 ? KSL : ((KSL + 23) / 32 * 32 + 8);   // patch row strides in words,
    static constexpr int GS = NP == 8 ? 8 : 40;                                     // = 8 mod 32: conflict-free
    static constexpr int GI = (2 * N + 31) / 32;            // 4 x 4 blocks of G per lane and job
    static constexpr int patch_words = 8 * (KS + GS);
    static constexpr size_t smem_bytes = ((size_t)kDwWarps * patch_words + (size_t)KSL * NP) * 4;
};

template <int N, int MT, bool A_UNSIGNED>
__global__ void __launch_bounds__(kDwWarps * 32, 1)
skinny_dw_kernel(const unsigned char *__restrict__ A, long long lda, const signed char *__restrict__ G, long long ldg,
                 int M, int K, int S, int32_t *__restrict__ acc_out, DwTail tail)
{
    using Geo = DwGeom<N, MT>;
    constexpr int NT = Geo::NT, NP = Geo::NP, KSL = Geo::KSL, KS = Geo::KS, GS = Geo::GS, GI = Geo::GI;
    extern __shared__ __align__(16) unsigned int smem_dw[];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = lane & 3, g = lane >> 2;
    unsigned int *At = smem_dw + warp * Geo::patch_words;       // [8][KS]: word (m4, k) = A[4 m4 .. 4 m4 + 3][k0 + k]
    unsigned int *Gt = At + 8 * KS;                             // [8][GS]
    int *red = reinterpret_cast<int *>(smem_dw + kDwWarps * Geo::patch_words);      // [KSL][NP]
    for (int i = threadIdx.x; i < KSL * NP; i += kDwWarps * 32) red[i] = 0;
    for (int i = lane; i < 8 * GS; i += 32) Gt[i] = 0u;         // columns N .. NP - 1 stay zero
    const int slice = blockIdx.x % S, k0 = slice * KSL;
    const long long cta_in_slice = blockIdx.x / S, ctas_per_slice = gridDim.x / S;
    const long long ngroups = ((long long)M + 31) / 32;
    const long long gstride = ctas_per_slice * kDwWarps;
    int acc[MT][NT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[i][j][c] = 0;
    unsigned int ra[MT][4], rg[GI][4];

    auto fetch = [&](long long grp) {
        const long long m0 = grp * 32;
#pragma unroll
        for (int j = 0; j < MT; ++j) {                          // 8 x 4 MT blocks: MT per lane
            const int i = lane + 32 * j;
            const int m4 = i / (4 * MT), k4 = i % (4 * MT);
            const int k = k0 + 4 * k4;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const long long m = m0 + 4 * m4 + b;
                ra[j][b] = (m < M && k < K) ? __ldg(reinterpret_cast<const unsigned int *>(A + m * lda + k)) : 0u;
            }
        }
#pragma unroll
        for (int j = 0; j < GI; ++j) {                          // 8 x N / 4 blocks
            const int i = lane + 32 * j;
            const int m4 = i / (N / 4), n4 = i % (N / 4);
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const long long m = m0 + 4 * m4 + b;
                rg[j][b] = (i < 2 * N && m < M) ? __ldg(reinterpret_cast<const unsigned int *>(G + m * ldg + 4 * n4)) : 0u;
            }
        }
    };

    long long grp = cta_in_slice * kDwWarps + warp;
    if (grp < ngroups) fetch(grp);
    __syncthreads();                                            // red and the patches are initialised
    for (; grp < ngroups; grp += gstride) {
#pragma unroll
        for (int j = 0; j < MT; ++j) {
            const int i = lane + 32 * j;
            const int m4 = i / (4 * MT), k4 = i % (4 * MT);
            unsigned int o[4];
            transpose4x4(ra[j][0], ra[j][1], ra[j][2], ra[j][3], o);
            *reinterpret_cast<uint4 *>(At + m4 * KS + 4 * k4) = make_uint4(o[0], o[1], o[2], o[3]);
        }
#pragma unroll
        for (int j = 0; j < GI; ++j) {
            const int i = lane + 32 * j;
            if (i < 2 * N) {
                const int m4 = i / (N / 4), n4 = i % (N / 4);
                unsigned int o[4];
                transpose4x4(rg[j][0], rg[j][1], rg[j][2], rg[j][3], o);
                *reinterpret_cast<uint4 *>(Gt + m4 * GS + 4 * n4) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        __syncwarp();
        if (grp + gstride < ngroups) fetch(grp + gstride);      // in flight while this job is multiplied
        unsigned int b0[NT], b1[NT];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            b0[j] = Gt[t * GS + 8 * j + g];
            b1[j] = Gt[(t + 4) * GS + 8 * j + g];
        }
#pragma unroll
        for (int i = 0; i < MT; ++i) {
            const unsigned int a0 = At[t * KS + 16 * i + g], a1 = At[t * KS + 16 * i + g + 8];
            const unsigned int a2 = At[(t + 4) * KS + 16 * i + g], a3 = At[(t + 4) * KS + 16 * i + g + 8];
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_k32<A_UNSIGNED>(acc[i][j], a0, a1, a2, a3, b0[j], b1[j]);
        }
        __syncwarp();                                           // the patch is free for the next job
    }
    // warps -> CTA (shared-memory adds) -> result (coalesced reductions)
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int row = 16 * i + g + (c >= 2 ? 8 : 0), col = 8 * j + 2 * t + (c & 1);
                if (acc[i][j][c] != 0) atomicAdd(red + row * NP + col, acc[i][j][c]);
            }
    __syncthreads();
    for (int i = threadIdx.x; i < KSL * N; i += kDwWarps * 32) {
        const int row = i / N, col = i % N;
        const int v = red[row * NP + col];
        if (v != 0 && k0 + row < K) atomicAdd(acc_out + (long long)(k0 + row) * N + col, v);
    }
    if (tail.f_out == nullptr) return;
    // the last CTA to get here turns the sums into floats
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(tail.counter, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int i = threadIdx.x; i < K * N; i += kDwWarps * 32) {
        const float v = __fmul_rn((float)__ldcg(acc_out + i), tail.scale);
        tail.f_out[i] = tail.accumulate ? __fadd_rn(tail.f_out[i], v) : v;
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

template <int N, int MT, bool A_UNSIGNED>
int launch_dw_t(const unsigned char *a, long long lda, const signed char *g, long long ldg, int M, int K, int32_t *acc,
                const DwTail &tail, cudaStream_t stream)
{
    using Geo = DwGeom<N, MT>;
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    const int S = (K + Geo::KSL - 1) / Geo::KSL;                 // column slices of A
    if (S > sms) return CDL_ERR_ARG;
    if (cudaFuncSetAttribute(skinny_dw_kernel<N, MT, A_UNSIGNED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Geo::smem_bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    const long long ngroups = ((long long)M + 31) / 32;
    long long per_slice = sms / S;                               // CTAs that share a slice: one CTA per SM in all
    const long long useful = (ngroups + kDwWarps - 1) / kDwWarps;
    if (per_slice > useful) per_slice = useful;
    const int grid = (int)(per_slice * S);
    skinny_dw_kernel<N, MT, A_UNSIGNED><<<grid, kDwWarps * 32, Geo::smem_bytes, stream>>>(a, lda, g, ldg, M, K, S, acc, tail);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

template <int N, int MT>
int launch_dw_n(const void *A, long long lda, bool a_unsigned, const void *G, long long ldg, int M, int K, int32_t *acc,
                const DwTail &tail, cudaStream_t stream)
{
    const unsigned char *a = static_cast<const unsigned char *>(A);
    const signed char *g = static_cast<const signed char *>(G);
    return a_unsigned ? launch_dw_t<N, MT, true>(a, lda, g, ldg, M, K, acc, tail, stream)
                      : launch_dw_t<N, MT, false>(a, lda, g, ldg, M, K, acc, tail, stream);
}

bool skinny_dw_ok(int M, int N, int K)
{
    (void)M;
    return (N == 4 || N == 8 || N == 16 || N == 32) && (K % 4) == 0 && K <= 2048;
}

size_t skinny_dw_scratch_bytes(int N, int K) { return ((size_t)K * N + 4) * sizeof(int32_t); }

// dW (K x N floats and / or int32) from A (M x K bytes) and G (M x N int8); scratch: skinny_dw_scratch_bytes
int launch_skinny_dw(const void *A, long long lda, bool a_unsigned, const void *G, long long ldg, int M, int N, int K,
                     int32_t *acc_out, float *f_out, float scale, bool accumulate, void *scratch, cudaStream_t stream)
{
    if (scratch == nullptr) return CDL_ERR_WORKSPACE;
    int32_t *sums = static_cast<int32_t *>(scratch);
    DwTail tail{f_out, scale, accumulate ? 1 : 0, reinterpret_cast<unsigned int *>(sums + (size_t)K * N)};
    int32_t *acc = acc_out != nullptr ? acc_out : sums;
    // the sums and the CTA counter behind them start at zero
    const size_t nsum = (size_t)K * N * sizeof(int32_t);
    cudaError_t e;
    if (acc_out == nullptr) {
        e = cudaMemsetAsync(sums, 0, nsum + 4 * sizeof(int32_t), stream);
    } else {
        e = cudaMemsetAsync(acc_out, 0, nsum, stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(tail.counter, 0, 4 * sizeof(int32_t), stream);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    switch (N) {
        case 4: return launch_dw_n<4, 9>(A, lda, a_unsigned, G, ldg, M, K, acc, tail, stream);
        case 8: return launch_dw_n<8, 9>(A, lda, a_unsigned, G, ldg, M, K, acc, tail, stream);
        case 16: return launch_dw_n<16, 9>(A, lda, a_unsigned, G, ldg, M, K, acc, tail, stream);
        case 32: return launch_dw_n<32, 4>(A, lda, a_unsigned, G, ldg, M, K, acc, tail, stream);
        default: return CDL_ERR_ARG;
    }
}

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
