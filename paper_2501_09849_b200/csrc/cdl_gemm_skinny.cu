// Layer products whose weight matrix has few output channels (N <= 32: the 16-channel layers of CIFAR ResNets).
// With K * N of a few thousand there are only ~10 multiply-adds per byte moved, so these products are bound by
// HBM, not by arithmetic, and a 128-row tile fed by TMA spends its time on hand-shakes: here they are streaming
// kernels in which every warp works alone, rows go from global memory straight into the fragments of the
// warp-level int8 matrix instruction (m16n8k32), exact in int32 like the tile path and with the same float epilogue.
//   forward  Y[m, :]  = A[m, :] W        a warp per 16 rows, W fragments in shared memory
//   dX       dA[m, :] = G[m, :] W^T      a warp per 16 rows, 16-byte stores; a dp4a kernel (lane = output column)
//                                        covers K that is not a multiple of 16
//   dW       dW       = A^T G            a warp per 32 rows, operands transposed in registers
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

// ------------------------------------------------------------------------------------------------ forward
// A warp takes 16 rows at a time: lane (g, t) = (lane / 4, lane % 4) reads 16 consecutive bytes of rows g and g + 8
// per 64 columns, which are the A fragments of two m16n8k32 steps once the k positions of a step are taken in the
// order the loads deliver them; the fragments of W are laid out in shared memory for the same order.  Output columns
// are dealt to the 8-column tiles so that a lane ends up with 2 N / 8 consecutive columns of a row (one or two
// 16-byte stores; a quad writes the whole row).  K a multiple of 16: after the 64-column chunks one 32- and / or one
// 16-column piece (8- and 4-byte loads).
__device__ __forceinline__ int fwd_kbase(int s, int t, int h, int c64, int rest)
{
    if (s < 2 * c64) return 64 * (s >> 1) + 16 * t + 8 * (s & 1) + 4 * h;
    const int base = 64 * c64, r = s - 2 * c64;
    if (rest >= 32 && r == 0) return base + 8 * t + 4 * h;
    return h == 0 ? base + (rest >= 32 ? 32 : 0) + 4 * t : -1;     // the 16-column tail: upper half of the step empty
}

template <int N, bool A_UNSIGNED>
__global__ void __launch_bounds__(kSkinnyThreads)
skinny_fwd_kernel(const unsigned char *__restrict__ A, long long lda, const signed char *__restrict__ W, long long ldw,
                  int M, int K, int32_t *__restrict__ acc_out, float *__restrict__ y_out, float scale,
                  const float *__restrict__ bias)
{
    constexpr int NT = N >= 8 ? N / 8 : 1;
    extern __shared__ __align__(16) unsigned int Bf[];          // [step][tile][half][lane]
    const int c64 = K >> 6, rest = K & 63;
    const int nsteps = 2 * c64 + (rest >= 32 ? 1 : 0) + ((rest & 31) == 16 ? 1 : 0);
    for (int i = threadIdx.x; i < nsteps * NT * 64; i += kSkinnyThreads) {
        const int ln = i & 31, h = (i >> 5) & 1, sj = i >> 6, j = sj % NT, s = sj / NT;
        const int kb = fwd_kbase(s, ln & 3, h, c64, rest);
        const int gg = ln >> 2;
        const int col = N >= 8 ? (gg >> 1) * (2 * NT) + 2 * j + (gg & 1) : gg;
        unsigned int w = 0;
        if (kb >= 0 && col < N) {
#pragma unroll
            for (int b = 0; b < 4; ++b) w |= (unsigned int)(unsigned char)W[(long long)(kb + b) * ldw + col] << (8 * b);
        }
        Bf[i] = w;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, t = lane & 3, g = lane >> 2;
    const long long warp = ((long long)blockIdx.x * kSkinnyThreads + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * kSkinnyThreads) >> 5;
    const long long ntiles = ((long long)M + 15) / 16;
    const int cb = N >= 8 ? t * 2 * NT : 2 * t;                 // this lane's first output column
    float bv[2 * NT];
#pragma unroll
    for (int q = 0; q < 2 * NT; ++q) bv[q] = (bias != nullptr && cb + q < N) ? bias[cb + q] : 0.0f;
    for (long long tile = warp; tile < ntiles; tile += nwarps) {
        __syncwarp();                                           // the matrix instruction wants the whole warp
        const long long r0 = tile * 16 + g, r1 = r0 + 8;
        const bool v0 = r0 < M, v1 = r1 < M;
        const unsigned char *p0 = A + r0 * lda, *p1 = A + r1 * lda;
        int acc[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[j][c] = 0;
        const unsigned int *bf = Bf + lane;
#pragma unroll 2
        for (int c = 0; c < c64; ++c) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            const uint4 x0 = v0 ? __ldcs(reinterpret_cast<const uint4 *>(p0 + 64 * c + 16 * t)) : z;
            const uint4 x1 = v1 ? __ldcs(reinterpret_cast<const uint4 *>(p1 + 64 * c + 16 * t)) : z;
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_k32<A_UNSIGNED>(acc[j], x0.x, x1.x, x0.y, x1.y, bf[j * 64], bf[j * 64 + 32]);
            bf += NT * 64;
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_k32<A_UNSIGNED>(acc[j], x0.z, x1.z, x0.w, x1.w, bf[j * 64], bf[j * 64 + 32]);
            bf += NT * 64;
        }
        int kb = 64 * c64;
        if (rest >= 32) {
            const uint2 z = make_uint2(0u, 0u);
            const uint2 x0 = v0 ? __ldcs(reinterpret_cast<const uint2 *>(p0 + kb + 8 * t)) : z;
            const uint2 x1 = v1 ? __ldcs(reinterpret_cast<const uint2 *>(p1 + kb + 8 * t)) : z;
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_k32<A_UNSIGNED>(acc[j], x0.x, x1.x, x0.y, x1.y, bf[j * 64], bf[j * 64 + 32]);
            bf += NT * 64;
            kb += 32;
        }
        if ((rest & 31) == 16) {
            const unsigned int x0 = v0 ? __ldcs(reinterpret_cast<const unsigned int *>(p0 + kb + 4 * t)) : 0u;
            const unsigned int x1 = v1 ? __ldcs(reinterpret_cast<const unsigned int *>(p1 + kb + 4 * t)) : 0u;
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_k32<A_UNSIGNED>(acc[j], x0, x1, 0u, 0u, bf[j * 64], 0u);
        }
        if (N == 4 && t >= 2) continue;                         // columns 4 .. 7 of the only tile do not exist
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const long long r = half == 0 ? r0 : r1;
            if (r >= M) continue;
            int v[2 * NT];
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                v[2 * j] = acc[j][2 * half];
                v[2 * j + 1] = acc[j][2 * half + 1];
            }
            if (acc_out != nullptr) {
                int *o = acc_out + r * N + cb;
                if constexpr (2 * NT >= 4) {
#pragma unroll
                    for (int q = 0; q < 2 * NT; q += 4) *reinterpret_cast<int4 *>(o + q) = make_int4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                } else {
                    *reinterpret_cast<int2 *>(o) = make_int2(v[0], v[1]);
                }
            }
            if (y_out != nullptr) {
                float f[2 * NT];
#pragma unroll
                for (int q = 0; q < 2 * NT; ++q) {
                    f[q] = __fmul_rn((float)v[q], scale);
                    if (bias != nullptr) f[q] = __fadd_rn(f[q], bv[q]);
                }
                float *o = y_out + r * N + cb;
                if constexpr (2 * NT >= 4) {
#pragma unroll
                    for (int q = 0; q < 2 * NT; q += 4) __stcs(reinterpret_cast<float4 *>(o + q), make_float4(f[q], f[q + 1], f[q + 2], f[q + 3]));
                } else {
                    __stcs(reinterpret_cast<float2 *>(o), make_float2(f[0], f[1]));
                }
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

// dX on the matrix instruction (K a multiple of 16): a warp takes 16 rows, its G fragment is one 4- or 8-byte load
// per row, and every pair of 8-column tiles of the output is two instructions whose results a lane stores as 16
// consecutive bytes per row (columns dealt to the tiles so that a quad writes 64 consecutive bytes).
template <int N>
__global__ void __launch_bounds__(kSkinnyThreads)
skinny_dx_mma_kernel(const signed char *__restrict__ G, long long ldg, const signed char *__restrict__ W, long long ldw,
                     int M, int K, int32_t *__restrict__ acc_out, float *__restrict__ f_out, float scale, int accumulate)
{
    constexpr int NH = N == 32 ? 2 : 1;                         // words per lane of a W fragment
    extern __shared__ __align__(16) unsigned int Bf[];          // [tile][half][lane]
    const int ntile = K / 8;
    for (int i = threadIdx.x; i < ntile * NH * 32; i += kSkinnyThreads) {
        const int ln = i & 31, h = NH == 2 ? (i >> 5) & 1 : 0, j = i / (32 * NH);
        const int tt = ln & 3, gg = ln >> 2;
        const int kc = 16 * (j >> 1) + 4 * (gg >> 1) + 2 * (j & 1) + (gg & 1);      // the output column behind (tile, gg)
        const int nb = N == 32 ? 8 * tt + 4 * h : 4 * tt;
        Bf[i] = nb < N ? *reinterpret_cast<const unsigned int *>(W + (long long)kc * ldw + nb) : 0u;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, t = lane & 3, g = lane >> 2;
    const long long warp = ((long long)blockIdx.x * kSkinnyThreads + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * kSkinnyThreads) >> 5;
    const long long ntiles = ((long long)M + 15) / 16;
    for (long long tile = warp; tile < ntiles; tile += nwarps) {
        __syncwarp();                                           // the matrix instruction wants the whole warp
        const long long r0 = tile * 16 + g, r1 = r0 + 8;
        const bool v0 = r0 < M, v1 = r1 < M;
        unsigned int a0 = 0u, a1 = 0u, a2 = 0u, a3 = 0u;
        if (N == 32) {
            if (v0) { const uint2 x = *reinterpret_cast<const uint2 *>(G + r0 * ldg + 8 * t); a0 = x.x; a2 = x.y; }
            if (v1) { const uint2 x = *reinterpret_cast<const uint2 *>(G + r1 * ldg + 8 * t); a1 = x.x; a3 = x.y; }
        } else if (4 * t < N) {
            if (v0) a0 = *reinterpret_cast<const unsigned int *>(G + r0 * ldg + 4 * t);
            if (v1) a1 = *reinterpret_cast<const unsigned int *>(G + r1 * ldg + 4 * t);
        }
        const unsigned int *bf = Bf + lane;
        for (int p = 0; p < K / 16; ++p, bf += 2 * NH * 32) {
            int d0[4] = {0, 0, 0, 0}, d1[4] = {0, 0, 0, 0};
            mma_k32<false>(d0, a0, a1, a2, a3, bf[0], NH == 2 ? bf[32] : 0u);
            mma_k32<false>(d1, a0, a1, a2, a3, bf[NH * 32], NH == 2 ? bf[NH * 32 + 32] : 0u);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const long long r = half == 0 ? r0 : r1;
                if (r >= M) continue;
                const long long o = r * K + 16 * p + 4 * t;
                const int v[4] = {d0[2 * half], d0[2 * half + 1], d1[2 * half], d1[2 * half + 1]};
                if (acc_out != nullptr) *reinterpret_cast<int4 *>(acc_out + o) = make_int4(v[0], v[1], v[2], v[3]);
                if (f_out != nullptr) {
                    float4 f = make_float4(__fmul_rn((float)v[0], scale), __fmul_rn((float)v[1], scale),
                                           __fmul_rn((float)v[2], scale), __fmul_rn((float)v[3], scale));
                    float4 *fo = reinterpret_cast<float4 *>(f_out + o);
                    if (accumulate) {
                        const float4 c = *fo;
                        *fo = make_float4(__fadd_rn(c.x, f.x), __fadd_rn(c.y, f.y), __fadd_rn(c.z, f.z), __fadd_rn(c.w, f.w));
                    } else {
                        __stcs(fo, f);
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

template <int N, bool A_UNSIGNED>
int launch_fwd_t(const unsigned char *a, long long lda, const signed char *w, long long ldw, int M, int K, int32_t *acc_out,
                 float *y_out, float scale, const float *bias, cudaStream_t stream)
{
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    constexpr int NT = N >= 8 ? N / 8 : 1;
    const int rest = K & 63;
    const int nsteps = 2 * (K >> 6) + (rest >= 32 ? 1 : 0) + ((rest & 31) == 16 ? 1 : 0);
    const size_t smem = (size_t)nsteps * NT * 64 * sizeof(unsigned int);
    auto kern = skinny_fwd_kernel<N, A_UNSIGNED>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    const long long need = (((long long)M + 15) / 16 + kSkinnyThreads / 32 - 1) / (kSkinnyThreads / 32);
    const int grid = (int)(need < 4ll * sms ? need : 4ll * sms);
    kern<<<grid, kSkinnyThreads, smem, stream>>>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

template <int N>
int launch_fwd_n(const void *A, long long lda, bool a_unsigned, const void *W, long long ldw, int M, int K,
                 int32_t *acc_out, float *y_out, float scale, const float *bias, cudaStream_t stream)
{
    const unsigned char *a = static_cast<const unsigned char *>(A);
    const signed char *w = static_cast<const signed char *>(W);
    return a_unsigned ? launch_fwd_t<N, true>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream)
                      : launch_fwd_t<N, false>(a, lda, w, ldw, M, K, acc_out, y_out, scale, bias, stream);
}

template <int N>
int launch_dx_mma(const void *G, long long ldg, const void *W, long long ldw, int M, int K, int32_t *acc_out, float *f_out,
                  float scale, bool accumulate, cudaStream_t stream)
{
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    const size_t smem = (size_t)(K / 8) * (N == 32 ? 2 : 1) * 32 * sizeof(unsigned int);
    auto kern = skinny_dx_mma_kernel<N>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    const long long need = (((long long)M + 15) / 16 + kSkinnyThreads / 32 - 1) / (kSkinnyThreads / 32);
    const int grid = (int)(need < 6ll * sms ? need : 6ll * sms);
    kern<<<grid, kSkinnyThreads, smem, stream>>>(static_cast<const signed char *>(G), ldg, static_cast<const signed char *>(W),
                                                 ldw, M, K, acc_out, f_out, scale, accumulate ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
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
    return (N == 4 || N == 8 || N == 16 || N == 32) && (K % 16) == 0 && (long long)K * (N < 8 ? 8 : N) <= 96 * 1024;
}

bool skinny_dx_ok(int M, int N, int K)
{
    (void)M;
    (void)K;
    return N == 4 || N == 8 || N == 16 || N == 32;
}

// Y (M x N floats and / or int32) = A (M x K bytes) W (K x N int8); outputs 16-byte aligned
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

// dX (M x K) = G (M x N int8) W^T (W: K x N int8): the matrix-instruction kernel when K is a multiple of 16, its
// fragment table fits and the outputs are 16-byte aligned, else the dp4a kernel
int launch_skinny_dx(const void *G, long long ldg, const void *W, long long ldw, int M, int N, int K, int32_t *acc_out,
                     float *f_out, float scale, bool accumulate, cudaStream_t stream)
{
    const bool aligned = ((reinterpret_cast<uintptr_t>(acc_out) | reinterpret_cast<uintptr_t>(f_out)) & 15u) == 0;
    if ((K % 16) == 0 && aligned && (long long)(K / 8) * (N == 32 ? 2 : 1) * 128 <= 96 * 1024) {
        switch (N) {
            case 4: return launch_dx_mma<4>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
            case 8: return launch_dx_mma<8>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
            case 16: return launch_dx_mma<16>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
            case 32: return launch_dx_mma<32>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
            default: return CDL_ERR_ARG;
        }
    }
    switch (N) {
        case 4: return launch_dx_nw<1>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 8: return launch_dx_nw<2>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 16: return launch_dx_nw<4>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        case 32: return launch_dx_nw<8>(G, ldg, W, ldw, M, K, acc_out, f_out, scale, accumulate, stream);
        default: return CDL_ERR_ARG;
    }
}

}  // namespace cdl
