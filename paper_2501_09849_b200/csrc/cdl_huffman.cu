// Huffman code lengths of a level histogram (Sec. VI-B: the average number of bits per weight / activation is
// measured by Huffman-coding the indices).  One CTA: the used levels are ranked by count in parallel, one thread
// builds the tree with the two-queue construction (leaves in ascending order, merged nodes are created in
// ascending order too, so the two lightest subtrees are always at the heads of the two queues), depths are read
// off the parent links, and the total Σ count × length is reduced by the CTA.  At most 256 levels: microseconds,
// off the per-step path (the paper codes the tensors once per epoch).
#include "cdl_internal.h"

namespace cdl {
namespace {

constexpr int kHT = 256;

__global__ void __launch_bounds__(kHT, 1)
huffman_kernel(const unsigned long long *__restrict__ hist, int nlev, unsigned char *__restrict__ lengths,
               unsigned long long *__restrict__ total_bits, double *__restrict__ avg_bits)
{
    __shared__ unsigned long long cnt[kHT];          // count of level k
    __shared__ unsigned long long wt[2 * kHT];       // weight of tree node (leaves first, ascending)
    __shared__ unsigned short parent[2 * kHT];
    __shared__ unsigned short depth[2 * kHT];
    __shared__ unsigned long long red[kHT / 32];
    __shared__ unsigned long long red_n[kHT / 32];
    __shared__ int m_s;
    const int k = threadIdx.x;
    cnt[k] = k < nlev ? hist[k] : 0ull;
    __syncthreads();
    const unsigned long long c = cnt[k];
    // rank among the used levels: by count, then by level
    int rank = 0, used = 0;
    for (int j = 0; j < nlev; ++j) {
        const unsigned long long cj = cnt[j];
        used += cj > 0ull;
        rank += (cj > 0ull) && (cj < c || (cj == c && j < k));
    }
    if (k == 0) m_s = used;
    if (c > 0ull) wt[rank] = c;                      // leaf `rank` is level k
    __syncthreads();
    const int m = m_s;
    if (k == 0 && m > 1) {
        int leaf = 0, inner = m, made = m;          // heads of the two queues, next node to create
        for (int step = 0; step < m - 1; ++step) {
            unsigned long long w = 0ull;
            for (int pick = 0; pick < 2; ++pick) {
                // the lighter head; a leaf wins a tie (keeps the tree shallow)
                const bool take_leaf = leaf < m && (inner >= made || wt[leaf] <= wt[inner]);
                const int node = take_leaf ? leaf++ : inner++;
                w += wt[node];
                parent[node] = (unsigned short)made;
            }
            wt[made++] = w;
        }
        depth[made - 1] = 0;                          // the root; every parent has a larger number than its children
        for (int node = made - 2; node >= 0; --node) depth[node] = (unsigned short)(depth[parent[node]] + 1);
    }
    __syncthreads();
    // lengths and totals
    unsigned long long bits = 0ull;
    if (k < nlev) {
        int len = 0;
        if (c > 0ull) len = m > 1 ? (int)depth[rank] : 1;     // a single used level still costs one bit per index
        if (lengths != nullptr) lengths[k] = (unsigned char)len;
        bits = c * (unsigned long long)len;
    }
    unsigned long long n = c;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        bits += __shfl_down_sync(0xffffffffu, bits, off);
        n += __shfl_down_sync(0xffffffffu, n, off);
    }
    if ((k & 31) == 0) {
        red[k >> 5] = bits;
        red_n[k >> 5] = n;
    }
    __syncthreads();
    if (k == 0) {
        unsigned long long tb = 0ull, tn = 0ull;
        for (int w = 0; w < kHT / 32; ++w) {
            tb += red[w];
            tn += red_n[w];
        }
        if (total_bits != nullptr) *total_bits = tb;
        if (avg_bits != nullptr) *avg_bits = tn > 0ull ? (double)tb / (double)tn : 0.0;
    }
}

}  // namespace

int launch_huffman(const unsigned long long *hist, int nlev, unsigned char *lengths, unsigned long long *total_bits,
                   double *avg_bits, cudaStream_t stream)
{
    huffman_kernel<<<1, kHT, 0, stream>>>(hist, nlev, lengths, total_bits, avg_bits);
    return cudaGetLastError() == cudaSuccess ? CDL_OK : CDL_ERR_LAUNCH;
}

}  // namespace cdl
