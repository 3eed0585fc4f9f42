// Index GEMM on the 5th-generation tensor cores of sm_100a: D[i,j] = sum_r X(i,r) Y(r,j) over int8/uint8
// index bytes, exact int32 accumulation (tcgen05.mma kind::i8, accumulator in TMEM), operands staged in
// shared memory by TMA (no multicast), float / int32 epilogue read back with tcgen05.ld.
//
// One kernel serves the three layer products; they differ only in which dimension of each stored matrix is
// contiguous, which is expressed by the "major" of the shared-memory operand descriptor:
//   forward  Y  = A W      X = A [M,K] (r = k contiguous: K-major)   Y-op = W [K,N] (j contiguous: MN-major)
//   dX       dA = G W^T    X = G [M,N] (r = n contiguous: K-major)   Y-op = W [K,N] (r = n contiguous: K-major)
//   dW       dW = A^T G    X = A [M,K] (i = k contiguous: MN-major)  Y-op = G [M,N] (j contiguous: MN-major)
//
// In convolution form the X operand is not a stored matrix: its tiles are gathered from an NHWC index tensor by
// TMA im2col loads (patch matrix of a convolution, or its transpose for dW), see ConvGather.  The kind of X operand
// is a template argument (the producers' stage loop tests nothing about it).
//
// Tiling: 128 x TN output tile per work unit (TN in {16..256}), a 256 x TN tile of one CTA when TN <= 128
// (256 rows of X per stage, two accumulators sharing the Y block: a narrow product gets twice the rows out of every
// pipeline stage), or a 256 x 256 tile shared by a pair of CTAs (tcgen05 cta_group::2) when the output is wide and
// tall enough; 128 bytes of the reduced dimension per pipeline stage, four tcgen05.mma (K = 32 each) per stage.
// Every shared-memory operand block is [rows][128 bytes] with the 128-byte swizzle, written by TMA boxes whose inner
// extent is 128 bytes; rows or columns outside the matrix are zero-filled by TMA, which makes ragged edges and R
// tails exact.  A convolution with 64 channels per filter tap would fill only half of such rows: its gathered
// blocks are 64 bytes wide under the 64-byte swizzle instead (K-major rows of 64 bytes and two MMAs per stage for
// forward and dX; MN-major boxes of 64 channels, two per 128 tile rows, for dW).
// Warp roles: warp 0 and the last warp issue TMA (X and Y operand), warp 1 owns TMEM and issues the MMAs, the
// 8 (or, for products that store more than they load, 16) warps between them run the epilogue; two TMEM
// accumulators let the epilogue of one tile overlap the MMAs of the next.
// Epilogue: each thread owns one output row in TMEM; 32 columns at a time are converted, written to the warp's
// swizzled 32 x 128-byte staging block in shared memory and handed to TMA (bulk tensor store), so that global
// memory sees whole 128-byte lines.  The per-chunk chain (TMEM load, convert, stage, proxy fence, store) is a
// string of latencies, so two warps share each TMEM lane quarter and take alternate chunks.  Work units are
// (tile, split of the reduced dimension); with more than one split every split stores its partial tile into a
// slab of its own and a small kernel sums the slabs in int64 (or, when the caller wants the int32 accumulators
// or scratch is tight, the staging blocks are added into one buffer with TMA bulk reduce-adds: integers, so the
// result does not depend on order).  Outputs whose pitch or base is not 16-byte aligned, and tiles 16 columns
// wide, go through the same staging block and are copied out by the warps one row at a time.  Optional extras
// of the epilogue: bias, the next layer's hard index, adding to the float output instead of storing it.
// Every wait is bounded: on expiry the kernel records CDL_ERR_TIMEOUT in the status word and winds down.
#include <cuda.h>

#include <atomic>
#include <string.h>

#include "cdl_internal.h"
#include "cdl_wait.cuh"

namespace cdl {
namespace {

// Epilogue warps per CTA: kEpiWarps / 4 per TMEM lane quarter, taking the 32-column chunks in turn.  Products whose
// time is the epilogue's (two stages of loads per 256 KB of output) get twice as many, with one chunk in flight each.
__host__ __device__ constexpr int epi_warps(bool store_heavy) { return store_heavy ? 16 : 8; }
constexpr bool kSplitProducer = true;   // a second TMA warp issues the Y-operand loads
__host__ __device__ constexpr int threads_tc(bool store_heavy) { return 64 + 32 * epi_warps(store_heavy) + (kSplitProducer ? 32 : 0); }
// Shared memory is divided between operand stages and epilogue staging blocks (4 KB each, per epilogue warp).
// Which of the two needs the bytes in flight depends on the shape: a long reduced dimension loads much more than
// it stores, a short one (two stages per 128 KB of output) the opposite.
//                                          load-heavy                     store-heavy
//   one CTA per tile  (48 KB stages)       4 stages, 8 epilogue warps     3 stages, 16 epilogue warps
//   CTA pair per tile (32 KB stages)       6 stages, 8 epilogue warps     4 stages, 16 epilogue warps
constexpr int kStagesMax = 6;
constexpr int TM = 128;                 // output rows per tile = UMMA M
constexpr int BR = 128;                 // bytes (= elements) of the reduced dimension per stage
constexpr int kABytes = TM * BR;        // 16 KB
constexpr int kBBytesMax = 256 * BR;    // 32 KB
constexpr int kStageBytesSingle = kABytes + kBBytesMax;
constexpr int kStageBytesPair = kABytes + 128 * BR;
constexpr int kOutWarpBytes = 32 * 128;  // epilogue staging block of one warp: 32 rows x 32 four-byte columns
// The whole 227 KB opt-in window is requested (stages need 193 KB): operand descriptors then address
// allocated shared memory for any stride a 128 x 256 x 128 tile can produce.
constexpr int kSmemBytes = 232448 - 1024;
constexpr int kMaxTaps = kConvMaxTaps;   // filter taps of a gathered patch matrix (7 x 7 fits)
constexpr int kPlanSMs = 148;           // B200: splits are planned for this count so that workspace sizes are fixed
constexpr unsigned long long kWaitNs = 2000000000ull;  // limit of every device-side wait: 2 s

struct TcParams {
    int I, J, R;            // rows the tiling runs over, output columns, reduced extent of the tiling
    int I_out;              // rows of the output matrix (differs from I only for a padded transposed patch matrix)
    int TN;                 // output columns per tile (multiple of 16, <= 256)
    int tiles_i, tiles_j;   // tile grid
    int splits;             // splits of the reduced dimension
    int rblocks;            // ceil(R / BR)
    int a_mn_major, b_mn_major;
    unsigned int idesc;
    int32_t *acc_out;       // int32 output or accumulation buffer (required when splits > 1)
    float *f_out;           // float output (written by the epilogue only when splits == 1)
    float scale;
    int f_acc;              // 1: the float output is added to what f_out holds (one binary32 addition per element)
    const float *bias;
    int *status;
    unsigned long long wait_ns;   // limit of each mbarrier wait
    int tma_f, tma_acc;     // the float / int32 output goes through shared memory and TMA
    // Implicit patch matrix (convolution): the X operand is gathered by TMA im2col loads from an [N,H,W,C] index
    // tensor instead of being read from a stored matrix.
    int conv;               // 0: stored matrix; 1: X(i = pixel, r = tap * C + c); 2: X(i = tap * C + c, r = pixel)
    int cH, cW, cC;         // base pixels per image column and row (the gather's output grid), channels
    int cblocks;            // 128-channel blocks per tap (C rounded up to 128: channels past C read as zero)
    int cpad;               // 128 * cblocks
    int pad_h, pad_w;       // the base pixel of grid position (p, q) sits at (p * c_stride - pad_h, q * c_stride - pad_w)
    int c_stride;
    int taps;
    int y_tap_rows;         // > 0: the Y block of tap t starts at row tap_y[t] * y_tap_rows of the stored matrix
    signed char tap_oh[kMaxTaps], tap_ow[kMaxTaps];   // offset of each tap from the base pixel
    unsigned char tap_y[kMaxTaps];
    // Scattered output rows (data gradient of a strided convolution, one residue class of pixels per launch): row i
    // of the product is position (n, p, q) of an sc_P x sc_Q grid per image and is stored as pixel
    // (n, sc_s p + sc_a, sc_s q + sc_b) of an sc_H x sc_W image.
    int sc_on, sc_P, sc_Q, sc_H, sc_W, sc_s, sc_a, sc_b;
    int copy_vec;           // outputs copied out by the warps may be written 16 bytes at a time (J % 4 == 0, aligned bases)
    // next layer's hard index from the float output (forward products, single split)
    unsigned char *nq_out;  // nullptr: not requested
    float nq_q, nq_rq, nq_flo, nq_fhi;
    int nq_fast, nq_vec;    // reciprocal product allowed; rows can be written 16 bytes at a time
    int slab_rows;          // 0: splits add into one I x J buffer.  > 0: split s stores its partial tile into rows
                            // [s * slab_rows, ...) of a (splits * slab_rows) x J buffer, summed in int64 afterwards
    int slots;              // work slots (CTA pairs, or CTAs) = the grid: slot p takes units p, p + slots, ...
    int tall;               // 1: a CTA's tile is 256 rows x TN (TN <= 128): one 256-row X box per stage, two accumulators
    int k64;                // 1: forward-type gather of 64 channels per tap: X rows are 64 bytes (64-byte swizzle), two MMAs per stage
    int k64t;               // 1: transposed gather of 64 channels per tap: 64 tile rows per tap (no padding to 128), X boxes of
                            //    64 channels x 128 pixels under the 64-byte swizzle, two per 128 tile rows
};

// One piece of work of a slot: pipeline stages [rb0, rb1) of a tile (a unit of tiles * splits).
struct WorkItem {
    int valid;
    int tile, split, rb0, rb1;
};

// The units of a slot, in order.  The threads that walk them are single lanes on the critical path of the pipeline
// (TMA producers, MMA issuer), and a product with a short reduced dimension has thousands of units of two or three
// stages each: stepping to the next unit is an addition, with divisions only when the reduced dimension is split
// (then a slot has few units).
struct SlotWork {
    long long units, u;
    int slots, rblocks, splits;
};

__device__ __forceinline__ SlotWork slot_work(const TcParams &P, int p)
{
    SlotWork s;
    s.units = (long long)P.tiles_i * P.tiles_j * P.splits;
    s.u = p;
    s.slots = P.slots;
    s.rblocks = P.rblocks;
    s.splits = P.splits;
    return s;
}

__device__ __forceinline__ WorkItem next_item(SlotWork &s)
{
    WorkItem w;
    w.valid = s.u < s.units;
    if (s.splits == 1) {
        w.tile = (int)s.u;
        w.split = 0;
        w.rb0 = 0;
        w.rb1 = s.rblocks;
    } else {
        const unsigned int u32 = (unsigned int)s.u, sp = (unsigned int)s.splits;      // units < 2^31 (checked by the launcher)
        const unsigned int tile = u32 / sp, split = u32 - tile * sp;
        w.tile = (int)tile;
        w.split = (int)split;
        w.rb0 = (int)(((long long)s.rblocks * split) / sp);
        w.rb1 = (int)(((long long)s.rblocks * (split + 1u)) / sp);
    }
    s.u += s.slots;
    return w;
}

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// im2col load: 128 consecutive pixels (w fastest, then h, then n) x 128 channel bytes starting at pixel (w, h, n)
// shifted by the filter tap (off_w, off_h); positions outside the tensor read as zero
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap *map, int c, int w, int h, int n,
                                                int off_w, int off_h, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"((unsigned short)off_w), "h"((unsigned short)off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_im2col_pair(uint32_t dst, const CUtensorMap *map, int c, int w, int h, int n,
                                                     int off_w, int off_h, uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .b32 rb;\n\t"
        "mapa.shared::cluster.u32 rb, %6, 0;\n\t"
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3, %4, %5}], [rb], {%7, %8};\n\t}"
        ::"r"(dst), "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"((unsigned short)off_w), "h"((unsigned short)off_h)
        : "memory");
}

// Load issued by either CTA of a pair into its own shared memory; the bytes are counted on the barrier at offset
// `bar` of CTA 0 (no multicast: each CTA fetches its own box).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .b32 rb;\n\t"
        "mapa.shared::cluster.u32 rb, %4, 0;\n\t"
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3}], [rb];\n\t}"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int c0, int c1, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, int c0, int c1, uint32_t src)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// AND over the epilogue threads (named barrier 1)
template <int THREADS>
__device__ __forceinline__ bool epi_all(bool v)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)v), "n"(THREADS)
        : "memory");
    return out != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- CTA-pair helpers (cluster of two CTAs, cta_group::2)
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank)
{
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(rank)
        : "memory");
}
// both CTAs of the pair get the arrival (same barrier offset in each)
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// The four MMAs (K = 32 each) of one 128-byte stage in one go: descriptor k is (lo + k * step, hi); the first one
// accumulates only when `accumulate` is set, the others always.
template <bool PAIR>
__device__ __forceinline__ void tc_mma4_i8(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t a_step, uint32_t b_lo,
                                           uint32_t b_hi, uint32_t b_step, uint32_t idesc, uint32_t accumulate)
{
    if (PAIR) {
        asm volatile(
            "{\n\t.reg .pred p, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
            "setp.ne.b32 p, %8, 0;\n\t"
            "setp.eq.b32 t, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%4, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, p;\n\t"
            "add.u32 al, %1, %3;\n\tadd.u32 bl, %4, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, t;\n\t"
            "add.u32 al, al, %3;\n\tadd.u32 bl, bl, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, t;\n\t"
            "add.u32 al, al, %3;\n\tadd.u32 bl, bl, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, t;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
            "setp.ne.b32 p, %8, 0;\n\t"
            "setp.eq.b32 t, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%4, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, p;\n\t"
            "add.u32 al, %1, %3;\n\tadd.u32 bl, %4, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, t;\n\t"
            "add.u32 al, al, %3;\n\tadd.u32 bl, bl, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, t;\n\t"
            "add.u32 al, al, %3;\n\tadd.u32 bl, bl, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, t;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
    }
}

// Two MMAs (K = 32 each) of a stage that holds 64 bytes of r.
template <bool PAIR>
__device__ __forceinline__ void tc_mma2_i8(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t a_step, uint32_t b_lo,
                                           uint32_t b_hi, uint32_t b_step, uint32_t idesc, uint32_t accumulate)
{
    if (PAIR) {
        asm volatile(
            "{\n\t.reg .pred p, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
            "setp.ne.b32 p, %8, 0;\n\t"
            "setp.eq.b32 t, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%4, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, p;\n\t"
            "add.u32 al, %1, %3;\n\tadd.u32 bl, %4, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9, %9, %9, %9, %9}, t;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
            "setp.ne.b32 p, %8, 0;\n\t"
            "setp.eq.b32 t, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%4, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, p;\n\t"
            "add.u32 al, %1, %3;\n\tadd.u32 bl, %4, %6;\n\t"
            "mov.b64 da, {al, %2};\n\tmov.b64 db, {bl, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %7, {%9, %9, %9, %9}, t;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
    }
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
// Wait for the TMEM loads in flight and tie the loaded registers to the wait, so that no use of them is scheduled
// ahead of it.
__device__ __forceinline__ void tc_wait_ld_pin(uint32_t (&v)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :
                 : "memory");
    asm volatile(""
                 : "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                   "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :
                 : "memory");
}

// Shared-memory operand descriptor (sm_100 format): start address, leading / stride byte offsets in 16-byte
// units, version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version for sm_100
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}

// The same for a K-major block whose rows are 64 bytes (64-byte swizzle): 8-row groups sbo_bytes = 512 apart.
__device__ __forceinline__ uint64_t make_desc64(uint32_t saddr, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;       // leading offset: not used by a swizzled K-major block narrower than the swizzle span
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version for sm_100
    d |= (uint64_t)4 << 61;   // SWIZZLE_64B
    return d;
}

// MN-major block of 64-byte lines (64-byte swizzle): r-rows are 64-byte lines, 8-row groups sbo_bytes = 512 apart,
// 64-wide blocks of the non-reduced dimension lbo_bytes apart.
__device__ __forceinline__ uint64_t make_desc64_mn(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version for sm_100
    d |= (uint64_t)4 << 61;   // SWIZZLE_64B
    return d;
}

// clamp(rint(y / q), lo, hi) exactly as the quantizer kernels compute it: reciprocal product, rounding by adding
// 1.5 * 2^23, and the IEEE quotient itself whenever the product lies within 2^-12 of a half-integer (the product
// is within 3 ulp of the quotient and indices are at most 255).  A NaN clamps to lo.
__device__ __forceinline__ int next_hard_index(float y, float q, float rq, float flo, float fhi, int fast)
{
    const float magic = 12582912.0f;
    float c = fminf(fmaxf(fast ? __fmul_rn(y, rq) : __fdiv_rn(y, q), flo), fhi);
    float t = __fadd_rn(c, magic);
    if (fast && fabsf(__fsub_rn(c, __fsub_rn(t, magic))) > 0.5f - 0.000244140625f) {
        c = fminf(fmaxf(__fdiv_rn(y, q), flo), fhi);
        t = __fadd_rn(c, magic);
    }
    return __float_as_int(t) - 0x4B400000;
}

// PAIR = false: one CTA per 128 x TN tile.  PAIR = true (TN = 256): a cluster of two CTAs per 256 x 256 tile with
// tcgen05.mma.cta_group::2: CTA r of the pair stages rows [128 r, 128 r + 128) of X and columns [128 r, 128 r + 128)
// of Y, the MMA issued by CTA 0 reads both halves from both shared memories and each CTA's TMEM receives its 128
// rows of the 256 x 256 accumulator.  A byte staged by either CTA then feeds twice as many multiply-adds, which is
// what the shared-memory-capacity x latency product of one SM cannot otherwise sustain.  Hand-shake in pair mode:
// the TMA loads of both CTAs count their bytes on CTA 0's "stage full" barrier; tcgen05.commit multicasts "stage
// free" and "accumulator full" to both CTAs; the epilogues of both CTAs arrive on CTA 0's "accumulator free" barrier.
// CONV (0 stored X, 1 forward-type gather, 2 transposed gather) is a template argument for the sake of the TMA
// producers' stage loop: every test of the mode taken out of it shows in the stage time.
template <bool PAIR, bool STORE_HEAVY, int CONV>
__global__ void __launch_bounds__(threads_tc(STORE_HEAVY), 1)
index_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ CUtensorMap map_f, const __grid_constant__ CUtensorMap map_acc,
                     const TcParams P)
{
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) unsigned long long bars[2 * kStagesMax + 4];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile int *abort_flag = &abort_s;

    constexpr int kEpiWarps = epi_warps(STORE_HEAVY);
    constexpr int kChunkStep = kEpiWarps / 4;                 // warps per TMEM lane quarter
    constexpr int kStages = PAIR ? (STORE_HEAVY ? 4 : 6) : (STORE_HEAVY ? 3 : 4);
    constexpr int kStageBytes = PAIR ? kStageBytesPair : kStageBytesSingle;
    constexpr int kOutBlocks = 1;                             // staging blocks per epilogue warp
    static_assert(kStages * kStageBytes + kEpiWarps * kOutBlocks * kOutWarpBytes + 1024 <= kSmemBytes, "shared memory");
    constexpr int TMU = PAIR ? 2 * TM : TM;                   // rows of a work unit's tile
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;      // CTA 0 of a pair issues the MMAs
    const int slot = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;     // this CTA's (pair's) work slot, of P.slots

    auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return smem_u32(&bars[kStagesMax + s]); };
    auto tfull_bar = [&](int b) { return smem_u32(&bars[2 * kStagesMax + b]); };
    auto tempty_bar = [&](int b) { return smem_u32(&bars[2 * kStagesMax + 2 + b]); };

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), PAIR ? 2 * kEpiWarps : kEpiWarps);       // one arrival per epilogue warp (of both CTAs in pair mode)
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();       // both CTAs' barriers exist before any remote arrive or multicast commit
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int b_blocks = PAIR ? 1 : (P.TN + 127) / 128;                   // 128-wide blocks of an MN-major B tile
    // (an MN-major Y block of a 64-channel tap holds the tap's 64 r-rows only)
    const uint32_t b_rrows = (P.k64 && P.b_mn_major) ? 64u : (uint32_t)BR;
    const uint32_t b_bytes = P.b_mn_major ? (uint32_t)b_blocks * 128u * b_rrows
                                          : (uint32_t)(PAIR ? 128 : P.TN) * (P.k64 ? 64u : (uint32_t)BR);     // (K-major: 64-byte rows as well)
    const int brow = PAIR ? (int)rank * 128 : 0;                          // this CTA's share of the Y tile
    // Tall tiles (one CTA per tile, TN <= 128, K-major X): a stage holds 256 rows of X, fetched by one TMA box, and the
    // same Y block serves two MMA sets whose accumulators sit 128 TMEM columns apart.  A stage costs its three single
    // threads about the same whatever it holds, so a narrow product, whose stages carry little, gets twice the rows
    // out of each.
    const int tall = PAIR ? 0 : P.tall;
    const int tmu = TMU << tall;                    // rows of a work unit's tile
    const int rows_cta = TM << tall;                // ... of which this CTA's
    const uint32_t a_bytes = (uint32_t)kABytes << tall;
    // a 64-channel tap fills half of the X block: rows of 64 bytes, 8 KB per 128 rows (the Y block keeps its place)
    // (a transposed 64-channel gather fills its block: two boxes of 64 channels x 128 pixels per 128 tile rows)
    const uint32_t stage_tx = (P.k64 ? a_bytes >> 1 : a_bytes) + b_bytes;
    bool failed = false;

    // The three roles below are single threads, and what bounds a pipeline stage is the length of their own
    // instruction streams (a poll of a barrier that is already complete costs some 40 cycles, every dependent
    // instruction a handful): each stage loop therefore keeps running addresses and coordinates, has no division,
    // no table look-up outside a tap change and no test of a launch parameter that could be taken outside.
    const uint32_t bar0 = smem_u32(&bars[0]);                    // full barriers; the empty ones follow at + 8 * kStagesMax
    constexpr uint32_t kEmptyOff = 8u * kStagesMax;
    constexpr uint32_t kRingBytes = (uint32_t)kStages * (uint32_t)kStageBytes;

    if (warp == 0 || warp == 2 + kEpiWarps) {
        // ------------------------------------------------------------ TMA producer (one lane; with a second TMA
        // warp the first issues the X-operand loads and arms the barrier, the second issues the Y-operand loads)
        const bool do_a = warp == 0, do_b = !kSplitProducer || warp != 0;
        if (lane == 0) {
            constexpr int conv = CONV;
            const int a_mn = P.a_mn_major, b_mn = P.b_mn_major, TNv = P.TN, tiles_j = P.tiles_j;
            const int cW = P.cW > 0 ? P.cW : 1, cH = P.cH > 0 ? P.cH : 1, cHW = cH * cW;
            const int cpad = P.cpad, cC = P.cC, c_stride = P.c_stride, pad_w = P.pad_w, pad_h = P.pad_h;
            const int last_tap = P.taps - 1, y_tap_rows = P.y_tap_rows;
            const int pix_dh = BR / cW, pix_dw = BR % cW;        // 128 pixels further on
            // pair: both CTAs' bytes are counted on CTA 0's barrier, which CTA 0 arms for the two of them
            const uint32_t arm_tx = PAIR ? 2u * stage_tx : stage_tx;
            const bool arm = do_a && rank == 0;
            const bool tall2 = tall != 0 && (conv == 2 || (conv == 0 && a_mn != 0));    // X fetched as two boxes per stage
            // boxes of a transposed patch tile
            const int t_box_rows = P.k64t ? 64 : TM, t_nbox = rows_cta / t_box_rows;
            const uint32_t t_box_bytes = (uint32_t)t_box_rows * BR;
            uint32_t st_off = 0u, st_bar = bar0, st_par = 1u;    // ring position: byte offset, full barrier, parity of "empty"
            // Forward-type patch gathers with one tile column and an unsplit reduction visit tiles slot, slot + slots,
            // ...: the pixel of a tile's first row then moves by a fixed step, kept as (image, row, column) with
            // carries instead of being divided out of the row index for every tile (a short tile has few stages to
            // hide that behind).
            const bool walk = conv == 1 && tiles_j == 1 && P.splits == 1;
            int wk_n = 0, wk_h = 0, wk_w = 0, wk_dn = 0, wk_dh = 0, wk_dw = 0;
            if (walk) {
                const int first = slot * tmu + (int)rank * rows_cta, step = P.slots * tmu;
                wk_n = first / cHW;
                wk_h = (first - wk_n * cHW) / cW;
                wk_w = first - wk_n * cHW - wk_h * cW;
                wk_dn = step / cHW;
                wk_dh = (step - wk_dn * cHW) / cW;
                wk_dw = step - wk_dn * cHW - wk_dh * cW;
            }
            SlotWork sw = slot_work(P, slot);
            while (!failed) {
                const WorkItem w = next_item(sw);
                if (!w.valid) break;
                const int tile = w.tile;
                const int ti = tiles_j == 1 ? tile : tile / tiles_j, tj = tile - ti * tiles_j;
                const int rb0 = w.rb0, nrb = w.rb1 - w.rb0;
                const int arow = ti * tmu + (int)rank * rows_cta;
                const int b_row0 = tj * TNv + brow;
                // Patch gather: pixel block, channel offset and filter tap of the first stage of this unit
                int g_c = 0, g_w = 0, g_h = 0, g_n = 0, g_ow = 0, g_oh = 0, g_tap = 0, b_tap_red = 0, b_tap_row = 0;
                if (walk) {
                    // a block wholly outside the matrix (second CTA of a ragged pair) loads block 0: never stored
                    const bool inside = arow < P.I;
                    g_n = inside ? wk_n : 0;
                    g_h = inside ? wk_h : 0;
                    g_w = inside ? wk_w : 0;
                    wk_w += wk_dw;
                    wk_h += wk_dh;
                    wk_n += wk_dn;
                    if (wk_w >= cW) {
                        wk_w -= cW;
                        ++wk_h;
                    }
                    if (wk_h >= cH) {
                        wk_h -= cH;
                        ++wk_n;
                    }
                    g_oh = P.tap_oh[0];
                    g_ow = P.tap_ow[0];
                    b_tap_row = y_tap_rows > 0 ? (int)P.tap_y[0] * y_tap_rows : 0;
                } else if (conv != 0) {
                    const int i0 = arow < P.I ? arow : 0;
                    g_tap = conv == 1 ? rb0 / P.cblocks : i0 / cpad;
                    g_c = conv == 1 ? (rb0 - g_tap * P.cblocks) * BR : i0 - g_tap * cpad;
                    const int pix = conv == 1 ? i0 : rb0 * BR;
                    g_n = pix / cHW;
                    const int rem = pix - g_n * cHW;
                    g_h = rem / cW;
                    g_w = rem - g_h * cW;
                    g_oh = P.tap_oh[g_tap];
                    g_ow = P.tap_ow[g_tap];
                    // Y coordinates of a tap: its own row block of a stacked matrix, or C (not the padded count)
                    // reduced columns per tap of a plain one
                    b_tap_row = y_tap_rows > 0 ? (int)P.tap_y[g_tap] * y_tap_rows : 0;
                    b_tap_red = y_tap_rows > 0 || conv != 1 ? 0 : g_tap * cC;
                }
                // further boxes of a transposed patch tile (128 tile rows each, or 64 for 64-channel taps): their own tap
                // and channel block
                int gx_c[3] = {0, 0, 0}, gx_ow[3] = {0, 0, 0}, gx_oh[3] = {0, 0, 0};
                if (conv == 2) {
#pragma unroll
                    for (int b = 1; b < 4; ++b) {           // (constant indices: the arrays stay in registers)
                        if (b < t_nbox) {
                            const int i1 = arow + b * t_box_rows < P.I ? arow + b * t_box_rows : 0;
                            const int tap1 = i1 / cpad;
                            gx_c[b - 1] = i1 - tap1 * cpad;
                            gx_oh[b - 1] = P.tap_oh[tap1];
                            gx_ow[b - 1] = P.tap_ow[tap1];
                        }
                    }
                }
                int c_red = rb0 * BR;                            // reduced coordinate of a stored operand
                int c_w = g_w * c_stride - pad_w, c_h = g_h * c_stride - pad_h;
                for (int i = 0; i < nrb; ++i) {
                    if (!mbar_try_wait_now(st_bar + kEmptyOff, st_par) &&
                        !mbar_wait(st_bar + kEmptyOff, st_par, abort_flag, P.wait_ns)) {
                        failed = true;
                        break;
                    }
                    const uint32_t sa = smem_base + st_off, sb = sa + a_bytes, fb = st_bar;
                    st_off += (uint32_t)kStageBytes;
                    st_bar += 8u;
                    if (st_off == kRingBytes) {
                        st_off = 0u;
                        st_bar = bar0;
                        st_par ^= 1u;
                    }
                    if (arm) mbar_expect_tx(fb, arm_tx);
                    if (conv == 0) {
                        if (do_a) {
                            const int x0 = a_mn ? arow : c_red, x1 = a_mn ? c_red : arow;    // {inner, outer}
                            if (PAIR) tma_load_2d_pair(sa, &map_a, x0, x1, fb);
                            else tma_load_2d(sa, &map_a, x0, x1, fb);
                            // (an MN-major box is 128 rows of the tile wide: a tall tile takes two)
                            if (tall2) tma_load_2d(sa + kABytes, &map_a, x0 + TM, x1, fb);
                        }
                        if (do_b) {
                            const int y0 = b_mn ? b_row0 : c_red, y1 = b_mn ? c_red : b_row0;
                            if (PAIR) tma_load_2d_pair(sb, &map_b, y0, y1, fb);
                            else if (b_mn) {
                                for (int bb = 0; bb < b_blocks; ++bb) tma_load_2d(sb + (uint32_t)bb * 128 * BR, &map_b, y0 + bb * 128, y1, fb);
                            } else tma_load_2d(sb, &map_b, y0, y1, fb);
                        }
                        c_red += BR;
                        continue;
                    }
                    if (do_a) {
                        if (PAIR) tma_load_im2col_pair(sa, &map_a, g_c, c_w, c_h, g_n, g_ow, g_oh, fb);
                        else tma_load_im2col(sa, &map_a, g_c, c_w, c_h, g_n, g_ow, g_oh, fb);
                        if (conv == 2) {
#pragma unroll
                            for (int b = 1; b < 4; ++b)
                                if (b < t_nbox) {
                                    if (PAIR) tma_load_im2col_pair(sa + (uint32_t)b * t_box_bytes, &map_a, gx_c[b - 1], c_w, c_h, g_n, gx_ow[b - 1], gx_oh[b - 1], fb);
                                    else tma_load_im2col(sa + (uint32_t)b * t_box_bytes, &map_a, gx_c[b - 1], c_w, c_h, g_n, gx_ow[b - 1], gx_oh[b - 1], fb);
                                }
                        }
                    }
                    if (do_b) {
                        const int red = conv == 1 ? b_tap_red + g_c : c_red, row = b_row0 + b_tap_row;
                        const int y0 = b_mn ? row : red, y1 = b_mn ? red : row;
                        if (PAIR) tma_load_2d_pair(sb, &map_b, y0, y1, fb);
                        else if (b_mn) {
                            for (int bb = 0; bb < b_blocks; ++bb) tma_load_2d(sb + (uint32_t)bb * 128 * BR, &map_b, y0 + bb * 128, y1, fb);
                        } else tma_load_2d(sb, &map_b, y0, y1, fb);
                    }
                    if (conv == 1) {              // next stage: next channel block, then next tap
                        g_c += BR;
                        if (g_c == cpad) {
                            g_c = 0;
                            g_tap = g_tap < last_tap ? g_tap + 1 : g_tap;      // (past the last tap nothing more is loaded)
                            g_oh = P.tap_oh[g_tap];
                            g_ow = P.tap_ow[g_tap];
                            if (y_tap_rows > 0) b_tap_row = (int)P.tap_y[g_tap] * y_tap_rows;
                            else b_tap_red = g_tap * cC;
                        }
                    } else {                      // next stage: 128 pixels further on
                        c_red += BR;
                        g_w += pix_dw;
                        g_h += pix_dh;
                        if (g_w >= cW) {
                            g_w -= cW;
                            ++g_h;
                        }
                        while (g_h >= cH) {
                            g_h -= cH;
                            ++g_n;
                        }
                        c_w = g_w * c_stride - pad_w;
                        c_h = g_h * c_stride - pad_h;
                    }
                }
            }
            if (failed) {
                abort_s = 1;
                record_timeout(P.status);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane; CTA 0 in pair mode)
        if (lane == 0 && rank == 0) {
            // Operand descriptors: the upper word is fixed per launch (stride between 8-row groups, version, swizzle),
            // the lower word holds the start address and the leading offset and moves with the stage and with k.
            // K-major: rows are 128-byte lines, 8-row groups 1024 bytes apart, 32 bytes per MMA along r.
            // MN-major: r-rows are 128-byte lines, 8-row groups 1024 bytes apart (SBO), 128-wide blocks of the
            // non-reduced dimension BR * 128 bytes apart (LBO), 32 r-rows = 4096 bytes per MMA.
            const uint64_t a_d0 = P.k64 ? make_desc64(smem_base, 512)
                                        : (P.k64t ? make_desc64_mn(smem_base, 64 * BR, 512)
                                                  : (P.a_mn_major ? make_desc(smem_base, 128 * BR, 1024) : make_desc(smem_base, 16, 1024)));
            const int k64 = P.k64;
            const uint32_t a_sub16 = (uint32_t)((k64 ? kABytes / 2 : kABytes) >> 4);      // 128 rows further on, in 16-byte units
            const uint64_t b_d0 = P.b_mn_major ? make_desc(smem_base + a_bytes, 128 * BR, 1024)
                                               : (P.k64 ? make_desc64(smem_base + a_bytes, 512) : make_desc(smem_base + a_bytes, 16, 1024));
            const uint32_t a_hi = (uint32_t)(a_d0 >> 32), b_hi = (uint32_t)(b_d0 >> 32);
            const uint32_t a_lo0 = (uint32_t)a_d0, b_lo0 = (uint32_t)b_d0;
            const uint32_t a_step = P.k64t ? (2048u >> 4) : (P.a_mn_major ? (4096u >> 4) : (32u >> 4));      // 32 r-rows, or 32 bytes of r
            const uint32_t b_step = P.b_mn_major ? (4096u >> 4) : (32u >> 4);
            const uint32_t idesc = P.idesc;
            uint32_t tcount = 0;
            uint32_t st_off16 = 0u, st_bar = bar0, st_par = 0u;     // ring position (offset in 16-byte units), parity of "full"
            SlotWork sw = slot_work(P, slot);
            for (; !failed; ++tcount) {
                const WorkItem w = next_item(sw);
                if (!w.valid) break;
                const int nrb = w.rb1 - w.rb0;
                const int buf = tcount & 1;
                const uint32_t tph = (tcount >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), tph ^ 1u, abort_flag, P.wait_ns)) {
                    failed = true;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * 256u;
                uint32_t acc = 0u;                                   // the first MMA of a unit overwrites the accumulator
                for (int i = 0; i < nrb; ++i) {
                    if (!mbar_try_wait_now(st_bar, st_par) && !mbar_wait(st_bar, st_par, abort_flag, P.wait_ns)) {
                        failed = true;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + st_off16, b_lo = b_lo0 + st_off16, eb = st_bar + kEmptyOff;
                    st_off16 += (uint32_t)(kStageBytes >> 4);
                    st_bar += 8u;
                    if (st_off16 == (kRingBytes >> 4)) {
                        st_off16 = 0u;
                        st_bar = bar0;
                        st_par ^= 1u;
                    }
                    if (k64) {          // 64 bytes of r per stage: two MMAs per 128-row block
                        if (PAIR) tc_mma2_i8<true>(d_tmem, a_lo, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                        else {
                            tc_mma2_i8<false>(d_tmem, a_lo, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                            if (tall) tc_mma2_i8<false>(d_tmem + 128u, a_lo + a_sub16, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                        }
                    } else if (PAIR) tc_mma4_i8<true>(d_tmem, a_lo, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                    else {
                        tc_mma4_i8<false>(d_tmem, a_lo, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                        if (tall) tc_mma4_i8<false>(d_tmem + 128u, a_lo + a_sub16, a_hi, a_step, b_lo, b_hi, b_step, idesc, acc);
                    }
                    acc = 1u;
                    // frees the stage (in both CTAs of a pair) once these MMAs have read it
                    if (PAIR) tc_commit_pair(eb);
                    else tc_commit(eb);
                }
                if (!failed) {                               // accumulator complete
                    if (PAIR) tc_commit_pair(tfull_bar(buf));
                    else tc_commit(tfull_bar(buf));
                }
            }
            if (failed) {
                abort_s = 1;
                record_timeout(P.status);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps 2..9
        // Each warp works on its own: it reads its 32 TMEM lanes (= 32 output rows), stages 32 columns of them in a
        // 4 KB block of its own and sends that block with its own TMA store, so the warps never wait for one
        // another inside a tile; the TMEM load of the next 32 columns is in flight while the current ones are sent.
        const int quarter = warp & 3;               // TMEM lanes this warp may read: 32 * (warp % 4) ..
        const int half = (warp - 2) >> 2;           // which of the two warps of this quarter: chunks half, half + 2, ..
        const uint32_t wbuf = smem_base + (uint32_t)(kStages * kStageBytes) + (uint32_t)((warp - 2) * kOutBlocks * kOutWarpBytes);
        uint32_t tcount = 0, ocount = 0;

        // 32 four-byte values of this thread's row -> this warp's swizzled staging block (its blocks in turn)
        auto stage = [&](const uint32_t (&w)[32]) -> uint32_t {
            const uint32_t blk = wbuf + ocount * (uint32_t)kOutWarpBytes;
            if (lane == 0) bulk_wait_read<kOutBlocks - 1>();      // the send that last used this block has read it
            __syncwarp();
            const uint32_t dst = blk + (uint32_t)lane * 128u;
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)((c4 ^ (lane & 7)) << 4)),
                             "r"(w[4 * c4]), "r"(w[4 * c4 + 1]), "r"(w[4 * c4 + 2]), "r"(w[4 * c4 + 3])
                             : "memory");
            return blk;
        };
        // staged block -> TMA store or reduce-add of a {32 columns, 32 rows} box at (col0, row0)
        auto stage_and_send = [&](const uint32_t (&w)[32], const CUtensorMap *map, bool reduce, int col0, int row0, int row_end) {
            const uint32_t blk = stage(w);
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && row0 < row_end) {
                if (reduce) tma_reduce_add_2d(map, col0, row0, blk);
                else tma_store_2d(map, col0, row0, blk);
                bulk_commit();
            }
            ocount = ocount + 1 == (uint32_t)kOutBlocks ? 0u : ocount + 1;      // next block; one copied out by the warp itself is reused at once
        };
        // Same staging, then the warp copies its 32 rows out itself, one row (up to 128 contiguous bytes) per
        // instruction: for outputs TMA cannot take (row pitch or base not a multiple of 16 bytes, 16-column tiles).
        int my_orow = 0;            // scattered output: where this thread's row of the current tile goes
        auto stage_and_copy = [&](const uint32_t (&w)[32], int32_t *out, bool reduce, long long row_off, int row0,
                                  int col0, int ncol, bool as_float = false) {
            const uint32_t blk = stage(w);
            __syncwarp();
            if (!reduce && ncol == 32 && P.copy_vec) {
                // whole 32-column chunk, 16-byte aligned rows: eight lanes write the 128 bytes of one row, four rows
                // per instruction
                const int c4 = lane & 7;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int rr = it * 4 + (lane >> 3);
                    int grow = row0 + rr;
                    const bool live = grow < P.I_out;
                    if (P.sc_on) grow = __shfl_sync(0xffffffffu, my_orow, rr);
                    uint4 val;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                 : "r"(blk + (uint32_t)rr * 128u + (uint32_t)((c4 ^ (rr & 7)) << 4)));
                    if (live) *reinterpret_cast<uint4 *>(out + (row_off + grow) * P.J + col0 + 4 * c4) = val;
                }
                __syncwarp();
                return;
            }
            for (int rr = 0; rr < 32; ++rr) {
                int grow = row0 + rr;
                if (grow >= P.I_out) break;                                // uniform over the warp
                if (P.sc_on) grow = __shfl_sync(0xffffffffu, my_orow, rr);
                uint32_t val;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(val)
                             : "r"(blk + (uint32_t)rr * 128u + (uint32_t)(((lane >> 2) ^ (rr & 7)) << 4) + (uint32_t)((lane & 3) << 2)));
                if (lane < ncol) {
                    int32_t *q = out + (row_off + grow) * P.J + col0 + lane;
                    if (reduce && as_float) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(q), "f"(__uint_as_float(val)) : "memory");
                    else if (reduce) asm volatile("red.global.add.s32 [%0], %1;" ::"l"(q), "r"(val) : "memory");
                    else *q = (int32_t)val;
                }
            }
            __syncwarp();
        };

        SlotWork sw = slot_work(P, slot);
        for (;; ++tcount) {
            const WorkItem w = next_item(sw);
            if (!w.valid) break;
            const int tile = w.tile;
            const int ti = tile / P.tiles_j, tj = tile % P.tiles_j;
            const int slab_row0 = w.split * P.slab_rows;             // 0 unless partial tiles go to per-split slabs
            const int buf = tcount & 1;
            const uint32_t tph = (tcount >> 1) & 1u;
            // the epilogue warps agree on the outcome, so that either all of them or none release the accumulator
            if (!epi_all<32 * kEpiWarps>(mbar_wait(tfull_bar(buf), tph, abort_flag, P.wait_ns))) {
                failed = true;
                break;
            }
            tc_fence_after();
            for (int sub = 0; sub <= tall; ++sub) {          // the two 128-row halves of a tall tile in turn
            // first output row of this warp; a transposed patch matrix whose taps are padded to 128 channels has
            // rows that exist only in the tiling (never stored) and the others move up
            int wrow0 = ti * tmu + (int)rank * rows_cta + sub * TM + quarter * 32;
            if (P.conv == 2 && P.cpad != P.cC) {
                const int tap = wrow0 / P.cpad, c = wrow0 - tap * P.cpad;
                wrow0 = c < P.cC ? tap * P.cC + c : 0x7fffff00;
            }
            if (P.sc_on) {
                const int grow = wrow0 + lane, per = P.sc_P * P.sc_Q;
                const int n = grow / per, rem = grow - n * per, pi = rem / P.sc_Q, qj = rem - pi * P.sc_Q;
                my_orow = (n * P.sc_H + P.sc_s * pi + P.sc_a) * P.sc_W + P.sc_s * qj + P.sc_b;
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * 256u + (uint32_t)sub * 128u;
            const int tile_cols = min(P.TN, P.J - tj * P.TN);
            const int nchunks = wrow0 < P.I_out ? (tile_cols + 31) / 32 : 0;   // uniform over the warp

            // one chunk = 32 columns of the warp's 32 rows
            auto emit = [&](const uint32_t (&v)[32], int ch) {
                const int c0 = ch * 32;
                const int col0 = tj * P.TN + c0;
                const int ncol = min(min(32, P.TN - c0), P.J - col0);
                if (P.splits > 1) {
                    if (P.tma_acc) stage_and_send(v, &map_acc, P.slab_rows == 0, col0, slab_row0 + wrow0, 0x7fffffff);
                    else stage_and_copy(v, P.acc_out, P.slab_rows == 0, slab_row0, wrow0, col0, ncol);
                    return;
                }
                if (P.acc_out != nullptr) {
                    if (P.tma_acc) stage_and_send(v, &map_acc, false, col0, wrow0, P.I_out);
                    else stage_and_copy(v, P.acc_out, false, 0, wrow0, col0, ncol);
                }
                if (P.f_out != nullptr || P.nq_out != nullptr) {
                    uint32_t f[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) f[c] = __float_as_uint(__fmul_rn((float)(int)v[c], P.scale));
                    if (P.bias != nullptr) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c < ncol) f[c] = __float_as_uint(__fadd_rn(__uint_as_float(f[c]), P.bias[col0 + c]));
                    }
                    if (P.nq_out != nullptr && wrow0 + lane < P.I_out) {
                        // the next layer's index of this thread's 32 outputs: 32 consecutive bytes of its row
                        uint32_t pk[8];
#pragma unroll
                        for (int c4 = 0; c4 < 8; ++c4) {
                            uint32_t word = 0u;
#pragma unroll
                            for (int b = 0; b < 4; ++b) {
                                const int k = next_hard_index(__uint_as_float(f[4 * c4 + b]), P.nq_q, P.nq_rq, P.nq_flo,
                                                              P.nq_fhi, P.nq_fast);
                                word |= ((uint32_t)k & 0xffu) << (8 * b);
                            }
                            pk[c4] = word;
                        }
                        unsigned char *dst = P.nq_out + (long long)(wrow0 + lane) * P.J + col0;
                        if (P.nq_vec) {         // J is a multiple of 16: each half of the chunk is wholly inside or outside
                            if (ncol > 0) *reinterpret_cast<uint4 *>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            if (ncol > 16) *reinterpret_cast<uint4 *>(dst + 16) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c < ncol) dst[c] = (unsigned char)(pk[c >> 2] >> (8 * (c & 3)));
                        }
                    }
                    if (P.f_out != nullptr) {
                        if (P.tma_f) stage_and_send(f, &map_f, P.f_acc != 0, col0, wrow0, P.I_out);
                        else stage_and_copy(f, reinterpret_cast<int32_t *>(P.f_out), P.f_acc != 0, 0, wrow0, col0, ncol, true);
                    }
                }
            };

            uint32_t va[32];
            int ch = half;
            if (STORE_HEAVY) {
                // many warps, one chunk in flight each: the other warps hide the TMEM load
                for (; ch < nchunks; ch += kChunkStep) {
                    tc_ld32(taddr + (uint32_t)(ch * 32), va);
                    tc_wait_ld_pin(va);
                    emit(va, ch);
                }
            } else {
                uint32_t vb[32];
                if (ch < nchunks) tc_ld32(taddr + (uint32_t)(ch * 32), va);
                while (ch < nchunks) {
                    tc_wait_ld_pin(va);
                    if (ch + kChunkStep < nchunks) tc_ld32(taddr + (uint32_t)((ch + kChunkStep) * 32), vb);
                    emit(va, ch);
                    ch += kChunkStep;
                    if (ch < nchunks) {
                        tc_wait_ld_pin(vb);
                        if (ch + kChunkStep < nchunks) tc_ld32(taddr + (uint32_t)((ch + kChunkStep) * 32), va);
                        emit(vb, ch);
                        ch += kChunkStep;
                    }
                }
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_remote(tempty_bar(buf), 0u);
                else mbar_arrive(tempty_bar(buf));
            }
        }
        if (lane == 0) bulk_wait_all();             // staged blocks are out before shared memory goes away
        if (failed && lane == 0) {
            abort_s = 1;
            record_timeout(P.status);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();       // neither CTA leaves while its partner may still touch its shared memory / TMEM
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// float output of a split run: f = (float)acc * scale (+ bias[j])
__global__ void scale_acc_kernel(const int32_t *__restrict__ acc, float *__restrict__ f, long long n, int J, float scale,
                                 const float *__restrict__ bias, int accumulate)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float v = __fmul_rn((float)acc[i], scale);
        if (bias != nullptr) v = __fadd_rn(v, bias[i % J]);
        f[i] = accumulate ? __fadd_rn(f[i], v) : v;
    }
}

// float output of a split run whose partial sums sit in per-split slabs: the slabs are summed in int64 (each
// slab is exact in int32, the total need not be), converted once and scaled.
__global__ void sum_slabs_kernel(const int32_t *__restrict__ slabs, int splits, long long slab_elems, float *__restrict__ f,
                                 long long n, int J, float scale, const float *__restrict__ bias, int accumulate)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        long long acc = 0;
        for (int sp = 0; sp < splits; ++sp) acc += (long long)slabs[sp * slab_elems + i];
        float v = __fmul_rn(__ll2float_rn(acc), scale);
        if (bias != nullptr) v = __fadd_rn(v, bias[i % J]);
        f[i] = accumulate ? __fadd_rn(f[i], v) : v;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Output matrix [rows][cols] of 4-byte elements, row pitch cols * 4; box = {32 columns (128 bytes), 32 rows}: one
// epilogue warp's staging block.
bool encode_out_map(CUtensorMap *map, const void *base, uint64_t cols, uint64_t rows, bool is_float)
{
    EncodeTiledFn fn = get_encode();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 4};
    const cuuint32_t box[2] = {32u, 32u};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, is_float ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_INT32, 2, const_cast<void *>(base),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2D byte tensor [outer][inner] with row pitch `pitch` bytes; box = {128 bytes, box_rows}, 128-byte swizzle.
bool encode_map(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint64_t pitch, uint32_t box_rows,
                bool rows64 = false)      // rows64: boxes of 64-byte rows under the 64-byte swizzle
{
    EncodeTiledFn fn = get_encode();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {pitch};
    const cuuint32_t box[2] = {rows64 ? 64u : 128u, box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, rows64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

// [N,H,W,C] byte tensor read in im2col mode: one load fetches 128 consecutive base pixels x 128 channel bytes, the
// base pixels running over the gather's grid (first at the lower corner, `stride` apart), the filter tap given per
// load as an offset.
bool encode_im2col_map(CUtensorMap *map, const void *base, const ConvGather &g, uint32_t pixels)
{
    const bool k64 = g.C == 64;      // 64-channel taps: boxes 64 channels wide, 64-byte swizzle
    static EncodeIm2colFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return false;
        }
        fn = reinterpret_cast<EncodeIm2colFn>(p);
    }
    const cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    const cuuint64_t strides[3] = {(cuuint64_t)g.C, (cuuint64_t)g.C * g.W, (cuuint64_t)g.C * g.W * g.H};
    const int lower[2] = {g.lower_w, g.lower_h};                    // {w, h}: first base pixel
    // last base pixel, relative to the far corner of the tensor
    const int upper[2] = {g.lower_w + (g.Q - 1) * g.stride - (g.W - 1), g.lower_h + (g.P - 1) * g.stride - (g.H - 1)};
    const cuuint32_t estr[4] = {1u, (cuuint32_t)g.stride, (cuuint32_t)g.stride, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, lower, upper, k64 ? 64u : 128u, pixels,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, k64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace {
// The template instance for a launch: CTA pair or single CTA, 16 or 8 epilogue warps, kind of X operand.
template <bool PAIR, bool STORE_HEAVY>
const void *kernel_variant_conv(int conv)
{
    if (conv == 1) return reinterpret_cast<const void *>(&index_gemm_tc_kernel<PAIR, STORE_HEAVY, 1>);
    if (conv == 2) return reinterpret_cast<const void *>(&index_gemm_tc_kernel<PAIR, STORE_HEAVY, 2>);
    return reinterpret_cast<const void *>(&index_gemm_tc_kernel<PAIR, STORE_HEAVY, 0>);
}
const void *kernel_variant(bool pair, bool store_heavy, int conv)
{
    if (pair) return store_heavy ? kernel_variant_conv<true, true>(conv) : kernel_variant_conv<true, false>(conv);
    return store_heavy ? kernel_variant_conv<false, true>(conv) : kernel_variant_conv<false, false>(conv);
}
}  // namespace

namespace {
// Split of the reduced dimension: when the tiles alone cannot occupy half of the device, and always into at
// least min_splits parts (the caller's bound that keeps every part's int32 partial sums exact).
struct Plan {
    int TN;         // output columns per tile
    int splits;     // parts of the reduced dimension
    int pair;       // 1: CTA pairs on 256-row tiles
    int tall;       // 1: one CTA per 256-row tile (narrow outputs, K-major X)
    int tile_rows;  // output rows per work unit (128, or 256 for a pair or a tall tile)
};

Plan plan(int I, int J, int R, int min_splits)
{
    Plan p;
    p.TN = 256;
    while (p.TN > 16 && p.TN / 2 >= J) p.TN /= 2;
    p.pair = (p.TN == 256 && I > TM) ? 1 : 0;
    p.tall = (!p.pair && p.TN >= 32 && p.TN <= 128 && I >= 4 * TM) ? 1 : 0;
    p.tile_rows = (p.pair || p.tall) ? 2 * TM : TM;
    const int slots = p.pair ? kPlanSMs / 2 : kPlanSMs;      // work units that run at once
    const long long tiles = (long long)((I + p.tile_rows - 1) / p.tile_rows) * ((J + p.TN - 1) / p.TN);
    const int rblocks = (R + BR - 1) / BR;
    p.splits = 1;
    if (tiles * 2 <= slots) {
        p.splits = (int)(slots / tiles);
        const int max_splits = (rblocks + 3) / 4;      // keep at least four stages of work per unit
        if (p.splits > max_splits) p.splits = max_splits;
        if (p.splits < 1) p.splits = 1;
    }
    if (p.splits < min_splits) p.splits = min_splits;
    return p;
}

// Parts the reduced dimension must be cut into so that a part's sum of |x| * |y| stays below 2^31 (whole r-blocks).
int min_exact_splits(int R, long long xmax, long long ymax)
{
    const long long per_term = xmax * ymax > 0 ? xmax * ymax : 1;
    const long long rows = (((long long)1 << 31) - 1) / per_term;     // rows one part may hold
    const long long rb_max = rows / BR;
    if (rb_max < 1) return -1;                                        // cannot happen for byte operands
    const long long rblocks = (R + BR - 1) / BR;
    return (int)((rblocks + rb_max - 1) / rb_max);
}
}  // namespace

// Scratch bytes a product may need: one int32 slab per split of the reduced dimension (also when the dimension is
// so long that its int32 total could overflow for byte operands of the widest range and it has to be cut).
size_t tc_gemm_scratch_bytes(int I, int J, int R)
{
    Plan p = plan(I, J, R, 1);
    size_t need = 0;
    if (p.splits > 1) need = (size_t)((I + p.tile_rows - 1) / p.tile_rows) * p.tile_rows * (size_t)J * sizeof(int32_t) * p.splits;
    if ((long long)R * 255 * 128 >= ((long long)1 << 31)) {
        p = plan(I, J, R, min_exact_splits(R, 255, 128));
        const size_t slab = (size_t)((I + p.tile_rows - 1) / p.tile_rows) * p.tile_rows * (size_t)J * sizeof(int32_t);
        if (slab * p.splits > need) need = slab * p.splits;
    }
    return (need + 255u) & ~(size_t)255u;
}

// X: the operand whose non-reduced dimension indexes output rows; Y: output columns.  An operand is MN-major
// when its non-reduced dimension is the contiguous one (stride_outer == 1).  scratch: tc_gemm_scratch_bytes(I, J, R)
// bytes, used only when the reduced dimension is split and no int32 output was requested.
int launch_index_gemm_tc(const GemmOperand &X, const GemmOperand &Y, int I, int J, int R, int32_t *acc_out,
                         float *f_out, float scale, const float *bias, void *scratch, int *status,
                         cudaStream_t stream, const ConvGather *conv, const NextQuant *next, bool accumulate_f,
                         bool compact_scratch)
{
    const bool a_mn = conv != nullptr ? conv->transposed != 0 : (X.stride_outer == 1 && X.stride_red != 1);
    const bool b_mn = Y.stride_outer == 1 && Y.stride_red != 1;
    // extents the tiling runs over: a patch matrix has its taps padded to whole 128-channel blocks
    int It = I, Rt = R;
    if (conv != nullptr) {
        const int cpad = (conv->C + BR - 1) / BR * BR;
        if (conv->transposed) It = conv->taps * (conv->C == 64 ? 64 : cpad);     // (64-channel taps are not padded)
        else Rt = conv->taps * cpad;
    }
    TcParams P;
    P.I = It;
    P.I_out = I;
    P.J = J;
    P.R = Rt;
    // Exactness: a part of the reduced dimension is summed in int32, so |sum| <= rows * xmax * ymax must stay
    // below 2^31 per part.  When the whole dimension does not satisfy that, it is cut into enough parts, each part
    // keeps its own slab, and the slabs are summed in int64 (float output only).
    const bool wide = (long long)Rt * X.absmax * Y.absmax >= ((long long)1 << 31);
    if (wide && acc_out != nullptr) return CDL_ERR_OVERFLOW_RISK;
    const Plan pl = plan(It, J, Rt, wide ? min_exact_splits(Rt, X.absmax, Y.absmax) : 1);
    const bool want_next = next != nullptr && next->idx_out != nullptr;
    if (want_next && wide) return CDL_ERR_OVERFLOW_RISK;     // the index is taken from one finished accumulator
    const int TN = pl.TN;
    const bool scatter = conv != nullptr && conv->sc_on != 0;
    if (scatter && wide) return CDL_ERR_OVERFLOW_RISK;       // scattered rows are written by the product's own epilogue
    const int splits = (want_next || scatter) ? 1 : pl.splits;
    const bool pair = pl.pair != 0;
    P.TN = TN;
    P.tall = pl.tall;
    P.k64 = (conv != nullptr && !conv->transposed && conv->C == 64) ? 1 : 0;
    P.k64t = (conv != nullptr && conv->transposed && conv->C == 64) ? 1 : 0;
    P.tiles_i = (It + pl.tile_rows - 1) / pl.tile_rows;
    // A split reduction with only a float output keeps one slab per split (plain stores, no clear, no atomics in L2)
    // and sums the slabs in the conversion kernel; with compact_scratch (or an int32 output) the splits add into
    // one I x J buffer instead.
    const bool slabs = wide || (splits > 1 && acc_out == nullptr && !compact_scratch);
    P.slab_rows = slabs ? P.tiles_i * pl.tile_rows : 0;
    P.tiles_j = (J + TN - 1) / TN;
    P.rblocks = (Rt + BR - 1) / BR;
    const int sms = sm_count();
    if (sms <= 0) return CDL_ERR_LAUNCH;
    const long long tiles = (long long)P.tiles_i * P.tiles_j;
    if (tiles > 0x3fffffff || tiles * splits > 0x7fffffff) return CDL_ERR_ARG;
    P.splits = splits;
    P.a_mn_major = a_mn ? 1 : 0;
    P.b_mn_major = b_mn ? 1 : 0;
    P.idesc = (2u << 4) | ((X.is_unsigned ? 0u : 1u) << 7) | ((Y.is_unsigned ? 0u : 1u) << 10) |
              ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)((pl.pair ? 2 * TM : TM) >> 4) << 24);
    P.nq_out = nullptr;
    P.nq_q = P.nq_rq = P.nq_flo = P.nq_fhi = 0.0f;
    P.nq_fast = P.nq_vec = 0;
    if (next != nullptr && next->idx_out != nullptr) {
        P.nq_out = static_cast<unsigned char *>(next->idx_out);
        P.nq_q = next->q;
        P.nq_rq = next->rq;
        P.nq_flo = next->flo;
        P.nq_fhi = next->fhi;
        P.nq_fast = next->fast_div;
        P.nq_vec = ((J & 15) == 0 && (reinterpret_cast<uintptr_t>(next->idx_out) & 15u) == 0) ? 1 : 0;
    }
    P.conv = 0;
    P.cH = P.cW = P.cC = P.cblocks = P.cpad = P.pad_h = P.pad_w = P.taps = P.y_tap_rows = 0;
    P.c_stride = 1;
    P.sc_on = P.sc_P = P.sc_Q = P.sc_H = P.sc_W = P.sc_s = P.sc_a = P.sc_b = 0;
    memset(P.tap_oh, 0, sizeof P.tap_oh);
    memset(P.tap_ow, 0, sizeof P.tap_ow);
    memset(P.tap_y, 0, sizeof P.tap_y);
    if (conv != nullptr) {
        if (conv->C % 64 != 0 || conv->taps < 1 || conv->taps > kMaxTaps || conv->stride < 1) return CDL_ERR_ARG;
        P.conv = conv->transposed ? 2 : 1;
        P.cH = conv->P;
        P.cW = conv->Q;
        P.cC = conv->C;
        P.cblocks = (conv->C + BR - 1) / BR;
        P.cpad = P.k64t ? 64 : P.cblocks * BR;
        P.pad_h = -conv->lower_h;
        P.pad_w = -conv->lower_w;
        P.c_stride = conv->stride;
        P.taps = conv->taps;
        P.y_tap_rows = conv->y_tap_rows;
        for (int t = 0; t < conv->taps; ++t) {
            if (conv->oh[t] < 0 || conv->ow[t] < 0) return CDL_ERR_ARG;
            P.tap_oh[t] = conv->oh[t];
            P.tap_ow[t] = conv->ow[t];
            P.tap_y[t] = conv->ytap[t];
        }
        if (scatter) {
            P.sc_on = 1;
            P.sc_P = conv->P;
            P.sc_Q = conv->Q;
            P.sc_H = conv->sc_H;
            P.sc_W = conv->sc_W;
            P.sc_s = conv->sc_s;
            P.sc_a = conv->sc_a;
            P.sc_b = conv->sc_b;
        }
    }
    P.scale = scale;
    P.f_acc = accumulate_f ? 1 : 0;
    P.bias = bias;
    P.status = status;
    P.wait_ns = kWaitNs;
    P.f_out = f_out;
    P.acc_out = acc_out;
    const long long n_out = (long long)I * J;
    if (slabs) {
        P.acc_out = static_cast<int32_t *>(scratch);       // slabs: every element is written, nothing to clear
        if (P.acc_out == nullptr) return CDL_ERR_WORKSPACE;
    } else if (splits > 1) {
        if (P.acc_out == nullptr) P.acc_out = static_cast<int32_t *>(scratch);
        if (P.acc_out == nullptr) return CDL_ERR_WORKSPACE;
        if (cudaMemsetAsync(P.acc_out, 0, (size_t)n_out * sizeof(int32_t), stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }

    CUtensorMap map_a, map_b;
    bool ok;
    // K-major operand: stored [outer][r], r contiguous -> inner = r.  MN-major: stored [r][outer] -> inner = outer.
    if (conv != nullptr) ok = encode_im2col_map(&map_a, X.ptr, *conv, conv->transposed ? (uint32_t)BR : (uint32_t)(TM << pl.tall));
    else if (a_mn) ok = encode_map(&map_a, X.ptr, (uint64_t)I, (uint64_t)R, (uint64_t)X.stride_red, BR);
    else ok = encode_map(&map_a, X.ptr, (uint64_t)R, (uint64_t)I, (uint64_t)X.stride_outer, (uint32_t)(TM << pl.tall));     // K-major: one box of the tile's rows
    if (b_mn) ok = ok && encode_map(&map_b, Y.ptr, (uint64_t)J, (uint64_t)R, (uint64_t)Y.stride_red, P.k64 ? 64u : (uint32_t)BR);
    else if (conv != nullptr && conv->y_tap_rows > 0)   // all taps' row blocks of the stored matrix, conv->C reduced columns each
        ok = ok && encode_map(&map_b, Y.ptr, (uint64_t)conv->C, (uint64_t)conv->y_rows,
                              (uint64_t)Y.stride_outer, pair ? 128u : (uint32_t)TN, P.k64 != 0);
    else ok = ok && encode_map(&map_b, Y.ptr, (uint64_t)R, (uint64_t)J, (uint64_t)Y.stride_outer, pair ? 128u : (uint32_t)TN, P.k64 != 0);
    // outputs through shared memory + TMA when their pitch and base allow it and the tile is at least one box wide
    CUtensorMap map_f = map_a, map_acc = map_a;      // placeholders when unused
    const bool out_ok = TN >= 32 && (J & 3) == 0 && !scatter;      // scattered rows are copied out by the warps
    P.tma_f = 0;
    P.tma_acc = 0;
    P.copy_vec = ((J & 3) == 0 && (reinterpret_cast<uintptr_t>(f_out) & 15u) == 0 && (reinterpret_cast<uintptr_t>(P.acc_out) & 15u) == 0) ? 1 : 0;
    if (out_ok && splits == 1 && !slabs && f_out != nullptr && (reinterpret_cast<uintptr_t>(f_out) & 15u) == 0) {
        ok = ok && encode_out_map(&map_f, f_out, (uint64_t)J, (uint64_t)I, true);
        P.tma_f = 1;
    }
    if (out_ok && P.acc_out != nullptr && (reinterpret_cast<uintptr_t>(P.acc_out) & 15u) == 0) {
        const uint64_t acc_rows = slabs ? (uint64_t)splits * (uint64_t)P.slab_rows : (uint64_t)I;
        ok = ok && encode_out_map(&map_acc, P.acc_out, (uint64_t)J, acc_rows, false);
        P.tma_acc = 1;
    }
    if (!ok) return CDL_ERR_LAUNCH;

    static bool attr_set[64];
    static int pair_slots[64];         // CTA pairs the device runs at once
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return CDL_ERR_LAUNCH;
    if (!attr_set[dev]) {
        for (int v = 0; v < 12; ++v) {
            if (cudaFuncSetAttribute(kernel_variant((v & 1) != 0, (v & 2) != 0, v >> 2), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
                (void)cudaGetLastError();
                return CDL_ERR_LAUNCH;
            }
        }
        cudaLaunchConfig_t qc = {};
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = 2;
        qa[0].val.clusterDim.y = 1;
        qa[0].val.clusterDim.z = 1;
        qc.gridDim = dim3(2 * (sms / 2));
        qc.blockDim = dim3(threads_tc(false));
        qc.dynamicSmemBytes = kSmemBytes;
        qc.attrs = qa;
        qc.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, kernel_variant(true, false, 0), &qc) != cudaSuccess || nclusters < 1) {
            (void)cudaGetLastError();
            nclusters = sms / 2;
        }
        pair_slots[dev] = nclusters < sms / 2 ? nclusters : sms / 2;
        attr_set[dev] = true;
    }
    const long long units = tiles * splits;
    const int dev_slots = pair ? pair_slots[dev] : sms;
    P.slots = (int)(units < dev_slots ? units : dev_slots);
    // bytes a CTA loads per work unit against the bytes it stores (4-byte outputs of a 128 x TN tile)
    const long long unit_load = (long long)((P.rblocks + splits - 1) / splits) * ((kABytes << pl.tall) + (pair ? 128 : TN) * BR);
    const bool store_heavy = unit_load <= 2ll * (TM << pl.tall) * TN * 4;
    {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3(pair ? 2u * (unsigned)P.slots : (unsigned)P.slots);
        cfg.blockDim = dim3(threads_tc(store_heavy));
        cfg.dynamicSmemBytes = kSmemBytes;
        cfg.stream = stream;
        cfg.attrs = at;
        cfg.numAttrs = pair ? 1 : 0;
        void *args[5] = {&map_a, &map_b, &map_f, &map_acc, &P};
        if (cudaLaunchKernelExC(&cfg, kernel_variant(pair, store_heavy, P.conv), args) != cudaSuccess) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
    }
    if (cudaGetLastError() != cudaSuccess) return CDL_ERR_LAUNCH;
    if (f_out != nullptr && (splits > 1 || slabs)) {
        const int blocks = (int)((n_out + 255) / 256 < 4096 ? (n_out + 255) / 256 : 4096);
        if (slabs)
            sum_slabs_kernel<<<blocks, 256, 0, stream>>>(P.acc_out, splits, (long long)P.slab_rows * J, f_out, n_out, J, scale, bias, P.f_acc);
        else
            scale_acc_kernel<<<blocks, 256, 0, stream>>>(P.acc_out, f_out, n_out, J, scale, bias, P.f_acc);
        if (cudaGetLastError() != cudaSuccess) return CDL_ERR_LAUNCH;
    }
    return CDL_OK;
}

}  // namespace cdl

// ------------------------------------------------------------------------------------------------
// Weight-gradient product without any caller-provided or allocated scratch (see include/cdl.h).
// The int32 accumulation buffer of the split reduction and the status word live in this file-scope
// device array.  Host code must not pass the symbol itself to a kernel: its device address is looked
// up once per device with cudaGetSymbolAddress and cached.
namespace {
constexpr size_t kStaticStatusBytes = 256;
constexpr size_t kStaticAccElems = CDL_NOALLOC_MAX_DW_ELEMS;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticStatusBytes + kStaticAccElems * sizeof(int32_t)];
std::atomic<unsigned char *> g_static_ptr[64];   // device address of g_static_scratch, per device
}  // namespace

extern "C" int cdl_qlinear_bwd_dw_noalloc(const void *G_idx, int64_t ldg, const cdl_index_desc *g, const void *A_idx,
                                          int64_t lda, const cdl_index_desc *a, int32_t M, int32_t N, int32_t K,
                                          float *dW, void *stream)
{
    using namespace cdl;
    if (G_idx == nullptr || A_idx == nullptr || dW == nullptr || g == nullptr || a == nullptr) return CDL_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || ldg < N || lda < K) return CDL_ERR_ARG;
    if ((int64_t)K * (int64_t)N > (int64_t)kStaticAccElems) return CDL_ERR_TOO_LARGE;
    if (!(g->q > 0.0f) || !(a->q > 0.0f) || g->hi < g->lo || a->hi < a->lo) return CDL_ERR_RANGE;
    if (g->lo < -128 || g->hi > 127 || a->lo < -128 || a->hi > 255 || (a->lo < 0 && a->hi > 127)) return CDL_ERR_RANGE;
    if ((ldg & 15) || (lda & 15) || (reinterpret_cast<uintptr_t>(G_idx) & 15u) || (reinterpret_cast<uintptr_t>(A_idx) & 15u) ||
        (reinterpret_cast<uintptr_t>(dW) & 3u))
        return CDL_ERR_ALIGN;
    auto absmax = [](int64_t lo, int64_t hi) {
        const int64_t x = lo < 0 ? -lo : lo, y = hi < 0 ? -hi : hi;
        return x > y ? x : y;
    };
    const int64_t amax = absmax(a->lo, a->hi), gmax = absmax(g->lo, g->hi);
    if ((int64_t)M * amax * gmax >= ((int64_t)1 << 31)) return CDL_ERR_OVERFLOW_RISK;
    int rc = check_device();
    if (rc != CDL_OK) return rc;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return CDL_ERR_LAUNCH;
    unsigned char *base = g_static_ptr[dev].load(std::memory_order_acquire);
    if (base == nullptr) {
        // one-time set-up for this device (the device is current): resolve the array's device address; threads
        // that race here all obtain the same address
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return CDL_ERR_LAUNCH;
        }
        base = static_cast<unsigned char *>(p);
        g_static_ptr[dev].store(base, std::memory_order_release);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: clear the status word here; the accumulation buffer is
    // cleared by the launcher whenever the reduction is split
    if (cudaMemsetAsync(base, 0, kStaticStatusBytes, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return CDL_ERR_LAUNCH;
    }
    GemmOperand X{A_idx, 1, lda, a->lo >= 0, (int)amax};
    GemmOperand Y{G_idx, 1, ldg, false, (int)gmax};
    return launch_index_gemm_tc(X, Y, K, N, M, nullptr, dW, g->q * a->q, nullptr, base + kStaticStatusBytes,
                                reinterpret_cast<int *>(base), st, nullptr, nullptr, false, true);
}

extern "C" int cdl_noalloc_status(void *stream)
{
    using namespace cdl;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return CDL_ERR_LAUNCH;
    unsigned char *base = g_static_ptr[dev].load(std::memory_order_acquire);
    if (base == nullptr) return CDL_OK;        // cdl_qlinear_bwd_dw_noalloc has not run on this device
    return read_status_block(base, static_cast<cudaStream_t>(stream));
}
