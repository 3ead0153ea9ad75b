// Split-KV decode attention and its log-sum-exp merge, for sm_100a.
//
// One query row per (sequence, head) against that head's cached K and V rows (the decode
// form of softmax(Q K^T / sqrt(d_k)) V, Sec. II-A / II-B; the "Logit" and "Attend"
// operators of Sec. III-B fused so that every K and V byte leaves HBM exactly once).
//
// The work is a GEMV at one flop per byte, so the kernel is built around keeping HBM busy,
// not around tensor cores:
//   * a thread block owns one chunk of logical token positions of one (sequence, head);
//   * each warp streams its own 8-token tiles of K and V through a private ring of shared
//     memory stages with no block-wide barrier in the main loop.  A tile of a contiguous or
//     paged cache is 2 KiB of K and 2 KiB of V, each one run of bytes in HBM: one lane moves
//     each with a single bulk asynchronous copy (cp.async.bulk, 1-D, this GPU's memory only)
//     that signals an mbarrier of the stage; the warp waits on it with a bounded try_wait.
//     Rows picked from a list (the sparse path) come as 16-byte cp.async copies instead;
//   * logits: 4 lanes share a key row (32 dims each, mixed-precision FMA: fp16 x fp16
//     products are exact in the fp32 accumulator; 2 xor-shuffles), so a warp scores the 8
//     rows of a tile at once.  Rows sit unpadded in shared memory; the 16-byte piece a lane
//     reads in a step is rotated by its row (piece ^ row), which spreads the 8 rows of a
//     quarter-warp over all banks, and the lane's query registers are loaded in that order.
//     The softmax reference is uniform over the warp, follows the true maximum lazily, and
//     each row's exponential (base 2, fp32) is computed once;
//   * weighted sum: 16 lanes share a value row (8 dims each), the half-warps take alternate
//     rows and fetch the row's weight (split into two fp16 parts) with one shuffle;
//   * rows come from a contiguous cache, from paged pools through the block table, or from
//     a list of selected rows (the sparse path);
//   * the 4 warp states of a block are merged once at the end of the chunk; chunk partials
//     go to the workspace and a small second kernel merges them.  Small problems (at most 8
//     chunks per sequence, about one wave of blocks) skip both: the chunks of a (sequence,
//     head) form one thread-block cluster, each block leaves its partial in its own shared
//     memory, and after a cluster barrier the first block merges them through distributed
//     shared memory and writes the row -- one launch less and no round trip through HBM.
#pragma once

#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace instinfer {

constexpr int kHeadDim = 128;                      // the paper's head size (Sec. IV-C)
constexpr int kRowBytes = kHeadDim * 2;            // one token's K (or V) row of one head
constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 8;                       // tokens per warp tile
constexpr int kStages = 3;                         // ring depth per warp
constexpr int kKTileBytes = kTileRows * kRowBytes;  // rows unpadded: a tile is one run of bytes
constexpr int kVTileBytes = kTileRows * kRowBytes;
constexpr int kStageBytes = kKTileBytes + kVTileBytes;
constexpr int kRingBytes = kWarps * kStages * kStageBytes;        // 48 KiB
constexpr int kSplitSmemBytes = kRingBytes + kWarps * kStages * 8; // + one mbarrier per stage
constexpr int kCtasPerSm = 4;
constexpr float kMinusHuge = -1.0e30f;             // finite stand-in for "no row seen yet"
constexpr float kLn2 = 0.69314718055994530942f;

constexpr int kFlagSeqLenRange = 1;
constexpr int kFlagBlockRange = 2;
constexpr int kFlagCopyTimeout = 4;
constexpr int kFlagBoundsCheck = 8;

// Bounds-checking build (-DINSTINFER_BOUNDS_CHECK): every data-dependent global offset that a
// kernel computes (from a block table, a length, a row list) is tested against the extent
// that the call's shapes imply before it is used; a violation sets kFlagBoundsCheck in the
// status word and the access is skipped.  It stands in for a memory checker: in a correct
// library the bit never appears.  In the ordinary build the test compiles to nothing.
#ifdef INSTINFER_BOUNDS_CHECK
__device__ __forceinline__ bool bounds_ok(bool inside, int32_t *status)
{
    if (!inside && status) atomicOr(status, kFlagBoundsCheck);
    return inside;
}
#else
__device__ __forceinline__ bool bounds_ok(bool, int32_t *) { return true; }
#endif

struct AttnParams {
    const __half *q;
    const __half *k;
    const __half *v;
    const int32_t *seq_lens;
    const int32_t *block_table;
    float *part_o;        // [pairs, n_splits, kHeadDim], each already divided by its own sum
    float *part_lse;      // [pairs, n_splits], base-2 log-sum-exp of the chunk
    __half *out;          // [pairs, kHeadDim]
    float *lse;           // [pairs], nullable, natural log
    int32_t *status;      // nullable
    int64_t num_phys_blocks;
    int32_t heads;
    int32_t pairs;        // batch * heads
    int32_t s_max;
    int32_t block_tokens;
    int32_t max_blocks_per_seq;
    int32_t chunk_tokens; // tokens per long chunk; the long chunks follow the short ones ...
    int32_t n_big;        // number of long chunks
    int32_t tail_chunk;   // ... tokens per short chunk: the first n_splits - n_big chunks of every
                          // sequence (scheduled last, so that every launch ends on short blocks)
    int32_t n_splits;     // short chunks + long chunks
    int32_t max_seq_len;
    float scale_log2e;    // scale * log2(e): logits are kept in the base-2 domain
    // gathered mode only (sparse attention over a list of selected rows):
    const int32_t *row_ids;    // [pairs, row_stride] physical row index (phys * H + h) * T + slot
    const int32_t *k_tokens;   // [batch] rows to attend per sequence (clipped to its length)
    int32_t row_stride;
    int32_t row_limit;         // number of rows in the pools: a listed id outside [0, row_limit) reads as zeros
    int64_t kv_bytes;          // bytes of the K cache (= of the V cache) that the call's shapes imply
};

// Where a (sequence, head)'s rows come from.
enum class Rows { kContiguous, kPaged, kGathered };

// Programmatic dependent launch: a kernel first lets the next kernel in the stream start
// being scheduled, then waits until the kernels before it have completed and their writes
// are visible.  Both are no-ops for a launch without the attribute.
__device__ __forceinline__ void allow_next_kernel() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void wait_for_previous_kernels() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void cp_async_16(unsigned dst, const void *gmem_src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16, %2;\n"
                 :: "r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" :: "n"(kPending) : "memory"); }

// Bulk asynchronous copies (global -> this block's shared memory) completing on an mbarrier.
// Addresses are 16-byte aligned and sizes multiples of 16 bytes by construction (256-byte rows).
__device__ __forceinline__ void mbarrier_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbarrier_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbarrier_expect_bytes(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// One attempt: the thread may be parked by the hardware until the phase completes or a time
// limit passes (the hint, in nanoseconds, asks for a long one, so that a warp that waits for
// data sleeps instead of spinning through issue slots).
__device__ __forceinline__ bool mbarrier_try_wait(unsigned bar, unsigned parity)
{
    unsigned done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(1000000u) : "memory");
    return done != 0;
}
// Waits for phase `parity` of the barrier, giving up after about kWaitCycles clock cycles (a
// copy of a few KiB completes in microseconds: running out means the hardware has a problem,
// and the kernel must end rather than hang).
constexpr long long kWaitCycles = 4000000000ll;
__device__ __forceinline__ bool mbarrier_wait_bounded(unsigned bar, unsigned parity)
{
    if (mbarrier_try_wait(bar, parity)) return true;
    const long long start = clock64();
    for (;;) {
        if (mbarrier_try_wait(bar, parity)) return true;
        if (clock64() - start > kWaitCycles) return false;
    }
}

// Sequence length as the kernels see it: out-of-range lengths make the slot inactive.
__device__ __forceinline__ int checked_seq_len(const AttnParams &p, int b, bool report)
{
    int len = p.seq_lens[b];
    if (len < 0 || len > p.max_seq_len) {
        if (report && p.status) atomicOr(p.status, kFlagSeqLenRange);
        len = 0;
    }
    return len;
}

// Gathered mode: number of listed rows of sequence b (its k, clipped to its length and to the list).
__device__ __forceinline__ int gathered_count(const AttnParams &p, int b, int len)
{
    return min(len, min(max(p.k_tokens[b], 0), p.row_stride));
}

// The split plan.  A sequence is cut at fixed logical positions, the same for every sequence:
// first n_short = n_splits - n_big short chunks of tail_chunk tokens, then n_big long chunks of
// chunk_tokens.  Chunks are numbered by position (that is also the order of the merge); the
// grid runs the long chunks first and the short ones last.  Every sequence of a ragged batch
// has its first tokens, so the last waves of a launch are made of many short blocks whatever
// the lengths are, instead of a few long blocks at the ends of the longest sequences.

// Logical token range [begin, begin + size) of chunk `split`.
__device__ __forceinline__ void chunk_range(const AttnParams &p, int split, int &begin, int &size)
{
    const int n_short = p.n_splits - p.n_big;
    if (split < n_short) {
        begin = split * p.tail_chunk;
        size = p.tail_chunk;
    } else {
        begin = n_short * p.tail_chunk + (split - n_short) * p.chunk_tokens;
        size = p.chunk_tokens;
    }
}

// The chunk that the `order`-th group of blocks of the grid works on: long chunks first.
__device__ __forceinline__ int scheduled_chunk(const AttnParams &p, int order)
{
    return order < p.n_big ? p.n_splits - p.n_big + order : order - p.n_big;
}

// Number of chunks of a sequence of `len` tokens that hold at least one token.
__device__ __forceinline__ int live_chunks(const AttnParams &p, int len)
{
    const int n_short = p.n_splits - p.n_big;
    const int short_span = n_short * p.tail_chunk;
    if (len <= short_span) return (len + p.tail_chunk - 1) / p.tail_chunk;
    return n_short + (len - short_span + p.chunk_tokens - 1) / p.chunk_tokens;
}

// d = a * b + c with fp16 a, b and fp32 c, d: the product of two fp16 values is exact in
// fp32, so this is one rounding, and one full-rate instruction with no conversion.
__device__ __forceinline__ float fma_h(unsigned short a, unsigned short b, float c)
{
    float d;
    asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
    return d;
}

__device__ __forceinline__ void halves(unsigned packed, unsigned short &lo, unsigned short &hi)
{
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(packed));
}

// A softmax weight w in [0, 2] as two fp16 numbers hi + lo ~ w * 2^14 (packed lo | hi << 16).
// The scaling keeps weights down to 2^-38 of the maximum representable; hi + lo carries
// about 22 significant bits, the precision of the exponential itself.
constexpr float kWeightScale = 16384.f;
constexpr float kMaxLag = 1.f;          // weights <= 2, so weight * kWeightScale <= 32768 < 65504
__device__ __forceinline__ unsigned split_weight(float w)
{
    const float scaled = w * kWeightScale;
    const __half hi = __float2half_rn(scaled);
    const __half lo = __float2half_rn(scaled - __half2float(hi));
    return (unsigned)__half_as_ushort(hi) << 16 | (unsigned)__half_as_ushort(lo);
}

__device__ __forceinline__ void unpack8(const uint4 &raw, float (&f)[8])
{
    const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __half22float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

__device__ __forceinline__ uint4 lds128(unsigned shared_addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(shared_addr));
    return v;
}

// One 8-token tile of one warp: logits of the 8 key rows, online softmax update, weighted sum
// of the 8 value rows.  k_row / v_seg are this lane's shared-memory addresses inside the tile
// (row `row` of K; the lane's 16-byte segment of V rows 0 and 1), k_piece its four rotated
// 16-byte pieces of the key row, qh the query dims that go with them.  m is the warp-uniform
// softmax reference, l this lane's partial sum of weights, acc its 8 output dims (scaled by
// kWeightScale); rows < 8 masks the rows past the end of the chunk.
__device__ __forceinline__ void attend_tile(unsigned k_row, const unsigned (&k_piece)[4], unsigned v_seg,
                                            const uint4 (&qh)[4], float scale_log2e, int rows, int row,
                                            int half_warp, float &m, float &l, float (&acc)[8])
{
    // Logit: this lane's quarter of row `row`, four independent fp32 chains.
    float part[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 kr = lds128(k_row + k_piece[i]);
        const unsigned kw[4] = {kr.x, kr.y, kr.z, kr.w};
        const unsigned qw[4] = {qh[i].x, qh[i].y, qh[i].z, qh[i].w};
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            unsigned short k0, k1, q0, q1;
            halves(kw[e], k0, k1);
            halves(qw[e], q0, q1);
            dot = fma_h(k0, q0, dot);
            dot = fma_h(k1, q1, dot);
        }
        part[i] = dot;
    }
    float s = ((part[0] + part[1]) + (part[2] + part[3])) * scale_log2e;
    s += __shfl_xor_sync(0xffffffffu, s, 8);
    s += __shfl_xor_sync(0xffffffffu, s, 16);
    if (row >= rows) s = -INFINITY;

    // Online softmax with a warp-uniform reference m that may lag the true maximum by up to
    // kMaxLag (base-2 units): weights then reach at most 2^kMaxLag, which is harmless in
    // fp32 and inside the range of the fp16 weight split.  The reference only moves (and
    // the accumulators are only rescaled) when some logit exceeds it by more than that,
    // so the common tile pays one vote instead of a shuffle reduction.
    if (__any_sync(0xffffffffu, s > m + kMaxLag)) {
        float tile_max = s;
        tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 1));
        tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 2));
        tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 4));
        const float alpha = fast_exp2(m - tile_max);
        l *= alpha;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] *= alpha;
        m = tile_max;
    }
    const float pw = fast_exp2(s - m);
    l += pw;

    // Attend: rows 2 r + half_warp, r < 4.
    const unsigned packed = split_weight(pw);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        unsigned short w_lo, w_hi;
        halves(__shfl_sync(0xffffffffu, packed, 2 * r + half_warp), w_lo, w_hi);
        const uint4 vr = lds128(v_seg + r * 512);
        const unsigned vw[4] = {vr.x, vr.y, vr.z, vr.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            unsigned short v0, v1;
            halves(vw[e], v0, v1);
            acc[2 * e] = fma_h(v0, w_hi, acc[2 * e]);
            acc[2 * e + 1] = fma_h(v1, w_hi, acc[2 * e + 1]);
            acc[2 * e] = fma_h(v0, w_lo, acc[2 * e]);
            acc[2 * e + 1] = fma_h(v1, w_lo, acc[2 * e + 1]);
        }
    }
}

// kCluster: the grid is pair-major and launched with clusters of n_splits blocks (the chunks of
// one (sequence, head)); the merge happens inside the kernel (see the file header).
template <Rows kRows, bool kCluster = false>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
decode_attn_split_kernel(const AttnParams p)
{
    static_assert(!(kCluster && kRows == Rows::kGathered), "row lists use the two-kernel form");
    constexpr bool kPaged = kRows == Rows::kPaged;
    constexpr bool kGathered = kRows == Rows::kGathered;
    constexpr bool kBulk = !kGathered;                   // whole tiles by one bulk copy each
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kStepTokens = kWarps * kTileRows;      // a warp's next tile is this far ahead
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Logit phase: 4 lanes per key row, lane (row = lane & 7, quarter = lane >> 3) owns 32 dims.
    // Attend phase: 16 lanes per value row, lane (col = lane & 15) owns 8 dims, half-warps
    // take alternate rows.
    const int row = lane & 7, quarter = lane >> 3;
    const int col = lane & 15, half_warp = lane >> 4;
    // Grid order: chunk slowest (long chunks first, short ones last), then sequence, head
    // fastest.  Blocks that run together then cover all heads of a few sequences (one paged
    // block's heads are adjacent in memory).
    const int order = kCluster ? (int)(blockIdx.x % p.n_splits) : (int)(blockIdx.x / p.pairs);
    const int pair = kCluster ? (int)(blockIdx.x / p.n_splits) : (int)(blockIdx.x - order * p.pairs);
    const int split = kCluster ? order : scheduled_chunk(p, order);      // cluster rank = chunk in position order
    const int b = pair / p.heads, h = pair - b * p.heads;
    const bool final_writer = !kGathered && !kCluster && p.n_splits == 1;
    // one mbarrier per stage, behind the rings: a stage's bulk copies report their bytes to it
    const unsigned bars = static_cast<unsigned>(__cvta_generic_to_shared(smem)) + kRingBytes + warp * (kStages * 8);
    if (kBulk && lane == 0) {                            // each warp owns the barriers of its ring
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbarrier_init(bars + s * 8, 1);
        mbarrier_init_fence();
    }
    allow_next_kernel();
    wait_for_previous_kernels();

    // With several splits the merge kernel reports a bad length; here only the lone writer does.
    // (the block that writes the final rows reports a bad length: the lone writer, or the
    // first block of a cluster)
    int len = checked_seq_len(p, b, threadIdx.x == 0 && h == 0 && (final_writer || (kCluster && split == 0)));
    if (kGathered) len = gathered_count(p, b, len);           // rows in this pair's list
    int begin, chunk_size;
    chunk_range(p, split, begin, chunk_size);
    if (!kCluster && begin >= len) {
        if (final_writer) {            // inactive slot: zero output, lse = -inf
            p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(0.f);
            if (p.lse && threadIdx.x == 0) p.lse[pair] = -INFINITY;
        }
        return;
    }
    const int end = min(begin + chunk_size, len);
    const int n_tiles = end > begin ? (end - begin + kTileRows - 1) / kTileRows : 0;   // 0: an empty chunk of a cluster
    const int my_tiles = warp < n_tiles ? (n_tiles - warp + kWarps - 1) / kWarps : 0;
    // Only the chunk's very last tile can be ragged; it belongs to exactly one warp.
    const int last_rows = n_tiles > 0 && warp == (n_tiles - 1) % kWarps ? (end - begin) - (n_tiles - 1) * kTileRows
                                                                        : kTileRows;

    // This lane's 32 query dims, kept in fp16 (16 registers): products with fp16 keys are
    // exact in fp32 and the scale is applied to the finished dot product.  In step i the lane
    // reads the 16-byte piece (4 quarter + i) ^ row of its key row (see k_rd below), so its
    // query registers are loaded in that order.
    uint4 qh[4];
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.q + (int64_t)pair * kHeadDim);
#pragma unroll
        for (int i = 0; i < 4; ++i) qh[i] = src[(quarter * 4 + i) ^ row];
    }

    // Shared-memory addresses (shared window, 32 bit).
    const unsigned ring = static_cast<unsigned>(__cvta_generic_to_shared(smem)) +
                          warp * (kStages * kStageBytes);
    // cp.async copies: 16-byte segment lane + 32 i, i < 4, lies in row 2 i + half_warp at column segment col
    const unsigned k_dst = half_warp * kRowBytes + col * 16;
    const unsigned v_dst = kKTileBytes + lane * 16;
    // The 8 lanes of a quarter-warp read one piece each of rows 0..7 in the same step; rows are
    // 256 bytes apart (the same banks), so the piece index is rotated by the row: 8 distinct
    // 16-byte bank groups, no conflict.
    const unsigned k_rd = row * kRowBytes;
    unsigned k_piece[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) k_piece[i] = (((quarter * 4 + i) ^ row) & 15) * 16;
    const unsigned v_rd = kKTileBytes + lane * 16;

    // ---- copy-issue side: walks this warp's tiles incrementally (no division per tile) ----
    const unsigned char *k_base = reinterpret_cast<const unsigned char *>(p.k);
    const unsigned char *v_base = reinterpret_cast<const unsigned char *>(p.v);
    const int first_token = begin + warp * kTileRows;
    int64_t src_off = 0;                       // contiguous: byte offset of the next tile
    int blk = 0, rem = 0, win_base = 0;        // paged: block index, row inside it, window start
    int window_now = 0, window_next = 0;       // block-table entries win_base + lane (+ 32)
    int64_t block_stride = 0, head_off = 0;
    int step_blk = 0, step_rem = 0, blocks_needed = 0;
    const int32_t *table_row = nullptr;
    // gathered: row ids of this warp's next 4 tiles, one per lane (tile = lane >> 3, row = lane & 7)
    const int32_t *row_list = kGathered ? p.row_ids + (int64_t)pair * p.row_stride : nullptr;
    int rows_now = 0, rows_next = 0;
    auto load_rows = [&](int tile_base) -> int {
        const int idx = begin + (warp + (tile_base + (lane >> 3)) * kWarps) * kTileRows + (lane & 7);
        return idx < end ? __ldg(row_list + idx) : 0;
    };
    if (kGathered) {
        if (my_tiles > 0) {
            rows_now = load_rows(0);
            rows_next = load_rows(4);
        }
    } else if (kPaged) {
        const int tokens = p.block_tokens;
        table_row = p.block_table + (int64_t)b * p.max_blocks_per_seq;
        blocks_needed = (end + tokens - 1) / tokens;
        blk = first_token / tokens;
        rem = first_token - blk * tokens;
        step_blk = kStepTokens / tokens;
        step_rem = kStepTokens - step_blk * tokens;
        block_stride = (int64_t)p.heads * tokens * kRowBytes;
        head_off = (int64_t)h * tokens * kRowBytes;
        win_base = blk;
    } else {
        src_off = ((int64_t)pair * p.s_max + first_token) * kRowBytes;
    }
    auto load_window = [&](int base) -> int {
        const int idx = base + lane;
        if (idx >= blocks_needed || !bounds_ok(idx < p.max_blocks_per_seq, p.status)) return 0;
        return __ldg(table_row + idx);
    };
    if (kPaged && my_tiles > 0) {
        window_now = load_window(win_base);
        window_next = load_window(win_base + 32);
    }

    int issue_j = 0;
    unsigned issue_stage = 0;
    auto issue = [&]() {
        if (issue_j < my_tiles) {
            const int rows = issue_j == my_tiles - 1 ? last_rows : kTileRows;
            const unsigned dst = ring + issue_stage * kStageBytes;
            if (kGathered) {
                if ((issue_j & 3) == 0 && issue_j > 0) {       // uniform: next window of 4 tiles
                    rows_now = rows_next;
                    rows_next = load_rows(issue_j + 4);
                }
                const unsigned char *k_col = k_base + col * 16;
                const unsigned char *v_col = v_base + col * 16;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int rid = __shfl_sync(0xffffffffu, rows_now, (issue_j & 3) * 8 + 2 * i + half_warp);
                    const bool valid = 2 * i + half_warp < rows && (unsigned)rid < (unsigned)p.row_limit;
                    const int64_t src = valid ? (int64_t)rid * kRowBytes : 0;
                    cp_async_16(dst + k_dst + i * 2 * kRowBytes, k_col + src, valid ? 16 : 0);
                    cp_async_16(dst + v_dst + i * 512, v_col + src, valid ? 16 : 0);
                }
            } else {
                bool usable = true;
                int64_t off;
                if (kPaged) {
                    int idx = blk - win_base;
                    if (idx >= 32) {               // uniform: slide the window of table entries
                        idx -= 32;
                        win_base += 32;
                        window_now = window_next;
                        window_next = load_window(win_base + 32);
                    }
                    const int phys = __shfl_sync(0xffffffffu, window_now, idx);
                    usable = phys >= 0 && (int64_t)phys < p.num_phys_blocks;
                    if (!usable && lane == 0 && p.status) atomicOr(p.status, kFlagBlockRange);
                    off = usable ? (int64_t)phys * block_stride + head_off + rem * kRowBytes : 0;
                    blk += step_blk;
                    rem += step_rem;
                    if (rem >= p.block_tokens) {
                        rem -= p.block_tokens;
                        ++blk;
                    }
                } else {
                    off = src_off;
                    src_off += kStepTokens * kRowBytes;
                }
                // The tile's rows are one run of bytes in the cache (a tile never straddles a
                // block: block_tokens is a multiple of the tile).  Rows past the chunk's end and
                // the rows of a block with a bad id are not fetched; their value slots are
                // zeroed (their weights are zero, but 0 x stale bits must not be NaN) and their
                // logits are masked below.
                usable = usable && bounds_ok(off >= 0 && off + rows * kRowBytes <= p.kv_bytes, p.status);
                const int fetch = usable ? rows : 0;
                if (fetch < kTileRows) {
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    for (int seg = fetch * 16 + lane; seg < kTileRows * 16; seg += 32) {
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                                     :: "r"(dst + kKTileBytes + seg * 16), "r"(zero.x), "r"(zero.y), "r"(zero.z), "r"(zero.w) : "memory");
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                                     :: "r"(dst + seg * 16), "r"(zero.x), "r"(zero.y), "r"(zero.z), "r"(zero.w) : "memory");
                    }
                    __syncwarp();
                }
                if (lane == 0) {
                    const unsigned bar = bars + issue_stage * 8;
                    const unsigned bytes = (unsigned)fetch * kRowBytes;
                    mbarrier_expect_bytes(bar, 2 * bytes);
                    if (fetch > 0) {
                        bulk_copy(dst, k_base + off, bytes, bar);
                        bulk_copy(dst + kKTileBytes, v_base + off, bytes, bar);
                    }
                }
            }
        }
        if (kGathered) cp_async_commit();                      // empty groups keep the count uniform
        ++issue_j;
        issue_stage = issue_stage + 1 == kStages ? 0 : issue_stage + 1;
    };

    // Running softmax state.  m is uniform over the warp; l is a per-lane partial sum (lanes
    // of one row hold equal values); acc covers this half-warp's rows and carries kWeightScale.
    float m = kMinusHuge, l = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;

    if (kBulk) __syncwarp();             // the barriers are initialised before the first copy
#pragma unroll
    for (int j = 0; j < kStages - 1; ++j) issue();

    unsigned stage = 0, phase = 0;
    bool stalled = false;
    for (int j = 0; j < my_tiles; ++j) {
        if (kGathered) {
            cp_async_wait<kStages - 2>();
        } else if (!__all_sync(0xffffffffu, mbarrier_wait_bounded(bars + stage * 8, phase))) {
            stalled = true;              // one decision for the whole warp
            break;
        }
        __syncwarp();                    // tile j visible to the warp; everyone is done with tile j-1
        issue();                         // refills the slot tile j-1 used
        const unsigned base = ring + stage * kStageBytes;
        if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
        }

        const int rows = j == my_tiles - 1 ? last_rows : kTileRows;
        attend_tile(base + k_rd, k_piece, base + v_rd, qh, p.scale_log2e, rows, row, half_warp, m, l, acc);
    }
    if (kGathered) cp_async_wait<0>();
    if (kBulk && stalled) {
        // A copy did not arrive in time.  Report it, give the copies still in flight one more
        // bounded chance to land (shared memory must not be handed on while they are pending)
        // and leave; this block's partial result stays unwritten and the call's output is
        // undefined, which the flag tells the caller.
        if (lane == 0 && p.status) atomicOr(p.status, kFlagCopyTimeout);
        const int issued = min(issue_j, my_tiles);
        for (int t = issued - min(issued, kStages - 1); t < issued; ++t)
            (void)mbarrier_wait_bounded(bars + (t % kStages) * 8, (t / kStages) & 1);
    }
    // (a block barrier follows: a stalled warp still joins it, then contributes an empty state)
    if (kBulk && stalled) {
        m = kMinusHuge;
        l = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    }

    // One state per warp: sum l over the 8 rows, fold the two half-warps' accumulators.
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    l += __shfl_xor_sync(0xffffffffu, l, 4);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
    __syncthreads();                     // every ring is idle: reuse shared memory for the merge

    float *sm_m = reinterpret_cast<float *>(smem);
    float *sm_l = sm_m + kWarps;
    float *sm_acc = sm_l + kWarps;                       // [kWarps][kHeadDim]
    if (lane == 0) {
        sm_m[warp] = m;
        sm_l[warp] = l;
    }
    if (half_warp == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) sm_acc[warp * kHeadDim + col * 8 + i] = acc[i];
    }
    __syncthreads();

    float top = kMinusHuge;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) top = fmaxf(top, sm_m[i]);
    float total = 0.f, o = 0.f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
        const float w = fast_exp2(sm_m[i] - top);
        total = fmaf(w, sm_l[i], total);
        o = fmaf(w, sm_acc[i * kHeadDim + threadIdx.x], o);
    }
    o /= total * kWeightScale;
    float lse2 = top + log2f(total);
    if (kCluster) {
        // This chunk's partial stays in this block's shared memory (behind the fold's scratch);
        // block 0 of the cluster merges all of them in position order, exactly as
        // lse_merge_kernel would, and writes the row.  Every block stays until that is done.
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        float *mine = reinterpret_cast<float *>(smem) + kWarps * (kHeadDim + 2);       // [kHeadDim] + lse
        if (n_tiles == 0) {              // empty chunk: nothing to contribute (total is 0 here)
            o = 0.f;
            lse2 = -INFINITY;
        }
        mine[threadIdx.x] = o;
        if (threadIdx.x == 0) mine[kHeadDim] = lse2;
        cluster.sync();
        if (split == 0) {
            const int live = live_chunks(p, len);
            if (live == 0) {
                p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(0.f);
                if (p.lse && threadIdx.x == 0) p.lse[pair] = -INFINITY;
            } else {
                float best = kMinusHuge;
                for (int s = 0; s < live; ++s) best = fmaxf(best, cluster.map_shared_rank(mine, s)[kHeadDim]);
                float weight_sum = 0.f, merged = 0.f;
                for (int s = 0; s < live; ++s) {
                    const float *theirs = cluster.map_shared_rank(mine, s);
                    const float w = fast_exp2(theirs[kHeadDim] - best);
                    weight_sum += w;
                    merged = fmaf(w, theirs[threadIdx.x], merged);
                }
                p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(merged / weight_sum);
                if (p.lse && threadIdx.x == 0) p.lse[pair] = (best + log2f(weight_sum)) * kLn2;
            }
        }
        cluster.sync();                  // no block's shared memory goes away while block 0 reads it
        return;
    }
    if (final_writer) {
        p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(o);
        if (p.lse && threadIdx.x == 0) p.lse[pair] = lse2 * kLn2;
    } else {
        const int64_t slot = (int64_t)pair * p.n_splits + split;
        p.part_o[slot * kHeadDim + threadIdx.x] = o;
        if (threadIdx.x == 0) p.part_lse[slot] = lse2;
    }
}

// Log-sum-exp merge of the chunk partials of one (sequence, head); one block per pair,
// one thread per output dim.  Only the chunks that hold tokens are read.
__global__ void __launch_bounds__(kHeadDim)
lse_merge_kernel(const AttnParams p)
{
    const int pair = blockIdx.x;
    const int b = pair / p.heads;
    allow_next_kernel();
    wait_for_previous_kernels();
    const int len = checked_seq_len(p, b, threadIdx.x == 0 && pair == b * p.heads);
    const int live = live_chunks(p, len);
    if (live == 0) {
        p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(0.f);
        if (p.lse && threadIdx.x == 0) p.lse[pair] = -INFINITY;
        return;
    }
    const float *lse2 = p.part_lse + (int64_t)pair * p.n_splits;
    const float *po = p.part_o + (int64_t)pair * p.n_splits * kHeadDim + threadIdx.x;
    float top = kMinusHuge;
    for (int s = 0; s < live; ++s) top = fmaxf(top, lse2[s]);
    float total = 0.f, o = 0.f;
    for (int s = 0; s < live; ++s) {
        const float w = fast_exp2(lse2[s] - top);
        total += w;
        o = fmaf(w, po[(int64_t)s * kHeadDim], o);
    }
    p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(o / total);
    if (p.lse && threadIdx.x == 0) p.lse[pair] = (top + log2f(total)) * kLn2;
}

}  // namespace instinfer
