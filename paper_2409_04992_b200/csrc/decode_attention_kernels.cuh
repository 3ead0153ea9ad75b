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
//     memory stages filled by 16-byte cp.async copies (coalesced 512 B per warp instruction),
//     with no block-wide barrier and no spin-wait anywhere in the main loop;
//   * a half-warp (16 lanes x 8 dims) owns one row at a time: dot product in fp32, a 4-step
//     shuffle reduction, then an fp32 online softmax (base-2 exponent) and the p.V update;
//   * the 8 half-warp states of a block are merged once at the end of the chunk; chunk
//     partials go to the workspace and a small second kernel merges them.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace instinfer {

constexpr int kHeadDim = 128;                      // the paper's head size (Sec. IV-C)
constexpr int kRowBytes = kHeadDim * 2;            // one token's K (or V) row of one head
constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 8;                       // tokens per warp tile
constexpr int kStages = 4;                         // ring depth per warp
constexpr int kTileBytes = kTileRows * kRowBytes;  // 2 KiB of K, same of V
constexpr int kStageBytes = 2 * kTileBytes;
constexpr int kSplitSmemBytes = kWarps * kStages * kStageBytes;   // 64 KiB
constexpr int kCtasPerSm = 3;
constexpr float kMinusHuge = -1.0e30f;             // finite stand-in for "no row seen yet"
constexpr float kLn2 = 0.69314718055994530942f;

constexpr int kFlagSeqLenRange = 1;
constexpr int kFlagBlockRange = 2;

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
    int32_t chunk_tokens; // tokens per chunk for the first n_big chunks of a sequence ...
    int32_t n_big;
    int32_t tail_chunk;   // ... and per chunk after that (scheduled last: short tail of the launch)
    int32_t n_splits;     // n_big + number of tail chunks
    int32_t max_seq_len;
    float scale_log2e;    // scale * log2(e): logits are kept in the base-2 domain
};

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gmem_src, int src_bytes)
{
    const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16, %2;\n"
                 :: "r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" :: "n"(kPending) : "memory"); }

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

// Logical token range [begin, begin + size) of chunk `split`.
__device__ __forceinline__ void chunk_range(const AttnParams &p, int split, int &begin, int &size)
{
    if (split < p.n_big) {
        begin = split * p.chunk_tokens;
        size = p.chunk_tokens;
    } else {
        begin = p.n_big * p.chunk_tokens + (split - p.n_big) * p.tail_chunk;
        size = p.tail_chunk;
    }
}

// Number of chunks of a sequence of `len` tokens that hold at least one token.
__device__ __forceinline__ int live_chunks(const AttnParams &p, int len)
{
    const int big_span = p.n_big * p.chunk_tokens;
    if (len <= big_span) return (len + p.chunk_tokens - 1) / p.chunk_tokens;
    return p.n_big + (len - big_span + p.tail_chunk - 1) / p.tail_chunk;
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

template <bool kPaged>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
decode_attn_split_kernel(const AttnParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = lane & 15, half_warp = lane >> 4;
    // Grid order: split slowest, then sequence, head fastest.  Blocks that run together then
    // cover all heads of a few sequences (one paged block's heads are adjacent in memory),
    // and the short last chunks of ragged sequences are scheduled last.
    const int split = blockIdx.x / p.pairs;
    const int pair = blockIdx.x - split * p.pairs;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const bool final_writer = p.n_splits == 1;

    // With several splits the merge kernel reports a bad length; here only the lone writer does.
    const int len = checked_seq_len(p, b, threadIdx.x == 0 && h == 0 && final_writer);
    int begin, chunk_size;
    chunk_range(p, split, begin, chunk_size);
    if (begin >= len) {
        if (final_writer) {            // inactive slot: zero output, lse = -inf
            p.out[(int64_t)pair * kHeadDim + threadIdx.x] = __float2half_rn(0.f);
            if (p.lse && threadIdx.x == 0) p.lse[pair] = -INFINITY;
        }
        return;
    }
    const int end = min(begin + chunk_size, len);
    const int n_tiles = (end - begin + kTileRows - 1) / kTileRows;
    const int my_tiles = warp < n_tiles ? (n_tiles - warp + kWarps - 1) / kWarps : 0;

    // This lane's 8 query dims, pre-multiplied by scale*log2(e).
    float qf[8];
    {
        const uint4 raw = *reinterpret_cast<const uint4 *>(p.q + (int64_t)pair * kHeadDim + col * 8);
        unpack8(raw, qf);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[i] *= p.scale_log2e;
    }

    unsigned char *ring = smem + warp * (kStages * kStageBytes);
    const int64_t contiguous_base = (int64_t)pair * p.s_max;          // rows
    const int32_t *table_row = kPaged ? p.block_table + (int64_t)b * p.max_blocks_per_seq : nullptr;

    // Block-table entries for this warp's next 32 tiles live one per lane (paged only).
    auto table_entry = [&](int j) -> int {
        if (j >= my_tiles) return 0;
        const int token0 = begin + (warp + j * kWarps) * kTileRows;
        return __ldg(table_row + token0 / p.block_tokens);
    };
    int table_now = 0, table_next = 0;
    if (kPaged) {
        table_now = table_entry(lane);
        table_next = table_entry(32 + lane);
    }

    auto issue = [&](int j) {
        if (j < my_tiles) {
            const int token0 = begin + (warp + j * kWarps) * kTileRows;
            int64_t row0;
            bool usable = true;
            if (kPaged) {
                if ((j & 31) == 0 && j > 0) {
                    table_now = table_next;
                    table_next = table_entry(j + 32 + lane);
                }
                const int phys = __shfl_sync(0xffffffffu, table_now, j & 31);
                usable = phys >= 0 && (int64_t)phys < p.num_phys_blocks;
                if (!usable && lane == 0 && p.status) atomicOr(p.status, kFlagBlockRange);
                row0 = usable ? ((int64_t)phys * p.heads + h) * p.block_tokens + token0 % p.block_tokens : 0;
            } else {
                row0 = contiguous_base + token0;
            }
            const unsigned char *k_src = reinterpret_cast<const unsigned char *>(p.k) + row0 * kRowBytes;
            const unsigned char *v_src = reinterpret_cast<const unsigned char *>(p.v) + row0 * kRowBytes;
            unsigned char *dst = ring + (j % kStages) * kStageBytes;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int seg = lane + 32 * i;                 // 16-byte segment of the tile
                const bool valid = usable && (token0 + (seg >> 4) < end);
                const int off = valid ? seg * 16 : 0;          // masked rows are zero-filled
                cp_async_16(dst + seg * 16, k_src + off, valid ? 16 : 0);
                cp_async_16(dst + kTileBytes + seg * 16, v_src + off, valid ? 16 : 0);
            }
        }
        cp_async_commit();                                     // empty groups keep the count uniform
    };

    float m = kMinusHuge, l = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;

#pragma unroll
    for (int j = 0; j < kStages - 1; ++j) issue(j);

    for (int j = 0; j < my_tiles; ++j) {
        cp_async_wait<kStages - 2>();
        __syncwarp();                    // tile j visible to the warp; everyone is done with tile j-1
        issue(j + kStages - 1);          // refills the slot tile j-1 used

        const unsigned char *stage = ring + (j % kStages) * kStageBytes;
        const int token0 = begin + (warp + j * kWarps) * kTileRows;
        float s[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            float kf[8];
            unpack8(*reinterpret_cast<const uint4 *>(stage + r * 512 + lane * 16), kf);
            float dot = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) dot = fmaf(kf[i], qf[i], dot);
            s[r] = dot;
        }
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
#pragma unroll
            for (int r = 0; r < 4; ++r) s[r] += __shfl_xor_sync(0xffffffffu, s[r], off);
        }
        float m_new = m;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (token0 + 2 * r + half_warp >= end) s[r] = -INFINITY;
            m_new = fmaxf(m_new, s[r]);
        }
        const float alpha = fast_exp2(m - m_new);
        float pw[4], psum = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            pw[r] = fast_exp2(s[r] - m_new);
            psum += pw[r];
        }
        l = fmaf(l, alpha, psum);
        m = m_new;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] *= alpha;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            float vf[8];
            unpack8(*reinterpret_cast<const uint4 *>(stage + kTileBytes + r * 512 + lane * 16), vf);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(pw[r], vf[i], acc[i]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();                     // every ring is idle: reuse shared memory for the merge

    // Merge the 8 half-warp states of this block.
    constexpr int kStates = 2 * kWarps;
    float *sm_m = reinterpret_cast<float *>(smem);
    float *sm_l = sm_m + kStates;
    float *sm_acc = sm_l + kStates;                      // [kStates][kHeadDim]
    const int state = warp * 2 + half_warp;
    if (col == 0) {
        sm_m[state] = m;
        sm_l[state] = l;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) sm_acc[state * kHeadDim + col * 8 + i] = acc[i];
    __syncthreads();

    float top = kMinusHuge;
#pragma unroll
    for (int i = 0; i < kStates; ++i) top = fmaxf(top, sm_m[i]);
    float total = 0.f, o = 0.f;
#pragma unroll
    for (int i = 0; i < kStates; ++i) {
        const float w = fast_exp2(sm_m[i] - top);
        total = fmaf(w, sm_l[i], total);
        o = fmaf(w, sm_acc[i * kHeadDim + threadIdx.x], o);
    }
    o /= total;
    const float lse2 = top + log2f(total);
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
