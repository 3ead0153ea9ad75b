// Sparse decode attention after the paper's Algorithm 1 (SparF: SparQ's arithmetic with
// page-granular loading), on the block-paged cache, for sm_100a.
//
//   sparf_append_kernel   the new token's k,v go to the token-major pools, k also to the
//                         embedding-major K copy (Sec. IV-C: K is stored twice), and v is
//                         added to the running V sum that gives the mean value vector.
//   sparf_scores_kernel   step 1 (the r largest |q_d|) and steps 2-4 without the softmax
//                         normalisation: approximate logits from the embedding-major copy.
//   steps 5-7             softmax statistics of the approximate logits, the k largest scores
//                         with the last l tokens forced in (ties to the lower position), alpha,
//                         and the ascending list of selected rows as physical row ids.  Two
//                         forms: one block per row with the row's logits in shared memory
//                         (sparf_fused_select_kernel), and for long rows a chain that never
//                         writes the logits out (sparf_staged_select.cuh: a sampled pre-pass
//                         brackets the threshold, the score kernel stages only the tokens that
//                         can still be selected, the rest is resolved on those).  Rows the
//                         chain cannot settle fall back to sparf_scores_kernel +
//                         sparf_select_kernel, the same steps with one block per row.
//   (steps 8-10 run in decode_attn_split_kernel<Rows::kGathered>)
//   sparf_merge_kernel    log-sum-exp merge of the chunk partials and step 11:
//                         out = alpha * attended + (1 - alpha) * v_sum / S.
#pragma once

#include <cstddef>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "decode_attention_kernels.cuh"

namespace instinfer {

// Per (sequence, head) state of the staged selection.  Zero-initialised per call.
struct SelectRow {
    float lo;                  // tokens whose logit is below this cannot be selected
    float hi;                  // tokens whose logit is above this are surely selected (never -0)
    float ref;                 // reference of the softmax sums (the largest sampled logit)
    int n_cand;                // candidates (lo <= logit <= hi, outside the window) collected so far
    int overflow;              // a logit far above ref was seen: the sums are not trustworthy
    unsigned tau;              // exact ordered key of the k-th largest
    int idx_cut;               // among keys equal to tau, positions <= idx_cut are taken
    int solved;                // 0: the single-block kernels must redo this row
};

struct SparfParams {
    // cache
    __half *k_pool;
    __half *v_pool;
    __half *kt_pool;           // [Pk, H, D, Tk]: its own block size and table
    float *v_sum;              // [B, H, D]
    const __half *q;
    const __half *k_new;
    const __half *v_new;
    const int32_t *seq_lens;
    const int32_t *k_tokens;
    const int32_t *block_table;
    const int32_t *kt_block_table;   // [batch, kt_max_blocks_per_seq]
    int32_t *status;
    // scratch
    float *scores;             // [pairs, score_stride]: logits of the staged tokens (staged chain), or
                               // all approximate logits of a row (fallback); base-2 domain
    int32_t *stage_pos;        // [pairs, score_stride]: positions of the staged tokens, per segment
    int32_t *row_ids;          // [pairs, max_k]
    float2 *stats;             // [pairs] (alpha, number of selected rows)
    struct SelectRow *rows_state;   // [pairs], zeroed before each call
    int *unsolved;             // rows the staged chain could not settle (zeroed with rows_state)
    uint2 *row_cand;           // [pairs, cand_capacity] (ordered key, token index)
    int32_t *seg_count;        // [pairs, segments] staged tokens per segment
    int32_t *seg_final;        // [pairs, segments] selected tokens per segment
    float *blk_z;              // [pairs, score_blocks] softmax denominator parts
    float *seg_mass;           // [pairs, segments] selected mass parts
    // outputs
    float *alpha_out;          // nullable [pairs]
    int32_t *selected;         // nullable [pairs, max_k] logical token index, ascending, -1 padded
    int64_t num_phys_blocks;
    int64_t num_kt_blocks;
    int64_t kt_elems;          // elements of kt_pool that the call's shapes imply (attention call only)
    int32_t batch, heads, block_tokens, max_blocks_per_seq;
    int32_t kt_block_tokens, kt_max_blocks_per_seq;
    int32_t max_seq_len, max_k, score_stride, segments, score_blocks, cand_capacity, r, window;
    float scale_log2e;
};

constexpr int kSparfThreads = 128;       // append and scores: one thread per head dim
constexpr int kSegmentTokens = 256;      // staged chain: tokens per staging segment (one pass of one warp)
constexpr int kScoreBlockTokens = 8192;  // tokens per block of the score kernels (amortises their prologue)
constexpr int kSelectThreads = 1024;

__device__ __forceinline__ int sparf_seq_len(const SparfParams &p, int b, bool report)
{
    int len = p.seq_lens[b];
    if (len < 0 || len > p.max_seq_len) {
        if (report && p.status) atomicOr(p.status, kFlagSeqLenRange);
        len = 0;
    }
    return len;
}

__global__ void __launch_bounds__(kSparfThreads)
sparf_append_kernel(const SparfParams p)
{
    const int pair = blockIdx.x, d = threadIdx.x;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const int len = p.seq_lens[b];
    if (len == 0) return;
    // Both capacities are checked before either table is read: a length that fits the K/V
    // table but not the transposed copy's must not index past that table's row.
    const int T = p.block_tokens, Tk = p.kt_block_tokens;
    if (len < 0 || (int64_t)len > (int64_t)p.max_blocks_per_seq * T ||
        (int64_t)len > (int64_t)p.kt_max_blocks_per_seq * Tk) {
        if (d == 0 && h == 0 && p.status) atomicOr(p.status, kFlagSeqLenRange);
        return;
    }
    const int pos = len - 1;
    const int phys = p.block_table[(int64_t)b * p.max_blocks_per_seq + pos / T];
    const int kt_phys = p.kt_block_table[(int64_t)b * p.kt_max_blocks_per_seq + pos / Tk];
    if (phys < 0 || (int64_t)phys >= p.num_phys_blocks || kt_phys < 0 || (int64_t)kt_phys >= p.num_kt_blocks) {
        if (d == 0 && h == 0 && p.status) atomicOr(p.status, kFlagBlockRange);
        return;
    }
    const int slot = pos % T;
    const int64_t base = ((int64_t)phys * p.heads + h) * T * kHeadDim;      // elements
    const __half k = p.k_new[(int64_t)pair * kHeadDim + d];
    const __half v = p.v_new[(int64_t)pair * kHeadDim + d];
    p.k_pool[base + (int64_t)slot * kHeadDim + d] = k;
    p.v_pool[base + (int64_t)slot * kHeadDim + d] = v;
    p.kt_pool[(((int64_t)kt_phys * p.heads + h) * kHeadDim + d) * Tk + pos % Tk] = k;
    p.v_sum[(int64_t)pair * kHeadDim + d] += __half2float(v);
}

// Bulk append, the part specific to the sparse state (K and V rows go through
// kv_append_bulk_kernel): one block per (sequence, head), one thread per dim.  The thread
// walks the new tokens in order, adds v to the running sum (fp32, one rounding per token, the
// order a token-by-token append would use) and writes k into the embedding-major copy, 8
// tokens (16 bytes) at a time where a whole aligned group is new.
struct SparfBulkParams {
    SparfParams base;             // k_new / v_new point at [batch, max_new, heads, 128]
    const int32_t *new_lens;
    int32_t max_new;
};

__global__ void __launch_bounds__(kSparfThreads)
sparf_append_bulk_kernel(const SparfBulkParams q)
{
    const SparfParams &p = q.base;
    const int pair = blockIdx.x, d = threadIdx.x;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const int len = p.seq_lens[b], fresh = q.new_lens[b];
    const int Tk = p.kt_block_tokens;
    if (len < 0 || (int64_t)len > (int64_t)p.max_blocks_per_seq * p.block_tokens ||
        (int64_t)len > (int64_t)p.kt_max_blocks_per_seq * Tk || fresh < 0 || fresh > q.max_new || fresh > len) {
        if (d == 0 && h == 0 && p.status) atomicOr(p.status, kFlagSeqLenRange);
        return;
    }
    if (fresh == 0) return;
    const int first = len - fresh;
    const int32_t *kt_table = p.kt_block_table + (int64_t)b * p.kt_max_blocks_per_seq;
    // Every block id the new tokens need, in both tables, is checked before anything is
    // written, so that a flagged sequence keeps its transposed copy and its running sum as
    // they were (its K and V rows go through kv_append_bulk_kernel, which skips the rows of
    // bad blocks only: the header calls the state of a flagged sequence undefined).
    {
        const int32_t *kv_table = p.block_table + (int64_t)b * p.max_blocks_per_seq;
        bool bad = false;
        for (int blk = first / Tk; blk <= (len - 1) / Tk; ++blk)
            bad |= kt_table[blk] < 0 || (int64_t)kt_table[blk] >= p.num_kt_blocks;
        for (int blk = first / p.block_tokens; blk <= (len - 1) / p.block_tokens; ++blk)
            bad |= kv_table[blk] < 0 || (int64_t)kv_table[blk] >= p.num_phys_blocks;
        if (bad) {
            if (d == 0 && h == 0 && p.status) atomicOr(p.status, kFlagBlockRange);
            return;
        }
    }
    const int64_t token_stride = (int64_t)p.heads * kHeadDim;                 // elements between tokens
    const __half *k_src = p.k_new + ((int64_t)b * q.max_new * p.heads + h) * kHeadDim + d;
    const __half *v_src = p.v_new + ((int64_t)b * q.max_new * p.heads + h) * kHeadDim + d;
    float sum = p.v_sum[(int64_t)pair * kHeadDim + d];
    int t = 0;
    while (t < fresh) {
        const int pos = first + t;
        const int phys = kt_table[pos / Tk];                                   // checked above
        __half *dst = p.kt_pool + (((int64_t)phys * p.heads + h) * kHeadDim + d) * Tk + pos % Tk;
        if ((pos & 7) == 0 && t + 8 <= fresh) {                                // a whole aligned group
            __align__(16) __half group[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                group[e] = k_src[(int64_t)(t + e) * token_stride];
                sum += __half2float(v_src[(int64_t)(t + e) * token_stride]);
            }
            *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(group);
            t += 8;
        } else {
            *dst = k_src[(int64_t)t * token_stride];
            sum += __half2float(v_src[(int64_t)t * token_stride]);
            t += 1;
        }
    }
    p.v_sum[(int64_t)pair * kHeadDim + d] = sum;
}

// Order-preserving map float -> uint32 (larger float, larger key).
__device__ __forceinline__ unsigned ordered_key(float x)
{
    const unsigned u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Step 1 and the temperature of steps 2-4, shared by the kernels that compute approximate
// logits.  Threads d < 128 each own one head dim; every thread of the block must call it.
struct __align__(16) ScoreShared {       // 16 bytes: the keys of step 1 are read four at a time
    float abs_q[kHeadDim];
    unsigned short q_bits[kHeadDim];   // q of the selected dims as fp16 bit patterns, in rank order
    int dim[kHeadDim];          // the selected dims, in rank order
    bool kept[kHeadDim];
    float approx_scale;
};

static_assert(offsetof(ScoreShared, dim) % 16 == 0, "the keys of step 1 are read as uint4");

__device__ __forceinline__ void score_setup(const SparfParams &p, int pair, ScoreShared &ss)
{
    const int d = threadIdx.x;
    // Step 1: rank of |q_d| (exact comparisons of fp16 magnitudes, ties to the lower index).
    // The 15 magnitude bits of an fp16 number order like the magnitude itself, so one integer
    // key per dim -- magnitude bits, then 127 - d -- makes every comparison a single one:
    // rank = number of larger keys.  (ss.dim doubles as the key array until the ranks are known.)
    unsigned short bits = 0;
    unsigned *keys = reinterpret_cast<unsigned *>(ss.dim);
    if (d < kHeadDim) {
        bits = __half_as_ushort(p.q[(int64_t)pair * kHeadDim + d]);
        ss.abs_q[d] = fabsf(__half2float(__ushort_as_half(bits)));
        keys[d] = (unsigned)(bits & 0x7fffu) << 8 | (unsigned)(kHeadDim - 1 - d);
    }
    __syncthreads();
    int rank = 0;
    if (d < kHeadDim) {
        const unsigned mine = keys[d];
        const uint4 *four = reinterpret_cast<const uint4 *>(keys);
#pragma unroll 8
        for (int e = 0; e < kHeadDim / 4; ++e) {
            const uint4 other = four[e];
            rank += (int)(other.x > mine) + (int)(other.y > mine) + (int)(other.z > mine) + (int)(other.w > mine);
        }
    }
    __syncthreads();                                         // every key has been read: ss.dim is free
    if (d < kHeadDim) {
        const bool kept = rank < p.r;
        if (kept) {
            ss.dim[rank] = d;
            ss.q_bits[rank] = bits;
        }
        ss.kept[d] = kept;
    }
    // |q|_1 and |q_I|_1 in fp32.  The temperature is one positive constant per row, so its
    // rounding cannot change the ranking of step 6; each logit is an fp32 sum of r exact
    // fp16 x fp16 products times that constant, i.e. within (r + 1) 2^-24 of sum |q_t k_t|.
    __syncthreads();
    if (d < 32) {                                            // warp 0: lane sums, then a butterfly
        float all = 0.f, sel = 0.f;
        for (int e = d; e < kHeadDim; e += 32) {
            all += ss.abs_q[e];
            if (ss.kept[e]) sel += ss.abs_q[e];
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            all += __shfl_xor_sync(0xffffffffu, all, off);
            sel += __shfl_xor_sync(0xffffffffu, sel, off);
        }
        const float ratio = all > 0.f ? sel / all : 1.f;
        if (d == 0) ss.approx_scale = p.scale_log2e / sqrtf(ratio);
    }
    __syncthreads();
}

// Steps 2-4 for the 8 consecutive tokens i .. i + 7 of (sequence b, head h): one 16-byte load
// per selected dim from the transposed copy (kt_block_tokens is a multiple of 8, so a group
// never straddles a block); the loads of 8 dims are issued together to keep bytes in flight.
__device__ __forceinline__ void score_group(const SparfParams &p, const ScoreShared &ss,
                                            const int32_t *table_row, int h, int i, float (&dot)[8])
{
    const int T = p.kt_block_tokens;
    const int t_shift = (T & (T - 1)) == 0 ? __ffs(T) - 1 : -1;      // blocks of 2^n tokens: no division
    const int blk = t_shift >= 0 ? i >> t_shift : i / T, slot = i - blk * T;
    const int phys = bounds_ok(blk < p.kt_max_blocks_per_seq, p.status) ? table_row[blk] : -1;
#pragma unroll
    for (int e = 0; e < 8; ++e) dot[e] = 0.f;
    const int64_t area = ((int64_t)phys * p.heads + h) * T * kHeadDim;      // this (block, head): [D][T]
    if (phys >= 0 && (int64_t)phys < p.num_kt_blocks &&
        bounds_ok(area + (int64_t)(kHeadDim - 1) * T + slot + 8 <= p.kt_elems, p.status)) {
        const __half *kt = p.kt_pool + area + slot;
        for (int t0 = 0; t0 < p.r; t0 += 8) {
            uint4 raw[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int t = min(t0 + u, p.r - 1);            // clamped: extra loads repeat the last dim
                raw[u] = __ldg(reinterpret_cast<const uint4 *>(kt + (int64_t)ss.dim[t] * T));
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (t0 + u < p.r) {                            // uniform; extra loads are ignored
                    // fp16 x fp16 products are exact in fp32: one rounding per addition, the
                    // same values as converting first, without the conversions
                    const unsigned short qv = ss.q_bits[t0 + u];
                    const unsigned kw[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        unsigned short k0, k1;
                        halves(kw[e], k0, k1);
                        dot[2 * e] = fma_h(k0, qv, dot[2 * e]);
                        dot[2 * e + 1] = fma_h(k1, qv, dot[2 * e + 1]);
                    }
                }
            }
        }
    } else if (p.status) {
        atomicOr(p.status, kFlagBlockRange);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) dot[e] *= ss.approx_scale;
}

// Every kernel of the attention call below starts with the programmatic-dependent-launch pair
// (let the next kernel's blocks become resident, then wait for all earlier kernels), before
// any return, so that the chain of short launches overlaps its launch latencies.
// All approximate logits of the rows the staged chain left unsolved, written to the workspace,
// kScoreBlockTokens tokens of one (sequence, head) per step of a block; the grid is bounded
// and its blocks walk over all (row, block) items, skipping those of solved rows.
__global__ void __launch_bounds__(kSparfThreads)
sparf_scores_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    __shared__ ScoreShared ss;
    const int d = threadIdx.x;
    if (*p.unsolved == 0) return;                            // the usual case: the chain settled every row
    const int64_t items = (int64_t)p.batch * p.heads * p.score_blocks;
    for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int pair = (int)(item / p.score_blocks);
        if (p.rows_state[pair].solved) continue;
        const int b = pair / p.heads, h = pair - b * p.heads;
        const int len = sparf_seq_len(p, b, false);
        const int begin = (int)(item - (int64_t)pair * p.score_blocks) * kScoreBlockTokens;
        if (begin >= len) continue;
        const int end = min(begin + kScoreBlockTokens, len);
        __syncthreads();                                     // the previous item's set-up is no longer read
        score_setup(p, pair, ss);

        const int32_t *table_row = p.kt_block_table + (int64_t)b * p.kt_max_blocks_per_seq;
        float *dst = p.scores + (int64_t)pair * p.score_stride;
        for (int i = begin + d * 8; i < end; i += kSparfThreads * 8) {
            float dot[8];
            score_group(p, ss, table_row, h, i, dot);
            // score_stride is a multiple of 8 and rows start 32-byte aligned; entries past `end`
            // inside the last group are scratch nobody reads.
            float4 *out4 = reinterpret_cast<float4 *>(dst + i);
            out4[0] = make_float4(dot[0], dot[1], dot[2], dot[3]);
            out4[1] = make_float4(dot[4], dot[5], dot[6], dot[7]);
        }
    }
}

template <typename T>
__device__ __forceinline__ T block_sum(T v, T *scratch)      // scratch: 32 entries
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    T total = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += scratch[w];
    return total;
}

constexpr int kLinearBins = 2048;        // select: linear bins between the smallest and largest logit
constexpr int kCandidates = 8192;        // select: keys of the threshold bin resolved in shared memory

struct SelectCore {
    unsigned hist[kLinearBins + 1];      // bin kLinearBins: the forced local window
    float red_f[32];
    unsigned red_u[2][32];
    int scan_gt[32], scan_eq[32];
    unsigned tau;
    int take_equal, bin, above, n_cand;
};
struct SelectShared : SelectCore {
    unsigned cand[kCandidates];
};

// Streams a score row as float4 with 4 loads in flight per thread; fn(first_index, values[4]).
template <int NT, typename Fn>
__device__ __forceinline__ void for_each_quad(const float4 *a4, int quads, Fn fn)
{
    for (int g0 = threadIdx.x; g0 < quads; g0 += 4 * NT) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int g = g0 + u * NT;
            v[u] = g < quads ? a4[g] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int g = g0 + u * NT;
            if (g < quads) {
                const float x[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                fn(4 * g, x);
            }
        }
    }
}

// Warp 0 finds, among 256 counters, the bucket (from the top) in which the running count
// reaches `remaining`; returns it with the count of the buckets above through shared memory.
__device__ __forceinline__ void locate_bucket(const unsigned *hist, int remaining, int *bucket_out, int *above_out)
{
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) mine += (int)hist[8 * lane + j];
        int above = 0;
        for (int src = 31; src >= 0; --src) {
            const int seg = __shfl_sync(0xffffffffu, mine, src);
            if (src > lane) above += seg;
        }
        if (above < remaining && remaining <= above + mine) {
            int bucket = 8 * lane + 7;
            for (; bucket > 8 * lane; --bucket) {
                const int c = (int)hist[bucket];
                if (above + c >= remaining) break;
                above += c;
            }
            *bucket_out = bucket;
            *above_out = above;
        }
    }
}

// Exact k-th largest among the keys key_at(i) of the members i < n (member(i) true), 8 bits
// per pass from the top.  Bytes on which all members agree are skipped without counting, so
// a set of (nearly) equal keys costs nothing.  Returns through sh.tau / sh.take_equal the
// threshold key and how many keys equal to it are among the `need` largest.
template <int NT, typename Member, typename KeyAt>
__device__ __forceinline__ void exact_threshold(SelectCore &sh, int n, int need, Member member, KeyAt key_at)
{
    const int tid = threadIdx.x;
    unsigned any = 0u, all = 0xffffffffu;
    for (int i = tid; i < n; i += NT) {
        if (member(i)) {
            const unsigned key = key_at(i);
            any |= key;
            all &= key;
        }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        any |= __shfl_xor_sync(0xffffffffu, any, off);
        all &= __shfl_xor_sync(0xffffffffu, all, off);
    }
    __syncthreads();
    if ((tid & 31) == 0) {
        sh.red_u[0][tid >> 5] = any;
        sh.red_u[1][tid >> 5] = all;
    }
    __syncthreads();
    any = 0u;
    all = 0xffffffffu;
    for (int w = 0; w < NT / 32; ++w) {
        any |= sh.red_u[0][w];
        all &= sh.red_u[1][w];
    }
    const unsigned differ = any ^ all;           // bits on which members disagree
    unsigned prefix = 0u;
    int remaining = need;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned done_mask = pass == 0 ? 0u : 0xffffffffu << (shift + 8);
        if (((differ >> shift) & 255u) == 0u) {  // every member has the same byte here
            prefix |= all & (255u << shift);
            continue;
        }
        __syncthreads();
        if (tid < 256) sh.hist[tid] = 0u;
        __syncthreads();
        for (int i = tid; i < n; i += NT) {
            if (member(i)) {
                const unsigned key = key_at(i);
                if ((key & done_mask) == prefix) atomicAdd(&sh.hist[(key >> shift) & 255u], 1u);
            }
        }
        __syncthreads();
        locate_bucket(sh.hist, remaining, &sh.bin, &sh.above);
        __syncthreads();
        prefix |= (unsigned)sh.bin << shift;
        remaining -= sh.above;
    }
    __syncthreads();
    if (tid == 0) {
        sh.tau = prefix;
        sh.take_equal = remaining;
    }
    __syncthreads();
}

// Steps 5-7 for one (sequence, head) by one block of NT threads (NT a multiple of 32, <= 1024): `a` is the row's
// S approximate logits (global or shared memory; 32-byte aligned, padded to a multiple of 8
// readable floats).  Writes the row-id list, the optional `selected` list, alpha and the count.
template <int NT>
__device__ __forceinline__ void select_row(const SparfParams &p, SelectShared &sh, const float *a,
                                           int pair, int b, int h, int S, int k, int window)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t *rows = p.row_ids + (int64_t)pair * p.max_k;
    int32_t *sel = p.selected ? p.selected + (int64_t)pair * p.max_k : nullptr;
    if (sel) for (int t = k + tid; t < p.max_k; t += NT) sel[t] = -1;
    if (k == 0) {
        if (tid == 0) {
            p.stats[pair] = make_float2(0.f, 0.f);
            if (p.alpha_out) p.alpha_out[pair] = 0.f;
        }
        return;
    }
    // The score row is 32-byte aligned and padded to a multiple of 8 floats (padding is
    // readable scratch), so every pass streams it as float4 and masks the tail by index.
    const float4 *a4 = reinterpret_cast<const float4 *>(a);
    const int quads = (S + 3) / 4;

    // Pass 1: largest and smallest approximate logit (base-2 domain).
    float top = kMinusHuge, low = -kMinusHuge;
    for_each_quad<NT>(a4, quads, [&](int i0, const float (&x)[4]) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (i0 + e < S) {
                top = fmaxf(top, x[e]);
                low = fminf(low, x[e]);
            }
        }
    });
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, off));
        low = fminf(low, __shfl_xor_sync(0xffffffffu, low, off));
    }
    if (lane == 0) {
        sh.red_f[warp] = top;
        sh.red_u[0][warp] = __float_as_uint(low);
    }
    for (int t = tid; t <= kLinearBins; t += NT) sh.hist[t] = 0u;
    __syncthreads();
    for (int w = 0; w < NT / 32; ++w) {
        top = fmaxf(top, sh.red_f[w]);
        low = fminf(low, __uint_as_float(sh.red_u[0][w]));
    }

    // Step 5: the last `window` positions rank above everything (s^ + 1 beats every s^).
    // Linear bins are monotone in the logit: a higher bin holds strictly larger logits.
    const float bin_scale = top > low ? (float)(kLinearBins - 1) / (top - low) : 0.f;
    auto bin_of = [&](int i, float x) -> int {
        return i >= S - window ? kLinearBins : min(kLinearBins - 1, (int)((x - low) * bin_scale));
    };
    auto key_of = [&](int i, float x) -> unsigned { return i >= S - window ? 0xffffffffu : ordered_key(x); };

    // Pass 2: histogram over the linear bins, and the softmax denominator.
    float z = 0.f;
    for_each_quad<NT>(a4, quads, [&](int i0, const float (&x)[4]) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (i0 + e < S) {
                z += fast_exp2(x[e] - top);
                atomicAdd(&sh.hist[bin_of(i0 + e, x[e])], 1u);
            }
        }
    });
    z = block_sum(z, sh.red_f);                  // its barriers also publish the histogram

    // The bin that holds the k-th largest: warp 0, lane L owns bins [64 L, 64 L + 64).
    if (warp == 0) {
        int mine = 0;
        for (int j = 0; j < 64; ++j) mine += (int)sh.hist[64 * lane + ((j + lane) & 63)];
        int above = (int)sh.hist[kLinearBins];   // members of higher bins
        for (int src = 31; src >= 0; --src) {
            const int seg = __shfl_sync(0xffffffffu, mine, src);
            if (src > lane) above += seg;
        }
        if ((int)sh.hist[kLinearBins] >= k) {
            if (lane == 0) {
                sh.bin = kLinearBins;
                sh.above = 0;
            }
        } else if (above < k && k <= above + mine) {
            int bin = 64 * lane + 63;
            for (; bin > 64 * lane; --bin) {
                const int c = (int)sh.hist[bin];
                if (above + c >= k) break;
                above += c;
            }
            sh.bin = bin;
            sh.above = above;
        }
        if (lane == 0) sh.n_cand = 0;
    }
    __syncthreads();
    const int bin = sh.bin, above = sh.above;
    const int in_bin = (int)sh.hist[bin];
    __syncthreads();                             // the histogram is reused below

    // Step 6: the exact threshold inside that bin.
    if (bin == kLinearBins) {                    // the window alone fills k
        if (tid == 0) {
            sh.tau = 0xffffffffu;
            sh.take_equal = k;
        }
        __syncthreads();
    } else if (in_bin <= kCandidates) {
        for_each_quad<NT>(a4, quads, [&](int i0, const float (&x)[4]) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (i0 + e < S && bin_of(i0 + e, x[e]) == bin)
                    sh.cand[atomicAdd(&sh.n_cand, 1)] = ordered_key(x[e]);
            }
        });
        __syncthreads();
        if (in_bin <= NT) {          // the usual case: rank every candidate directly
            const int need = k - above;
            if (tid < in_bin) {
                const unsigned mine = sh.cand[tid];
                int greater = 0, equal = 0;
                for (int j = 0; j < in_bin; ++j) {
                    const unsigned other = sh.cand[j];
                    greater += other > mine;
                    equal += other == mine;
                }
                if (greater < need && need <= greater + equal) {     // all holders of this key agree
                    sh.tau = mine;
                    sh.take_equal = need - greater;
                }
            }
            __syncthreads();
        } else {
            exact_threshold<NT>(sh, in_bin, k - above, [](int) { return true; },
                            [&](int i) { return sh.cand[i]; });
        }
    } else {                                     // very many near-equal logits: work from global memory
        exact_threshold<NT>(sh, S, k - above, [&](int i) { return bin_of(i, a[i]) == bin; },
                        [&](int i) { return ordered_key(a[i]); });
    }
    const unsigned tau = sh.tau;                 // key of the k-th largest
    const int take_equal = sh.take_equal;        // how many keys equal to tau belong to the top k

    // Ordered compaction: position = #greater before + min(#equal before, take_equal).
    const int T = p.block_tokens;
    const int t_shift = (T & (T - 1)) == 0 ? __ffs(T) - 1 : -1;      // blocks of 2^n tokens: no division per token
    const int32_t *table_row = p.block_table + (int64_t)b * p.max_blocks_per_seq;
    float mass = 0.f;
    // Each warp owns a contiguous span of the row, each lane 4 consecutive positions at a time.
    // The warps count their spans, exchange the totals once, and then emit without meeting again.
    constexpr int kWarps = NT / 32;
    const int span = (quads + kWarps - 1) / kWarps;
    const int q_begin = min(warp * span, quads), q_end = min(q_begin + span, quads);
    // counts of one thread's 4 positions travel packed (greater | equal << 16)
    auto classify = [&](int g, const float4 &v, bool (&gt)[4], bool (&eq)[4]) -> int {
        const float x[4] = {v.x, v.y, v.z, v.w};
        int packed = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = 4 * g + e;
            const unsigned key = key_of(i, x[e]);
            gt[e] = i < S && key > tau;
            eq[e] = i < S && key == tau;
            packed += (int)gt[e] + ((int)eq[e] << 16);
        }
        return packed;
    };
    int span_gt = 0, span_eq = 0;
    for (int g = q_begin + lane; g < q_end; g += 32) {
        bool gt[4], eq[4];
        const int packed = classify(g, a4[g], gt, eq);
        span_gt += packed & 0xffff;
        span_eq += packed >> 16;
    }
    span_gt = __reduce_add_sync(0xffffffffu, span_gt);
    span_eq = __reduce_add_sync(0xffffffffu, span_eq);
    if (lane == 0) {
        sh.scan_gt[warp] = span_gt;
        sh.scan_eq[warp] = span_eq;
    }
    __syncthreads();
    int base_gt = __reduce_add_sync(0xffffffffu, lane < warp ? sh.scan_gt[lane] : 0);
    int base_eq = __reduce_add_sync(0xffffffffu, lane < warp ? sh.scan_eq[lane] : 0);
    for (int g0 = q_begin; g0 < q_end; g0 += 32) {
        const int g = g0 + lane;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        bool gt[4] = {false, false, false, false}, eq[4] = {false, false, false, false};
        int mine = 0;
        if (g < q_end) {
            v = a4[g];
            mine = classify(g, v, gt, eq);
        }
        int incl = mine;                          // inclusive scan over the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        const int tile_total = __shfl_sync(0xffffffffu, incl, 31);
        int gt_before = base_gt + ((incl - mine) & 0xffff), eq_before = base_eq + ((incl - mine) >> 16);
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (gt[e] || (eq[e] && eq_before < take_equal)) {
                const int i = 4 * g + e;
                const int pos = gt_before + min(eq_before, take_equal);
                const int blk = t_shift >= 0 ? i >> t_shift : i / T, slot = i - blk * T;
                const int phys = bounds_ok(blk < p.max_blocks_per_seq && pos < p.max_k, p.status) ? table_row[blk] : -1;
                const bool ok = phys >= 0 && (int64_t)phys < p.num_phys_blocks;
                if (!ok && p.status) atomicOr(p.status, kFlagBlockRange);
                rows[pos] = ok ? (phys * p.heads + h) * T + slot : 0;
                if (sel) sel[pos] = i;
                mass += fast_exp2(x[e] - top);
            }
            gt_before += (int)gt[e];
            eq_before += (int)eq[e];
        }
        base_gt += tile_total & 0xffff;
        base_eq += tile_total >> 16;
    }
    mass = block_sum(mass, sh.red_f);
    if (tid == 0) {
        const float alpha = mass / z;
        p.stats[pair] = make_float2(alpha, (float)k);
        if (p.alpha_out) p.alpha_out[pair] = alpha;
    }
}

// One block per (sequence, head) at a time, logits from the workspace: redoes the rows that
// the staged chain left unsolved.  Those are rare, so the grid is a few blocks per SM that walk
// over all rows and skip the solved ones (a block per row would be thousands of blocks that
// start only to leave).
__global__ void __launch_bounds__(kSelectThreads)
sparf_select_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    __shared__ SelectShared sh;
    if (*p.unsolved == 0) return;                            // the usual case: the chain settled every row
    const int pairs = p.batch * p.heads;
    for (int pair = blockIdx.x; pair < pairs; pair += gridDim.x) {
        if (p.rows_state[pair].solved) continue;             // done by the staged chain
        const int b = pair / p.heads, h = pair - b * p.heads;
        const int S = sparf_seq_len(p, b, threadIdx.x == 0 && h == 0);
        const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
        __syncthreads();                                     // the scratch of the previous row is free
        select_row<kSelectThreads>(p, sh, p.scores + (int64_t)pair * p.score_stride, pair, b, h, S, k, min(p.window, k));
    }
}

// Steps 1-7 for one (sequence, head) by one block: the row's approximate logits are computed
// straight into shared memory and selected from there, so they never travel through HBM.
// For rows of at most kFusedMaxTokens tokens.  Two blocks share an SM, so one block's selection
// (instruction-bound) overlaps the other's loads.
constexpr int kFusedMaxTokens = 16384;
constexpr int kFusedSmemBytes = kFusedMaxTokens * (int)sizeof(float);
constexpr int kFusedThreads = 512;       // two blocks per SM: one selects while the other loads

__global__ void __launch_bounds__(kFusedThreads, 2)
sparf_fused_select_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    extern __shared__ __align__(32) float row_scores[];
    __shared__ SelectShared sh;
    __shared__ ScoreShared ss;
    const int pair = blockIdx.x;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const int S = sparf_seq_len(p, b, threadIdx.x == 0 && h == 0);
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    if (k > 0) {                                 // uniform; with k == 0 no logit is needed
        score_setup(p, pair, ss);
        const int32_t *table_row = p.kt_block_table + (int64_t)b * p.kt_max_blocks_per_seq;
        for (int i = threadIdx.x * 8; i < S; i += kFusedThreads * 8) {
            float dot[8];
            score_group(p, ss, table_row, h, i, dot);
            float4 *out4 = reinterpret_cast<float4 *>(row_scores + i);    // S <= kFusedMaxTokens, whole groups
            out4[0] = make_float4(dot[0], dot[1], dot[2], dot[3]);
            out4[1] = make_float4(dot[4], dot[5], dot[6], dot[7]);
        }
        __syncthreads();
    }
    select_row<kFusedThreads>(p, sh, row_scores, pair, b, h, S, k, min(p.window, k));
}

// Merge of the gathered-attention partials and step 11.
struct SparfMergeParams {
    AttnParams attn;
    const float2 *stats;
    const float *v_sum;
};

__global__ void __launch_bounds__(kHeadDim)
sparf_merge_kernel(const SparfMergeParams m)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    const AttnParams &p = m.attn;
    const int pair = blockIdx.x;
    const int b = pair / p.heads;
    const int S = checked_seq_len(p, b, false);
    __half *out = p.out + (int64_t)pair * kHeadDim + threadIdx.x;
    if (S == 0) {
        *out = __float2half_rn(0.f);
        return;
    }
    const float alpha = m.stats[pair].x;
    const int count = gathered_count(p, b, S);
    const float vbar = m.v_sum[(int64_t)pair * kHeadDim + threadIdx.x] / (float)S;
    const int live = live_chunks(p, count);
    float attended = 0.f;
    if (live > 0) {
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
        attended = o / total;
    }
    *out = __float2half_rn(alpha * attended + (1.f - alpha) * vbar);
}

}  // namespace instinfer
