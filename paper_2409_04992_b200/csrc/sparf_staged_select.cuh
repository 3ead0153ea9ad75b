// Steps 1-7 of Algorithm 1 for long rows without ever writing the approximate logits to HBM.
//
// Selecting the k largest of S scores needs the k-th largest value, which is only known once
// all scores are; the plain way writes the S logits out and passes over them again and again.
// Here a cheap pre-pass brackets that value first, so that the one pass that computes the
// logits can already drop what cannot be selected:
//
//   sparf_sample_kernel   one block per row: the logits of a systematic sample of the row (runs
//                         of 256 tokens, an eighth of a long row: whole 512-byte pieces of the
//                         transposed copy, which HBM serves well; 64-byte pieces cost as much
//                         as four times their bytes), a histogram of them, and from it two bounds
//                         lo < hi such that the k-th largest logit of the whole row lies
//                         between them unless the sample is off by more than five standard
//                         deviations of its rank statistic.  Also the reference of the
//                         softmax sums (the largest sampled logit).
//   sparf_stage_kernel    computes every logit of the row (the big read of the transposed
//                         K copy) and keeps, in position order per 256-token segment (one warp
//                         pass, so no block barrier is needed), only
//                         the tokens of the local window and those with logit >= lo; counts
//                         the ones above hi (surely selected) and collects the ones between
//                         lo and hi as candidates.  Adds up the softmax denominator.
//   sparf_resolve_kernel  one block per row: the exact threshold among the candidates (the
//                         missing k - sure largest; ties to the lower position), and the final
//                         number of selected tokens per segment.  Declares the row unsolved if
//                         the bracket missed or the candidates overflowed.
//   sparf_emit_kernel     passes over the staged tokens only (about k + candidates per row):
//                         ordered compaction into the list of physical row ids, selected mass.
//   sparf_finish_kernel   alpha = selected mass / denominator, padding of `selected`.
//
// Rows left unsolved (a bracket that missed, thousands of equal scores) are redone by
// sparf_scores_kernel + sparf_select_kernel, which skip the solved ones.
#pragma once

#include "sparf_kernels.cuh"

namespace instinfer {

constexpr int kSampleRun = 256;          // consecutive tokens sampled per stride
constexpr int kMaxSamples = 16384;       // per row (64 KiB of shared memory)
constexpr int kEmitThreads = 256;
constexpr float kRefSlack = 64.f;        // logits this far (base 2) above the sampled maximum void the sums

// Distance between sampled runs: an eighth of the row from 8k tokens on and a sixteenth from
// 64k on (the bracket's relative width shrinks with the square root of the sample), denser
// below, sparser for rows so long that the sample would not fit.
__device__ __forceinline__ int sample_stride(int S)
{
    if (S > 16 * kMaxSamples) return 16 * kSampleRun * ((S + 16 * kMaxSamples - 1) / (16 * kMaxSamples));
    if (S >= 65536) return 16 * kSampleRun;
    return kSampleRun * max(1, min(8, S / 1024));
}

// One warp: among the linear bins (lane L owns bins [64 L, 64 L + 64)), the bin in which the
// count from the top, started at `from_top`, reaches `target`; also the count above that bin.
__device__ __forceinline__ void locate_linear_bin(const unsigned *hist, int from_top, int target, int *bin_out, int *above_out)
{
    const int lane = threadIdx.x & 31;
    int mine = 0;
    for (int j = 0; j < 64; ++j) mine += (int)hist[64 * lane + ((j + lane) & 63)];
    int above = from_top;
    for (int src = 31; src >= 0; --src) {
        const int seg = __shfl_sync(0xffffffffu, mine, src);
        if (src > lane) above += seg;
    }
    if (above < target && target <= above + mine) {
        int bin = 64 * lane + 63;
        for (; bin > 64 * lane; --bin) {
            const int c = (int)hist[bin];
            if (above + c >= target) break;
            above += c;
        }
        *bin_out = bin;
        *above_out = above;
    }
}

// Shared memory (floats) that the samples of a row of at most max_seq_len tokens need.
inline int sample_capacity(int max_seq_len)
{
    const int64_t most = max_seq_len >= 65536 ? (int64_t)max_seq_len / 16 + 4096 : (int64_t)max_seq_len / 8 + 2 * kSampleRun;
    const int64_t floor = 8 * kSampleRun;                    // rows below 8k tokens are sampled more densely
    const int64_t need = most > floor ? most : floor;
    return (int)(need < kMaxSamples ? need : kMaxSamples);
}

// grid pairs, kSampleThreads threads (512 for long rows, 256 for rows whose sample is small,
// so that more blocks share an SM), dynamic shared memory sample_capacity(max_seq_len) floats.
template <int kSampleThreads>
__global__ void __launch_bounds__(kSampleThreads)
sparf_sample_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    extern __shared__ __align__(32) float samples[];
    __shared__ ScoreShared ss;
    __shared__ unsigned hist[kLinearBins];
    __shared__ float red[2][kSampleThreads / 32];
    __shared__ int found[4];             // bin / count above it, for the two ranks
    const int pair = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const int S = sparf_seq_len(p, b, tid == 0 && h == 0);
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    const int window = min(p.window, k);
    SelectRow *row = p.rows_state + pair;
    const int outside = S - window, want = k - window;       // tokens and selections outside the window
    if (k == 0) {                        // nothing to select (also every inactive slot): no kernel has work
        if (tid == 0) {
            row->lo = row->hi = INFINITY;
            row->solved = 1;
        }
        return;
    }
    score_setup(p, pair, ss);
    const int32_t *table_row = p.kt_block_table + (int64_t)b * p.kt_max_blocks_per_seq;
    const int stride = sample_stride(S);
    const int runs = (S + stride - 1) / stride;
    constexpr int kGroupsPerRun = kSampleRun / 8;
    float top = kMinusHuge, low = -kMinusHuge;
    int n_samples = 0;                   // the same count on every thread: tokens < S in the sampled groups
    for (int g = tid; g < runs * kGroupsPerRun; g += kSampleThreads) {
        const int i = (g / kGroupsPerRun) * stride + (g % kGroupsPerRun) * 8;
        float dot[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (i < S) score_group(p, ss, table_row, h, i, dot);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const bool live = i + e < S;
            samples[g * 8 + e] = live ? dot[e] : kMinusHuge;
            if (live) {
                top = fmaxf(top, dot[e]);
                low = fminf(low, dot[e]);
            }
        }
    }
    // live samples: whole runs but the last, which may be cut by the end of the row
    {
        const int last_begin = (runs - 1) * stride;
        n_samples = (runs - 1) * kSampleRun + min(kSampleRun, S - last_begin);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, off));
        low = fminf(low, __shfl_xor_sync(0xffffffffu, low, off));
    }
    if (lane == 0) {
        red[0][warp] = top;
        red[1][warp] = low;
    }
    for (int t = tid; t < kLinearBins; t += kSampleThreads) hist[t] = 0u;
    __syncthreads();
    for (int w = 0; w < kSampleThreads / 32; ++w) {
        top = fmaxf(top, red[0][w]);
        low = fminf(low, red[1][w]);
    }
    if (want <= 0 || want >= outside) {
        // Nothing, or everything, outside the window is selected: there is no threshold to
        // bracket, only the reference of the sums was needed.
        if (tid == 0) {
            row->lo = row->hi = want <= 0 ? INFINITY : -INFINITY;        // stage nothing / everything, all sure
            row->ref = top;
        }
        return;
    }
    const float bin_scale = top > low ? (float)(kLinearBins - 1) / (top - low) : 0.f;
    const int total = runs * kGroupsPerRun * 8;
    for (int t = tid; t < total; t += kSampleThreads) {
        const float x = samples[t];
        if (x > kMinusHuge) atomicAdd(&hist[min(kLinearBins - 1, (int)((x - low) * bin_scale))], 1u);
    }
    __syncthreads();
    // Rank of the threshold in the sample and its five-sigma bracket.
    const float frac = (float)want / (float)outside;
    const float centre = frac * (float)n_samples;
    const float margin = 5.f * sqrtf(fmaxf((float)n_samples * frac * (1.f - frac), 0.f)) + 2.f;
    const int rank_hi = (int)floorf(centre - margin);        // this many samples are surely above the threshold
    const int rank_lo = (int)ceilf(centre + margin);         // the threshold is among the rank_lo largest
    if (warp < 2) {
        const int target = warp == 0 ? rank_hi : rank_lo;
        if (target >= 1 && target <= n_samples) locate_linear_bin(hist, 0, target, &found[2 * warp], &found[2 * warp + 1]);
    }
    __syncthreads();
    if (tid == 0) {
        // hi: the upper edge of the bin that holds the rank_hi-th largest sample (everything
        // above it is among the rank_hi largest); lo: the lower edge of the bin that holds the
        // rank_lo-th largest.  Edges are nudged outwards by one bin against float rounding of
        // the bin arithmetic; only the width of the bracket depends on them, never the result.
        float hi = INFINITY, lo = -INFINITY;
        if (bin_scale > 0.f) {
            if (rank_hi >= 1 && rank_hi <= n_samples) hi = low + (float)(found[0] + 2) / bin_scale;
            if (rank_lo >= 1 && rank_lo <= n_samples) lo = low + (float)(found[2] - 1) / bin_scale;
        }
        row->lo = lo;
        row->hi = hi + 0.f;              // -0 becomes +0: "logit > hi" then agrees with the order of the keys
        row->ref = top;
    }
}

struct StageShared {
    ScoreShared score;
    float red[32];
    uint2 staged[kSparfThreads / 32][kSegmentTokens];       // per warp: a segment's staged tokens (logit bits, position)
};

// grid pairs * score_blocks, kSparfThreads threads: kScoreBlockTokens tokens of one row.  Each
// warp takes whole segments of kSegmentTokens consecutive tokens (8 per lane), so the ordered
// staging of a segment is a warp scan and the block never synchronises inside the loop.
__global__ void __launch_bounds__(kSparfThreads, 8)
sparf_stage_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    __shared__ StageShared sh;
    static_assert(kSegmentTokens == 32 * 8, "one warp pass covers one segment");
    constexpr int kWarpsPerBlock = kSparfThreads / 32;
    const int pair = blockIdx.x / p.score_blocks, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int block_in_row = blockIdx.x - pair * p.score_blocks;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const int S = sparf_seq_len(p, b, false);
    const int begin = block_in_row * kScoreBlockTokens;
    if (begin >= S) return;
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    if (k == 0) return;
    const int window_from = S - min(p.window, k);
    SelectRow *row = p.rows_state + pair;
    const float lo = row->lo, hi = row->hi, ref = row->ref;
    const int end = min(begin + kScoreBlockTokens, S);
    score_setup(p, pair, sh.score);

    const int32_t *table_row = p.kt_block_table + (int64_t)b * p.kt_max_blocks_per_seq;
    float *stage_x = p.scores + (int64_t)pair * p.score_stride;
    int32_t *stage_pos = p.stage_pos + (int64_t)pair * p.score_stride;
    uint2 *cand = p.row_cand + (int64_t)pair * p.cand_capacity;
    const unsigned buf = static_cast<unsigned>(__cvta_generic_to_shared(sh.staged[warp]));
    float z = 0.f;
    bool far_above = false;
    for (int seg_begin = begin + warp * kSegmentTokens; seg_begin < end; seg_begin += kWarpsPerBlock * kSegmentTokens) {
        const int i = seg_begin + lane * 8;
        float dot[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (i < end) score_group(p, sh.score, table_row, h, i, dot);
        // bit e: token i + e exists / lies in the local window
        const unsigned live = i >= end ? 0u : i + 8 <= end ? 0xffu : (1u << (end - i)) - 1u;
        const unsigned in_window = i + 8 <= window_from ? 0u : i >= window_from ? 0xffu : 0xffu << (window_from - i) & 0xffu;
        unsigned staged = 0u, sure = 0u;
        float biggest = kMinusHuge;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float x = (live >> e & 1u) ? dot[e] : kMinusHuge;       // a missing token counts for nothing
            z += fast_exp2(x - ref);
            biggest = fmaxf(biggest, x);
            staged |= (unsigned)(x >= lo) << e;
            sure |= (unsigned)(x > hi) << e;
        }
        far_above |= biggest > ref + kRefSlack;
        staged = (staged | in_window) & live;
        sure = (sure | in_window) & live;
        // One scan for three counts (each at most 256): staged | candidates << 10 | sure << 20.
        const unsigned cands = staged & ~sure;
        const int mine = __popc(staged) | __popc(cands) << 10 | __popc(sure) << 20;
        int incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        const int seg = seg_begin / kSegmentTokens;
        // the segment's candidates take consecutive slots of the row's list: one atomic per segment
        int cand_base = 0;
        if (lane == 0) {
            p.seg_count[(int64_t)pair * p.segments + seg] = total & 1023;
            p.seg_final[(int64_t)pair * p.segments + seg] = total >> 20;
            if ((total >> 10 & 1023) != 0) cand_base = atomicAdd(&row->n_cand, total >> 10 & 1023);
        }
        cand_base = __shfl_sync(0xffffffffu, cand_base, 0);
        // The staged tokens go, in position order, through the warp's piece of shared memory (one
        // predicated 8-byte store per token, no branch), and from there to global memory as whole
        // runs written by consecutive lanes; which of them are candidates (not surely selected,
        // not in the window) is decided again on the way out, their slots come from a vote.
        unsigned at = buf + ((incl - mine) & 1023) * 8;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %0, 0;\n\t@p st.shared.v2.b32 [%1], {%2, %3};\n\t}"
                         :: "r"(staged >> e & 1u), "r"(at), "r"(__float_as_uint(dot[e])), "r"(i + e) : "memory");
            at += (staged >> e & 1u) * 8;
        }
        __syncwarp();
        const int n = total & 1023;
        for (int t0 = 0; t0 < n; t0 += 32) {
            const int t = t0 + lane;
            const bool have = t < n && bounds_ok(seg_begin + t < p.score_stride, p.status);
            uint2 v = make_uint2(0u, 0u);
            if (have) {
                asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(buf + t * 8));
                stage_x[seg_begin + t] = __uint_as_float(v.x);
                stage_pos[seg_begin + t] = (int)v.y;
            }
            const bool between = have && !(__uint_as_float(v.x) > hi) && (int)v.y < window_from;
            const unsigned votes = __ballot_sync(0xffffffffu, between);
            if (between) {
                const int slot = cand_base + __popc(votes & ((1u << lane) - 1u));
                if (slot < p.cand_capacity) cand[slot] = make_uint2(ordered_key(__uint_as_float(v.x)), v.y);
            }
            cand_base += __popc(votes);
        }
        __syncwarp();                        // the piece of shared memory is reused by the next segment
    }
    z = block_sum(z, sh.red);
    if (tid == 0) p.blk_z[(int64_t)pair * p.score_blocks + block_in_row] = z;
    if (far_above) row->overflow = 1;
}

// grid pairs, kResolveThreads threads (512, or 256 when the candidate lists are short), dynamic
// shared memory cand_capacity * 4 bytes (the candidates' keys; their positions are read from
// the list in global memory, which keeps the block small enough for many to share an SM).
// cand_capacity <= kCandidates.
template <int kResolveThreads>
__global__ void __launch_bounds__(kResolveThreads)
sparf_resolve_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    extern __shared__ __align__(16) unsigned keys[];
    __shared__ SelectCore sh;
    const int pair = blockIdx.x, tid = threadIdx.x;
    const int b = pair / p.heads;
    SelectRow *row = p.rows_state + pair;
    if (row->solved) return;                                 // k == 0
    const int S = sparf_seq_len(p, b, false);
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    const int segments = (S + kSegmentTokens - 1) / kSegmentTokens;
    int32_t *seg_final = p.seg_final + (int64_t)pair * p.segments;
    int sure = 0;
    for (int s = tid; s < segments; s += kResolveThreads) sure += seg_final[s];
    sure = block_sum(sure, reinterpret_cast<int *>(sh.red_f));
    const int n = row->n_cand, need = k - sure;
    // The bracket must hold the threshold: the sure tokens do not exceed k, and together with
    // the candidates they reach it.
    if (row->overflow || n > p.cand_capacity || need < 0 || need > n) {               // unsolved
        if (tid == 0) atomicAdd(p.unsolved, 1);
        return;
    }
    if (need == 0) {                     // exactly the sure tokens: every logit above the upper bound, no candidate
        if (tid == 0) {
            row->tau = ordered_key(row->hi);
            row->idx_cut = -1;
            row->solved = 1;
        }
        return;
    }
    const uint2 *cand = p.row_cand + (int64_t)pair * p.cand_capacity;
    for (int t = tid; t < n; t += kResolveThreads) keys[t] = cand[t].x;
    __syncthreads();
    // the need-th largest key, and how many of the keys equal to it are taken
    exact_threshold<kResolveThreads>(sh, n, need, [](int) { return true; }, [&](int i) { return keys[i]; });
    const unsigned tau = sh.tau;
    const int take = sh.take_equal;
    // among the keys equal to tau the `take` lowest positions: the take-th smallest position,
    // found as the take-th largest of the complemented positions
    __syncthreads();
    int ties = 0;
    for (int t = tid; t < n; t += kResolveThreads) ties += keys[t] == tau;
    ties = block_sum(ties, reinterpret_cast<int *>(sh.red_f));
    int cut = 0x7fffffff;                                    // every token that ties with tau is taken ...
    if (take < ties) {                                       // ... unless the cut falls among them (uniform)
        exact_threshold<kResolveThreads>(sh, n, take, [&](int i) { return keys[i] == tau; },
                                         [&](int i) { return ~cand[i].y; });
        cut = (int)~sh.tau;
    }
    for (int t = tid; t < n; t += kResolveThreads) {
        if (keys[t] >= tau) {
            const int where = (int)cand[t].y;
            if (keys[t] > tau || where <= cut) atomicAdd(&seg_final[where / kSegmentTokens], 1);
        }
    }
    if (tid == 0) {
        row->tau = tau;
        row->idx_cut = cut;
        row->solved = 1;
    }
}

// grid pairs * score_blocks, kEmitThreads threads: the staged tokens of the block's segments,
// one warp per segment at a time (4 consecutive entries per lane and pass), no block barrier.
__global__ void __launch_bounds__(kEmitThreads)
sparf_emit_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    constexpr int kSegmentsPerBlock = kScoreBlockTokens / kSegmentTokens;
    static_assert(kSegmentsPerBlock == 32, "a lane per segment of the block in the prefix scan");
    const int pair = blockIdx.x / p.score_blocks, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int block_in_row = blockIdx.x - pair * p.score_blocks;
    const int b = pair / p.heads, h = pair - b * p.heads;
    const SelectRow row = p.rows_state[pair];
    if (!row.solved) return;
    const int S = sparf_seq_len(p, b, false);
    const int begin = block_in_row * kScoreBlockTokens;
    if (begin >= S) return;
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    if (k == 0) return;
    const int window_from = S - min(p.window, k);
    const int first_seg = begin / kSegmentTokens;
    const int row_segs = (S + kSegmentTokens - 1) / kSegmentTokens;
    const int32_t *seg_count = p.seg_count + (int64_t)pair * p.segments;
    const int32_t *seg_final = p.seg_final + (int64_t)pair * p.segments;
    // Where a segment's selected tokens go: everything selected before it in the row.  Each warp
    // adds up the segments before the block and scans the block's own 32 (no shared memory).
    int before = 0;
    for (int s = lane; s < first_seg; s += 32) before += seg_final[s];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) before += __shfl_xor_sync(0xffffffffu, before, off);
    const int own = first_seg + lane < row_segs ? seg_final[first_seg + lane] : 0;
    int own_incl = own;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, own_incl, off);
        if (lane >= off) own_incl += up;
    }
    const int own_excl = own_incl - own;                     // lane j: selected in the block's segments before j

    const int T = p.block_tokens;
    const int t_shift = (T & (T - 1)) == 0 ? __ffs(T) - 1 : -1;      // blocks of 2^n tokens: no division per token
    const int32_t *table_row = p.block_table + (int64_t)b * p.max_blocks_per_seq;
    const float *stage_x = p.scores + (int64_t)pair * p.score_stride;
    const int32_t *stage_pos = p.stage_pos + (int64_t)pair * p.score_stride;
    int32_t *rows = p.row_ids + (int64_t)pair * p.max_k;
    int32_t *sel = p.selected ? p.selected + (int64_t)pair * p.max_k : nullptr;
    // Eight lanes per segment, four segments per warp at a time (a segment holds a few dozen
    // staged tokens, so a whole warp per segment would leave most lanes idle): lane group g of
    // warp w takes segment 4 w + g of the block, 4 consecutive entries per lane and pass.
    const int group = lane >> 3, sub = lane & 7;
    const int j = warp * 4 + group;
    const int seg = first_seg + j;
    const bool have = seg < row_segs;
    const int n = have ? seg_count[seg] : 0;
    const int base = seg * kSegmentTokens;
    int at = before + __shfl_sync(0xffffffffu, own_excl, j);
    float mass = 0.f;
    int longest = n;
#pragma unroll
    for (int off = 16; off >= 8; off >>= 1) longest = max(longest, __shfl_xor_sync(0xffffffffu, longest, off));
    for (int t0 = 0; t0 < longest; t0 += 32) {               // staged entries are dense from the segment's start
        const int t = t0 + sub * 4;
        float4 xq = make_float4(0.f, 0.f, 0.f, 0.f);
        int4 pq = make_int4(0, 0, 0, 0);
        if (t < n) {                                         // 16-byte loads: every offset is a multiple of 4
            xq = *reinterpret_cast<const float4 *>(stage_x + base + t);
            pq = *reinterpret_cast<const int4 *>(stage_pos + base + t);
        }
        const float x[4] = {xq.x, xq.y, xq.z, xq.w};
        const int pos[4] = {pq.x, pq.y, pq.z, pq.w};
        unsigned take = 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const unsigned key = ordered_key(x[e]);
            const bool chosen = pos[e] >= window_from || key > row.tau || (key == row.tau && pos[e] <= row.idx_cut);
            take |= (unsigned)(t + e < n && chosen) << e;
        }
        const int mine = __popc(take);
        int incl = mine;
#pragma unroll
        for (int off = 1; off < 8; off <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, off, 8);
            if (sub >= off) incl += up;
        }
        int dst = at + incl - mine;
        at += __shfl_sync(0xffffffffu, incl, 7, 8);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (take >> e & 1u) {
                const int i = pos[e];
                const int blk = t_shift >= 0 ? i >> t_shift : i / T, slot = i - blk * T;
                const int phys = bounds_ok(blk < p.max_blocks_per_seq && dst < p.max_k, p.status) ? table_row[blk] : -1;
                const bool ok = phys >= 0 && (int64_t)phys < p.num_phys_blocks;
                if (!ok && p.status) atomicOr(p.status, kFlagBlockRange);
                if (dst < p.max_k) {         // always true for a consistent count; guards the buffer
                    rows[dst] = ok ? (phys * p.heads + h) * T + slot : 0;
                    if (sel) sel[dst] = i;
                }
                mass += fast_exp2(x[e] - row.ref);
                ++dst;
            }
        }
    }
#pragma unroll
    for (int off = 4; off >= 1; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
    if (have && sub == 0) p.seg_mass[(int64_t)pair * p.segments + seg] = mass;
}

// grid pairs, 64 threads.
__global__ void __launch_bounds__(64)
sparf_finish_kernel(const SparfParams p)
{
    allow_next_kernel();
    wait_for_previous_kernels();
    __shared__ float part[64];
    const int pair = blockIdx.x, tid = threadIdx.x;
    const int b = pair / p.heads;
    const SelectRow row = p.rows_state[pair];
    if (!row.solved) return;
    const int S = sparf_seq_len(p, b, false);
    const int k = min(S, min(max(p.k_tokens[b], 0), p.max_k));
    if (p.selected)
        for (int t = k + tid; t < p.max_k; t += 64) p.selected[(int64_t)pair * p.max_k + t] = -1;
    // selected mass: every thread adds its share of the segments, thread 0 the 64 shares (fixed order)
    float mine = 0.f;
    const int segs = k > 0 ? (S + kSegmentTokens - 1) / kSegmentTokens : 0;
    for (int s = tid; s < segs; s += 64) mine += p.seg_mass[(int64_t)pair * p.segments + s];
    part[tid] = mine;
    __syncthreads();
    if (tid == 0) {
        float alpha = 0.f;
        if (k > 0) {
            float mass = 0.f, z = 0.f;
            for (int t = 0; t < 64; ++t) mass += part[t];
            const int blocks = (S + kScoreBlockTokens - 1) / kScoreBlockTokens;
            for (int c = 0; c < blocks; ++c) z += p.blk_z[(int64_t)pair * p.score_blocks + c];
            alpha = mass / z;
        }
        p.stats[pair] = make_float2(alpha, (float)k);
        if (p.alpha_out) p.alpha_out[pair] = alpha;
    }
}

}  // namespace instinfer
