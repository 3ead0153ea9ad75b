// Host-side helpers shared by the parts of the C ABI (instinfer_api.cu, api_*.inl): argument checks, the
// launch helper, and the split planner.  Nothing here allocates or synchronises.
#pragma once

#include "../../include/instinfer.h"

#include <cmath>
#include <cuda_runtime.h>
#include <stdint.h>

#include "decode_attention_kernels.cuh"

namespace instinfer {
namespace api {

constexpr int kMaxDevices = 64;
constexpr int kChunkGranule = 64;        // chunk_tokens is a multiple of this
constexpr int kChunkCeiling = 2048;      // automatic plan: chunk never longer than this ...
constexpr int kChunkFloor = 256;         // ... nor shorter than this, sequence permitting
constexpr int kTargetWaves = 8;          // automatic plan: aim for this many waves of blocks
constexpr int kTailChunk = 256;          // automatic plan: chunk size at the end of long sequences
constexpr int kTailWaves = 2;            // ... covering about this many waves of blocks

inline int g_forced_chunk = 0;
inline cudaEvent_t g_before_split = nullptr;    // measurement aid, see instinfer_set_timing_events
inline cudaEvent_t g_after_split = nullptr;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool usable(const void *p) { return p != nullptr && aligned16(p); }

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// SM count of the current device; 148 (B200) when no device can be asked.
inline int sm_count()
{
    static int cached[kMaxDevices] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return 148;
    }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = 148;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

// Launch with programmatic stream serialization: the kernel may be scheduled while the
// previous kernel in the stream drains; it orders itself with griddepcontrol.wait.  Falls
// back to an ordinary launch if the runtime refuses the attribute.
template <typename... Params>
inline cudaError_t launch_overlapped(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem,
                              cudaStream_t stream, const Params &...params)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, params...);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        cfg.numAttrs = 0;
        err = cudaLaunchKernelEx(&cfg, kernel, params...);
    }
    return err;
}

struct SplitPlan {
    int32_t chunk_tokens;   // size of the first n_big chunks
    int32_t n_big;
    int32_t tail_chunk;     // size of the chunks after them
    int32_t n_splits;
};

// Cuts are at fixed logical token positions, the same for every sequence, so a result never
// depends on the physical placement of blocks.  Blocks are scheduled chunk-major, so the
// chunks at the end of the longest sequences run last: making those short keeps the tail of
// a launch (SMs idling while the last blocks finish) short without paying the per-block
// overhead of small chunks everywhere.
// What differs between the kernels that share the planner.
struct PlanRules {
    int ctas_per_sm;
    int target_waves;
    int chunk_ceiling;
    int tail_chunk_tokens;       // 0: no short chunks at the end of long sequences
    int block_overhead_tokens;   // > 0: choose the chunk count by modelled time (see make_plan)
};
constexpr PlanRules kOneRowRules = {kCtasPerSm, kTargetWaves, kChunkCeiling, kTailChunk, 0};

inline SplitPlan make_plan(int64_t pairs, int32_t max_seq_len, const PlanRules &rules = kOneRowRules)
{
    SplitPlan plan;
    if (g_forced_chunk > 0) {
        plan.chunk_tokens = plan.tail_chunk = g_forced_chunk;
        plan.n_big = (int32_t)ceil_div(max_seq_len, g_forced_chunk);
        plan.n_splits = plan.n_big;
        return plan;
    }
    const int64_t slots = (int64_t)sm_count() * rules.ctas_per_sm;
    const int64_t fewest = ceil_div(max_seq_len, rules.chunk_ceiling);
    // Small problems that cannot fill the GPU with kChunkFloor-token chunks are latency-bound:
    // cut them down to the granule so that more blocks share the work.
    const int64_t floor_tokens = pairs * ceil_div(max_seq_len, kChunkFloor) < slots ? kChunkGranule : kChunkFloor;
    const int64_t most = ceil_div(max_seq_len, floor_tokens);
    int64_t n = ceil_div(slots * rules.target_waves, pairs);
    if (n > most) n = most;
    if (n < fewest) n = fewest;
    if (rules.block_overhead_tokens > 0) {
        // Latency-bound blocks of equal length run in whole waves, so time goes as
        // (waves of blocks) x (chunk length + a fixed per-block cost): take the chunk count
        // that minimises it, assuming sequences of max_seq_len.
        int64_t best = -1;
        const int64_t last = most < fewest + 96 ? most : fewest + 96;
        for (int64_t c = fewest; c <= last; ++c) {
            const int64_t len = ceil_div(ceil_div(max_seq_len, c), kChunkGranule) * kChunkGranule;
            const int64_t cost = ceil_div(pairs * ceil_div(max_seq_len, len), slots) *
                                 (len + rules.block_overhead_tokens);
            if (best < 0 || cost < best) {
                best = cost;
                n = c;
            }
        }
    }
    int64_t chunk = ceil_div(ceil_div(max_seq_len, n), kChunkGranule) * kChunkGranule;
    // Tail region: about kTailWaves waves of kTailChunk-token blocks at the end of the longest
    // sequences, at most a quarter of the sequence; none when the chunks are that short anyway.
    const int64_t tail_chunk = rules.tail_chunk_tokens > 0 ? rules.tail_chunk_tokens : kTailChunk;
    int64_t tail_tokens = ceil_div(slots * kTailWaves, pairs) * tail_chunk;
    if (tail_tokens > max_seq_len / 4) tail_tokens = max_seq_len / 4 / tail_chunk * tail_chunk;
    if (chunk <= 2 * tail_chunk || tail_tokens < tail_chunk || rules.tail_chunk_tokens <= 0) tail_tokens = 0;
    if (tail_tokens > 0)      // rounded down, so that at least tail_tokens are left for the tail
        chunk = (max_seq_len - tail_tokens) / n / kChunkGranule * kChunkGranule;
    int64_t big_span = n * chunk;
    while (big_span - chunk >= max_seq_len) big_span -= chunk;
    plan.chunk_tokens = (int32_t)chunk;
    plan.n_big = (int32_t)(big_span / chunk);
    plan.tail_chunk = tail_tokens > 0 ? (int32_t)tail_chunk : (int32_t)chunk;
    plan.n_splits = plan.n_big + (big_span < max_seq_len
                                      ? (int32_t)ceil_div(max_seq_len - big_span, plan.tail_chunk) : 0);
    return plan;
}

inline size_t workspace_for(int64_t pairs, const SplitPlan &plan)
{
    const size_t floats = (size_t)pairs * (size_t)plan.n_splits * (kHeadDim + 1);
    return (floats * sizeof(float) + 255) / 256 * 256 + 256;
}

// The appends are bit copies and take every head size the attention entry points take.
inline bool append_head_dim_ok(int32_t head_dim) { return head_dim == 64 || head_dim == 128 || head_dim == 256; }

inline bool sizes_ok(int32_t batch, int32_t heads, int32_t max_seq_len)
{
    if (batch < 0 || heads <= 0 || max_seq_len <= 0) return false;
    return (int64_t)batch * heads <= (int64_t)1 << 24;     // keeps every grid below 2^31 blocks
}

}  // namespace api
}  // namespace instinfer
