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
constexpr int kTailChunk = 256;          // automatic plan: size of the short chunks at the start of a sequence
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

// The same with the grid cut into thread-block clusters of `cluster` consecutive blocks
// (grid must be a multiple of it).  No fallback: a refused cluster launch is an error.
template <typename... Params>
inline cudaError_t launch_clustered(void (*kernel)(Params...), unsigned grid, unsigned cluster, unsigned block,
                                    size_t smem, cudaStream_t stream, const Params &...params)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, params...);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        cfg.numAttrs = 1;                // without the programmatic overlap
        err = cudaLaunchKernelEx(&cfg, kernel, params...);
    }
    return err;
}

struct SplitPlan {
    int32_t chunk_tokens;   // size of the n_big long chunks, which follow the short ones
    int32_t n_big;
    int32_t tail_chunk;     // size of the n_splits - n_big short chunks at the start of a sequence
    int32_t n_splits;
    bool cluster;           // small problem: the chunks of a (sequence, head) form one thread-block
                            // cluster that merges its partials itself (no merge kernel)
};

// Cuts are at fixed logical token positions, the same for every sequence, so a result never
// depends on the physical placement of blocks.  Blocks are scheduled chunk-major with the
// short chunks last.  The short chunks cover the first tokens of a sequence, which every
// sequence of a ragged batch has: a launch then ends on about kTailWaves waves of short
// blocks whatever the lengths are (SMs idle only while the last short blocks finish),
// without paying the per-block overhead of small chunks everywhere.
// What differs between the kernels that share the planner.
struct PlanRules {
    int ctas_per_sm;
    int target_waves;
    int chunk_ceiling;
    int tail_chunk_tokens;       // 0: no short chunks at the end of long sequences
    int block_overhead_tokens;   // > 0: choose the chunk count by modelled time (see make_plan)
    bool allow_cluster;          // the kernel has the cluster form for small problems
    int chunk_granule;           // chunk lengths are multiples of this (0: kChunkGranule)
};
constexpr PlanRules kOneRowRules = {kCtasPerSm, kTargetWaves, kChunkCeiling, kTailChunk, 0, true, 0};
constexpr PlanRules kNoClusterRules = {kCtasPerSm, kTargetWaves, kChunkCeiling, kTailChunk, 0, false, 0};
constexpr int kClusterMaxChunks = 8;     // portable cluster size
constexpr int kClusterMaxChunkTokens = 512;

inline SplitPlan make_plan(int64_t pairs, int32_t max_seq_len, const PlanRules &rules = kOneRowRules)
{
    SplitPlan plan;
    plan.cluster = false;
    if (g_forced_chunk > 0) {               // uniform chunks, no short ones
        plan.chunk_tokens = plan.tail_chunk = g_forced_chunk;
        plan.n_big = (int32_t)ceil_div(max_seq_len, g_forced_chunk);
        plan.n_splits = plan.n_big;
        return plan;
    }
    const int64_t slots = (int64_t)sm_count() * rules.ctas_per_sm;
    const int64_t granule = rules.chunk_granule > 0 ? rules.chunk_granule : kChunkGranule;
    if (rules.allow_cluster) {
        // Small problems are bound by launch and memory latency, not by bandwidth: at most 8
        // chunks per sequence, all resident at once, merged inside the kernel by a cluster.
        const int64_t chunk = ceil_div(ceil_div(max_seq_len, kClusterMaxChunks), kChunkGranule) * kChunkGranule;
        const int64_t n = ceil_div(max_seq_len, chunk);
        if (n >= 2 && chunk <= kClusterMaxChunkTokens && pairs * n <= 2 * slots) {
            plan.chunk_tokens = plan.tail_chunk = (int32_t)chunk;
            plan.n_big = plan.n_splits = (int32_t)n;
            plan.cluster = true;
            return plan;
        }
    }
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
            const int64_t len = ceil_div(ceil_div(max_seq_len, c), granule) * granule;
            const int64_t cost = ceil_div(pairs * ceil_div(max_seq_len, len), slots) *
                                 (len + rules.block_overhead_tokens);
            if (best < 0 || cost < best) {
                best = cost;
                n = c;
            }
        }
    }
    int64_t chunk = ceil_div(ceil_div(max_seq_len, n), granule) * granule;
    // Short region: about kTailWaves waves of tail_chunk-token blocks at the start of every
    // sequence, at most a quarter of the longest; none when the chunks are that short anyway.
    const int64_t tail_chunk = rules.tail_chunk_tokens > 0 ? rules.tail_chunk_tokens : kTailChunk;
    int64_t short_tokens = ceil_div(slots * kTailWaves, pairs) * tail_chunk;
    if (short_tokens > max_seq_len / 4) short_tokens = max_seq_len / 4 / tail_chunk * tail_chunk;
    if (chunk <= 2 * tail_chunk || short_tokens < tail_chunk || rules.tail_chunk_tokens <= 0) short_tokens = 0;
    if (short_tokens > 0)
        chunk = ceil_div(ceil_div(max_seq_len - short_tokens, n), granule) * granule;
    const int64_t n_short = short_tokens > 0 ? short_tokens / tail_chunk : 0;
    plan.chunk_tokens = (int32_t)chunk;
    plan.n_big = (int32_t)ceil_div(max_seq_len - short_tokens, chunk);
    plan.tail_chunk = short_tokens > 0 ? (int32_t)tail_chunk : (int32_t)chunk;
    plan.n_splits = (int32_t)(n_short + plan.n_big);
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
