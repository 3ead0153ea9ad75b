// C ABI of the decode-attention library: argument checks, the split plan, the workspace
// layout and the launches.  Nothing here allocates or synchronises; all work is enqueued on
// the caller's stream.
#include "../../include/instinfer.h"

#include <cmath>

#include "allgather_merge_kernel.cuh"
#include "decode_attention_kernels.cuh"
#include "grouped_attention_kernels.cuh"
#include "kv_append_kernel.cuh"
#include "sparf_kernels.cuh"

namespace {

using namespace instinfer;

constexpr int kMaxDevices = 64;
constexpr int kChunkGranule = 64;        // chunk_tokens is a multiple of this
constexpr int kChunkCeiling = 2048;      // automatic plan: chunk never longer than this ...
constexpr int kChunkFloor = 256;         // ... nor shorter than this, sequence permitting
constexpr int kTargetWaves = 8;          // automatic plan: aim for this many waves of blocks
constexpr int kTailChunk = 256;          // automatic plan: chunk size at the end of long sequences
constexpr int kTailWaves = 2;            // ... covering about this many waves of blocks

int g_forced_chunk = 0;
cudaEvent_t g_before_split = nullptr;    // measurement aid, see instinfer_set_timing_events
cudaEvent_t g_after_split = nullptr;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool usable(const void *p) { return p != nullptr && aligned16(p); }

int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// SM count of the current device; 148 (B200) when no device can be asked.
int sm_count()
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
cudaError_t launch_overlapped(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem,
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
    bool short_tail_chunks;
    int block_overhead_tokens;   // > 0: choose the chunk count by modelled time (see make_plan)
};
constexpr PlanRules kOneRowRules = {kCtasPerSm, kTargetWaves, kChunkCeiling, true, 0};

SplitPlan make_plan(int64_t pairs, int32_t max_seq_len, const PlanRules &rules = kOneRowRules)
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
    int64_t tail_tokens = ceil_div(slots * kTailWaves, pairs) * kTailChunk;
    if (tail_tokens > max_seq_len / 4) tail_tokens = max_seq_len / 4 / kTailChunk * kTailChunk;
    if (chunk <= 2 * kTailChunk || tail_tokens < kTailChunk || !rules.short_tail_chunks) tail_tokens = 0;
    if (tail_tokens > 0)      // rounded down, so that at least tail_tokens are left for the tail
        chunk = (max_seq_len - tail_tokens) / n / kChunkGranule * kChunkGranule;
    int64_t big_span = n * chunk;
    while (big_span - chunk >= max_seq_len) big_span -= chunk;
    plan.chunk_tokens = (int32_t)chunk;
    plan.n_big = (int32_t)(big_span / chunk);
    plan.tail_chunk = tail_tokens > 0 ? kTailChunk : (int32_t)chunk;
    plan.n_splits = plan.n_big + (big_span < max_seq_len
                                      ? (int32_t)ceil_div(max_seq_len - big_span, plan.tail_chunk) : 0);
    return plan;
}

size_t workspace_for(int64_t pairs, const SplitPlan &plan)
{
    const size_t floats = (size_t)pairs * (size_t)plan.n_splits * (kHeadDim + 1);
    return (floats * sizeof(float) + 255) / 256 * 256 + 256;
}

// The appends are bit copies and take every head size the attention entry points take.
bool append_head_dim_ok(int32_t head_dim) { return head_dim == 64 || head_dim == 128 || head_dim == 256; }

bool sizes_ok(int32_t batch, int32_t heads, int32_t max_seq_len)
{
    if (batch < 0 || heads <= 0 || max_seq_len <= 0) return false;
    return (int64_t)batch * heads <= (int64_t)1 << 24;     // keeps every grid below 2^31 blocks
}

int ensure_split_smem(bool paged)
{
    static bool done[kMaxDevices][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INSTINFER_ERR_CUDA;
    if (!done[dev][paged]) {
        const cudaError_t err = paged
            ? cudaFuncSetAttribute(decode_attn_split_kernel<Rows::kPaged>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, kSplitSmemBytes)
            : cudaFuncSetAttribute(decode_attn_split_kernel<Rows::kContiguous>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, kSplitSmemBytes);
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        done[dev][paged] = true;
    }
    return INSTINFER_OK;
}

// Bytes of finished fp16 rows parked in the workspace, behind the partials, by the
// head-sharded path when the plan has a single chunk.
size_t staging_for(int64_t pairs) { return ((size_t)pairs * kHeadDim * sizeof(__half) + 255) / 256 * 256; }

// gather == nullptr: outputs go to p.out.  Otherwise p.out is unused and every finished row
// is stored into all of gather->out (the fused all-gather of the head-sharded path).
int launch_attention(AttnParams p, bool paged, int32_t batch, void *workspace,
                     size_t workspace_bytes, cudaStream_t stream,
                     const GatherTargets *gather = nullptr)
{
    const int64_t pairs = (int64_t)batch * p.heads;
    const SplitPlan plan = make_plan(pairs, p.max_seq_len);
    const size_t partial_bytes = workspace_for(pairs, plan);
    if (workspace == nullptr || !aligned16(workspace) ||
        workspace_bytes < partial_bytes + (gather ? staging_for(pairs) : 0))
        return INSTINFER_ERR_WORKSPACE;
    if (pairs * plan.n_splits >= (int64_t)1 << 31) return INSTINFER_ERR_INVALID_ARG;
    p.chunk_tokens = plan.chunk_tokens;
    p.n_big = plan.n_big;
    p.tail_chunk = plan.tail_chunk;
    p.n_splits = plan.n_splits;
    p.pairs = (int32_t)pairs;
    p.part_o = static_cast<float *>(workspace);
    p.part_lse = p.part_o + (size_t)pairs * plan.n_splits * kHeadDim;
    GatherTargets targets = {};
    if (gather) {
        targets = *gather;
        p.out = reinterpret_cast<__half *>(static_cast<unsigned char *>(workspace) + partial_bytes);
        targets.staged = p.out;
    }

    const int rc = ensure_split_smem(paged);
    if (rc != INSTINFER_OK) return rc;
    const unsigned grid = (unsigned)(pairs * plan.n_splits);
    if (g_before_split) cudaEventRecord(g_before_split, stream);
    const bool timed = g_before_split != nullptr;          // event records break the overlap anyway
    cudaError_t err;
    if (paged)
        err = launch_overlapped(decode_attn_split_kernel<Rows::kPaged>, grid, kThreads, kSplitSmemBytes, stream, p);
    else
        err = launch_overlapped(decode_attn_split_kernel<Rows::kContiguous>, grid, kThreads, kSplitSmemBytes, stream, p);
    if (timed) cudaEventRecord(g_after_split, stream);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    if (gather) {
        err = launch_overlapped(lse_merge_allgather_kernel, (unsigned)pairs, kHeadDim, 0, stream, p, targets);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    } else if (plan.n_splits > 1) {
        err = launch_overlapped(lse_merge_kernel, (unsigned)pairs, kHeadDim, 0, stream, p);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    }
    return INSTINFER_OK;
}

// Built-in scratch for instinfer_decode_attention_static: lives in every GPU context that
// loads the library, from load until exit.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
constexpr size_t kStaticWorkspaceBytes = INSTINFER_STATIC_WORKSPACE_BYTES;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

// Device address of the built-in scratch on the current device, looked up once per device.
int static_workspace(void **address)
{
    static void *cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    if (cached[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        cached[dev] = ptr;
    }
    *address = cached[dev];
    return INSTINFER_OK;
}

}  // namespace

extern "C" {

int instinfer_kv_append(void *k_cache, void *v_cache, const void *k_new, const void *v_new,
                        const int32_t *seq_lens, const int32_t *block_table,
                        int32_t max_blocks_per_seq, int32_t block_tokens, int64_t num_phys_blocks,
                        int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max,
                        int32_t *status_flags, void *cuda_stream)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0) return INSTINFER_ERR_INVALID_ARG;
    if (!append_head_dim_ok(head_dim)) return INSTINFER_ERR_UNSUPPORTED;
    if ((int64_t)batch * heads > (int64_t)1 << 24) return INSTINFER_ERR_INVALID_ARG;
    if (block_table != nullptr) {
        if (max_blocks_per_seq <= 0 || block_tokens <= 0 || num_phys_blocks <= 0)
            return INSTINFER_ERR_INVALID_ARG;
        if (block_tokens % 8 != 0) return INSTINFER_ERR_UNSUPPORTED;
    } else if (s_max <= 0) {
        return INSTINFER_ERR_INVALID_ARG;
    }
    if (batch == 0) return INSTINFER_OK;
    if (!usable(k_cache) || !usable(v_cache) || !usable(k_new) || !usable(v_new) || seq_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;

    AppendParams p;
    p.k_cache = static_cast<uint4 *>(k_cache);
    p.v_cache = static_cast<uint4 *>(v_cache);
    p.k_new = static_cast<const uint4 *>(k_new);
    p.v_new = static_cast<const uint4 *>(v_new);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.status = status_flags;
    p.num_phys_blocks = num_phys_blocks;
    p.batch = batch;
    p.heads = heads;
    p.s_max = s_max;
    p.block_tokens = block_tokens;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.segs_per_row = head_dim / 8;
    const int64_t threads = (int64_t)batch * heads * p.segs_per_row;
    const unsigned grid = (unsigned)ceil_div(threads, kAppendThreads);
    const cudaError_t err = launch_overlapped(kv_append_kernel, grid, kAppendThreads, 0,
                                              static_cast<cudaStream_t>(cuda_stream), p);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? INSTINFER_OK : INSTINFER_ERR_CUDA;
}

int instinfer_kv_append_bulk(void *k_cache, void *v_cache, const void *k_new, const void *v_new,
                             const int32_t *seq_lens, const int32_t *new_lens,
                             const int32_t *block_table, int32_t max_blocks_per_seq,
                             int32_t block_tokens, int64_t num_phys_blocks, int32_t batch,
                             int32_t max_new, int32_t heads, int32_t head_dim, int32_t s_max,
                             int32_t *status_flags, void *cuda_stream)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0 || max_new < 0) return INSTINFER_ERR_INVALID_ARG;
    if (!append_head_dim_ok(head_dim)) return INSTINFER_ERR_UNSUPPORTED;
    if ((int64_t)batch * heads > (int64_t)1 << 24) return INSTINFER_ERR_INVALID_ARG;
    if (block_table != nullptr) {
        if (max_blocks_per_seq <= 0 || block_tokens <= 0 || num_phys_blocks <= 0)
            return INSTINFER_ERR_INVALID_ARG;
        if (block_tokens % 8 != 0) return INSTINFER_ERR_UNSUPPORTED;
    } else if (s_max <= 0) {
        return INSTINFER_ERR_INVALID_ARG;
    }
    if (batch == 0 || max_new == 0) return INSTINFER_OK;
    if (!usable(k_cache) || !usable(v_cache) || !usable(k_new) || !usable(v_new) ||
        seq_lens == nullptr || new_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;
    const int64_t threads = (int64_t)batch * max_new * heads * (head_dim / 8);
    const int64_t grid = ceil_div(threads, kAppendThreads);
    if (grid >= (int64_t)1 << 31) return INSTINFER_ERR_INVALID_ARG;

    BulkAppendParams q = {};
    AppendParams &p = q.base;
    p.k_cache = static_cast<uint4 *>(k_cache);
    p.v_cache = static_cast<uint4 *>(v_cache);
    p.k_new = static_cast<const uint4 *>(k_new);
    p.v_new = static_cast<const uint4 *>(v_new);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.status = status_flags;
    p.num_phys_blocks = num_phys_blocks;
    p.batch = batch;
    p.heads = heads;
    p.s_max = s_max;
    p.block_tokens = block_tokens;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.segs_per_row = head_dim / 8;
    q.new_lens = new_lens;
    q.max_new = max_new;
    kv_append_bulk_kernel<<<(unsigned)grid, kAppendThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(q);
    return cudaGetLastError() == cudaSuccess ? INSTINFER_OK : INSTINFER_ERR_CUDA;
}

int instinfer_decode_attention(void *out, float *lse, const void *q, const void *k_cache,
                               const void *v_cache, const int32_t *seq_lens, int32_t batch,
                               int32_t heads, int32_t head_dim, int32_t s_max,
                               int32_t max_seq_len, float scale, void *workspace,
                               size_t workspace_bytes, int32_t *status_flags, void *cuda_stream)
{
    if (head_dim <= 0 || !sizes_ok(batch, heads, max_seq_len) || s_max <= 0 || max_seq_len > s_max)
        return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return INSTINFER_ERR_UNSUPPORTED;
    if (!std::isfinite(scale)) return INSTINFER_ERR_INVALID_ARG;
    if (batch == 0) return INSTINFER_OK;
    if (!usable(out) || !usable(q) || !usable(k_cache) || !usable(v_cache) || seq_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;

    AttnParams p = {};
    p.q = static_cast<const __half *>(q);
    p.k = static_cast<const __half *>(k_cache);
    p.v = static_cast<const __half *>(v_cache);
    p.seq_lens = seq_lens;
    p.out = static_cast<__half *>(out);
    p.lse = lse;
    p.status = status_flags;
    p.heads = heads;
    p.s_max = s_max;
    p.max_seq_len = max_seq_len;
    p.scale_log2e = scale * 1.44269504088896340736f;
    return launch_attention(p, false, batch, workspace, workspace_bytes,
                            static_cast<cudaStream_t>(cuda_stream));
}

int instinfer_decode_attention_paged(void *out, float *lse, const void *q, const void *k_pool,
                                     const void *v_pool, const int32_t *block_table,
                                     const int32_t *seq_lens, int32_t batch, int32_t heads,
                                     int32_t head_dim, int32_t block_tokens,
                                     int32_t max_blocks_per_seq, int64_t num_phys_blocks,
                                     int32_t max_seq_len, float scale, void *workspace,
                                     size_t workspace_bytes, int32_t *status_flags,
                                     void *cuda_stream)
{
    if (head_dim <= 0 || !sizes_ok(batch, heads, max_seq_len) || block_tokens <= 0 ||
        max_blocks_per_seq <= 0 || num_phys_blocks <= 0)
        return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || block_tokens % 8 != 0) return INSTINFER_ERR_UNSUPPORTED;
    if ((int64_t)max_seq_len > (int64_t)max_blocks_per_seq * block_tokens || !std::isfinite(scale))
        return INSTINFER_ERR_INVALID_ARG;
    if (batch == 0) return INSTINFER_OK;
    if (!usable(out) || !usable(q) || !usable(k_pool) || !usable(v_pool) || seq_lens == nullptr ||
        block_table == nullptr)
        return INSTINFER_ERR_INVALID_ARG;

    AttnParams p = {};
    p.q = static_cast<const __half *>(q);
    p.k = static_cast<const __half *>(k_pool);
    p.v = static_cast<const __half *>(v_pool);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.out = static_cast<__half *>(out);
    p.lse = lse;
    p.status = status_flags;
    p.num_phys_blocks = num_phys_blocks;
    p.heads = heads;
    p.block_tokens = block_tokens;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.max_seq_len = max_seq_len;
    p.scale_log2e = scale * 1.44269504088896340736f;
    return launch_attention(p, true, batch, workspace, workspace_bytes,
                            static_cast<cudaStream_t>(cuda_stream));
}

int instinfer_decode_attention_static(void *out, float *lse, const void *q, const void *k_cache,
                                      const void *v_cache, const int32_t *block_table,
                                      const int32_t *seq_lens, int32_t batch, int32_t heads,
                                      int32_t head_dim, int32_t s_max, int32_t block_tokens,
                                      int32_t max_blocks_per_seq, int64_t num_phys_blocks,
                                      int32_t max_seq_len, float scale, int32_t *status_flags,
                                      void *cuda_stream)
{
    // Size check first: it needs no device and must not depend on the set-up below.
    if (head_dim == kHeadDim && sizes_ok(batch, heads, max_seq_len) && batch > 0 &&
        workspace_for((int64_t)batch * heads, make_plan((int64_t)batch * heads, max_seq_len)) >
            kStaticWorkspaceBytes)
        return INSTINFER_ERR_WORKSPACE;
    void *scratch = nullptr;
    if (batch > 0) {
        const int rc = static_workspace(&scratch);
        if (rc != INSTINFER_OK) return rc;
    }
    if (block_table == nullptr)
        return instinfer_decode_attention(out, lse, q, k_cache, v_cache, seq_lens, batch, heads,
                                          head_dim, s_max, max_seq_len, scale, scratch,
                                          kStaticWorkspaceBytes, status_flags, cuda_stream);
    return instinfer_decode_attention_paged(out, lse, q, k_cache, v_cache, block_table, seq_lens,
                                            batch, heads, head_dim, block_tokens,
                                            max_blocks_per_seq, num_phys_blocks, max_seq_len,
                                            scale, scratch, kStaticWorkspaceBytes, status_flags,
                                            cuda_stream);
}

int instinfer_decode_attention_allgather(void *const *out_all, int32_t n_ranks, float *lse,
                                         const void *q, const void *k_cache, const void *v_cache,
                                         const int32_t *block_table, const int32_t *seq_lens,
                                         int32_t batch, int32_t heads, int32_t head_offset,
                                         int32_t total_heads, int32_t head_dim, int32_t s_max,
                                         int32_t block_tokens, int32_t max_blocks_per_seq,
                                         int64_t num_phys_blocks, int32_t max_seq_len, float scale,
                                         void *workspace, size_t workspace_bytes,
                                         int32_t *status_flags, void *cuda_stream)
{
    const bool paged = block_table != nullptr;
    if (head_dim <= 0 || !sizes_ok(batch, heads, max_seq_len) || out_all == nullptr ||
        n_ranks < 1 || n_ranks > kMaxRanks || head_offset < 0 || total_heads <= 0 ||
        (int64_t)head_offset + heads > total_heads || !std::isfinite(scale))
        return INSTINFER_ERR_INVALID_ARG;
    if (paged) {
        if (block_tokens <= 0 || max_blocks_per_seq <= 0 || num_phys_blocks <= 0 ||
            (int64_t)max_seq_len > (int64_t)max_blocks_per_seq * block_tokens)
            return INSTINFER_ERR_INVALID_ARG;
    } else if (s_max <= 0 || max_seq_len > s_max) {
        return INSTINFER_ERR_INVALID_ARG;
    }
    if (head_dim != kHeadDim || (paged && block_tokens % 8 != 0)) return INSTINFER_ERR_UNSUPPORTED;
    if (batch == 0) return INSTINFER_OK;
    if (!usable(q) || !usable(k_cache) || !usable(v_cache) || seq_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;

    GatherTargets targets = {};
    for (int r = 0; r < n_ranks; ++r) {
        if (!usable(out_all[r])) return INSTINFER_ERR_INVALID_ARG;
        targets.out[r] = static_cast<__half *>(out_all[r]);
    }
    targets.n_ranks = n_ranks;
    targets.head_offset = head_offset;
    targets.total_heads = total_heads;

    AttnParams p = {};
    p.q = static_cast<const __half *>(q);
    p.k = static_cast<const __half *>(k_cache);
    p.v = static_cast<const __half *>(v_cache);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.lse = lse;
    p.status = status_flags;
    p.num_phys_blocks = paged ? num_phys_blocks : 0;
    p.heads = heads;
    p.s_max = paged ? 0 : s_max;
    p.block_tokens = paged ? block_tokens : 0;
    p.max_blocks_per_seq = paged ? max_blocks_per_seq : 0;
    p.max_seq_len = max_seq_len;
    p.scale_log2e = scale * 1.44269504088896340736f;
    return launch_attention(p, paged, batch, workspace, workspace_bytes,
                            static_cast<cudaStream_t>(cuda_stream), &targets);
}

size_t instinfer_allgather_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim,
                                           int32_t max_seq_len)
{
    if (head_dim != kHeadDim || !sizes_ok(batch, heads, max_seq_len)) return 0;
    const int64_t pairs = (int64_t)batch * heads;
    if (pairs == 0) return 256;
    return workspace_for(pairs, make_plan(pairs, max_seq_len)) + staging_for(pairs);
}

extern "C++" {
namespace {

// The grouped kernel's blocks are heavier (query fragments to load, 16 rows to merge at the
// end: about the cost of 20 tiles) and its warps are latency-bound, so a launch takes whole
// waves of blocks: the chunk count is chosen by that model, chunks up to 4096 tokens, no
// short tail chunks.
PlanRules grouped_rules(int32_t head_dim)
{
    const int ctas = head_dim == 64 ? GroupedGeometry<64>::kCtasPerSm
                   : head_dim == 128 ? GroupedGeometry<128>::kCtasPerSm : GroupedGeometry<256>::kCtasPerSm;
    return PlanRules{ctas, 2, 4096, false, 320};
}

size_t grouped_workspace_for(int64_t pairs, int32_t rows, int32_t head_dim, const SplitPlan &plan)
{
    const size_t floats = (size_t)pairs * (size_t)plan.n_splits * rows * (head_dim + 1);
    return (floats * sizeof(float) + 255) / 256 * 256 + 256;
}

template <int D, bool kPaged>
int launch_grouped(const GroupedParams &p, unsigned grid, cudaStream_t stream)
{
    static bool done[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INSTINFER_ERR_CUDA;
    if (!done[dev]) {
        if (cudaFuncSetAttribute(grouped_attn_split_kernel<D, kPaged>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 GroupedGeometry<D>::kSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        done[dev] = true;
    }
    cudaError_t err = launch_overlapped(grouped_attn_split_kernel<D, kPaged>, grid, kThreads,
                                        GroupedGeometry<D>::kSmemBytes, stream, p);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    if (p.a.n_splits > 1) {
        err = launch_overlapped(grouped_merge_kernel<D>, (unsigned)(p.a.pairs * p.rows), D, 0, stream, p);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    }
    return INSTINFER_OK;
}

// Shape checks shared by the entry point and its workspace query.
int grouped_shape(int32_t batch, int32_t q_tokens, int32_t q_heads, int32_t kv_heads,
                  int32_t head_dim, int32_t max_seq_len)
{
    if (head_dim <= 0 || q_tokens <= 0 || q_heads <= 0 || kv_heads <= 0 || q_heads % kv_heads != 0 ||
        !sizes_ok(batch, kv_heads, max_seq_len))
        return INSTINFER_ERR_INVALID_ARG;
    if ((head_dim != 64 && head_dim != 128 && head_dim != 256) ||
        (int64_t)(q_heads / kv_heads) * q_tokens > kGroupRows)
        return INSTINFER_ERR_UNSUPPORTED;
    return INSTINFER_OK;
}

}  // namespace
}  // extern "C++"

int instinfer_decode_attention_grouped(void *out, float *lse, const void *q, const void *k_cache,
                                       const void *v_cache, const int32_t *block_table,
                                       const int32_t *seq_lens, int32_t batch, int32_t q_tokens,
                                       int32_t q_heads, int32_t kv_heads, int32_t head_dim,
                                       int32_t s_max, int32_t block_tokens,
                                       int32_t max_blocks_per_seq, int64_t num_phys_blocks,
                                       int32_t max_seq_len, float scale, void *workspace,
                                       size_t workspace_bytes, int32_t *status_flags,
                                       void *cuda_stream)
{
    const bool paged = block_table != nullptr;
    int rc = grouped_shape(batch, q_tokens, q_heads, kv_heads, head_dim, max_seq_len);
    if (rc != INSTINFER_OK) return rc;
    if (!std::isfinite(scale)) return INSTINFER_ERR_INVALID_ARG;
    if (paged) {
        if (block_tokens <= 0 || max_blocks_per_seq <= 0 || num_phys_blocks <= 0 ||
            (int64_t)max_seq_len > (int64_t)max_blocks_per_seq * block_tokens)
            return INSTINFER_ERR_INVALID_ARG;
        if (block_tokens % kGroupTile != 0) return INSTINFER_ERR_UNSUPPORTED;
    } else if (s_max <= 0 || max_seq_len > s_max) {
        return INSTINFER_ERR_INVALID_ARG;
    }
    if (batch == 0) return INSTINFER_OK;
    if (!usable(out) || !usable(q) || !usable(k_cache) || !usable(v_cache) || seq_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;

    const int64_t pairs = (int64_t)batch * kv_heads;
    const SplitPlan plan = make_plan(pairs, max_seq_len, grouped_rules(head_dim));
    GroupedParams p = {};
    p.group = q_heads / kv_heads;
    p.q_tokens = q_tokens;
    p.rows = p.group * q_tokens;
    if (workspace == nullptr || !aligned16(workspace) ||
        workspace_bytes < grouped_workspace_for(pairs, p.rows, head_dim, plan))
        return INSTINFER_ERR_WORKSPACE;
    if (pairs * plan.n_splits >= (int64_t)1 << 31) return INSTINFER_ERR_INVALID_ARG;
    p.a.q = static_cast<const __half *>(q);
    p.a.k = static_cast<const __half *>(k_cache);
    p.a.v = static_cast<const __half *>(v_cache);
    p.a.seq_lens = seq_lens;
    p.a.block_table = block_table;
    p.a.out = static_cast<__half *>(out);
    p.a.lse = lse;
    p.a.status = status_flags;
    p.a.num_phys_blocks = paged ? num_phys_blocks : 0;
    p.a.heads = kv_heads;
    p.a.pairs = (int32_t)pairs;
    p.a.s_max = paged ? 0 : s_max;
    p.a.block_tokens = paged ? block_tokens : 0;
    p.a.max_blocks_per_seq = paged ? max_blocks_per_seq : 0;
    p.a.chunk_tokens = plan.chunk_tokens;
    p.a.n_big = plan.n_big;
    p.a.tail_chunk = plan.tail_chunk;
    p.a.n_splits = plan.n_splits;
    p.a.max_seq_len = max_seq_len;
    p.a.scale_log2e = scale * 1.44269504088896340736f;
    p.a.part_o = static_cast<float *>(workspace);
    p.a.part_lse = p.a.part_o + (size_t)pairs * plan.n_splits * p.rows * head_dim;

    const unsigned grid = (unsigned)(pairs * plan.n_splits);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    switch (head_dim) {
    case 64: return paged ? launch_grouped<64, true>(p, grid, stream) : launch_grouped<64, false>(p, grid, stream);
    case 128: return paged ? launch_grouped<128, true>(p, grid, stream) : launch_grouped<128, false>(p, grid, stream);
    default: return paged ? launch_grouped<256, true>(p, grid, stream) : launch_grouped<256, false>(p, grid, stream);
    }
}

size_t instinfer_grouped_workspace_bytes(int32_t batch, int32_t q_tokens, int32_t q_heads,
                                         int32_t kv_heads, int32_t head_dim, int32_t max_seq_len)
{
    if (grouped_shape(batch, q_tokens, q_heads, kv_heads, head_dim, max_seq_len) != INSTINFER_OK) return 0;
    const int64_t pairs = (int64_t)batch * kv_heads;
    if (pairs == 0) return 256;
    return grouped_workspace_for(pairs, q_heads / kv_heads * q_tokens, head_dim,
                                 make_plan(pairs, max_seq_len, grouped_rules(head_dim)));
}

int instinfer_decode_step_host(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev,
                               float *lse, void *k_cache, void *v_cache, const int32_t *seq_lens,
                               const int32_t *block_table, int32_t max_blocks_per_seq,
                               int32_t block_tokens, int64_t num_phys_blocks, int32_t batch,
                               int32_t heads, int32_t head_dim, int32_t s_max, int32_t max_seq_len,
                               float scale, void *workspace, size_t workspace_bytes,
                               int32_t *status_flags, void *cuda_stream)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0) return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return INSTINFER_ERR_UNSUPPORTED;
    if (batch == 0) return INSTINFER_OK;
    if (out_host == nullptr || qkv_host == nullptr || !usable(qkv_dev) || !usable(out_dev))
        return INSTINFER_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t one = (size_t)batch * heads * head_dim * sizeof(__half);
    if (cudaMemcpyAsync(qkv_dev, qkv_host, 3 * one, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    const unsigned char *staged = static_cast<const unsigned char *>(qkv_dev);
    int rc = instinfer_kv_append(k_cache, v_cache, staged + one, staged + 2 * one, seq_lens, block_table,
                                 max_blocks_per_seq, block_tokens, num_phys_blocks, batch, heads,
                                 head_dim, s_max, status_flags, cuda_stream);
    if (rc != INSTINFER_OK) return rc;
    if (block_table == nullptr)
        rc = instinfer_decode_attention(out_dev, lse, staged, k_cache, v_cache, seq_lens, batch, heads,
                                        head_dim, s_max, max_seq_len, scale, workspace,
                                        workspace_bytes, status_flags, cuda_stream);
    else
        rc = instinfer_decode_attention_paged(out_dev, lse, staged, k_cache, v_cache, block_table,
                                              seq_lens, batch, heads, head_dim, block_tokens,
                                              max_blocks_per_seq, num_phys_blocks, max_seq_len,
                                              scale, workspace, workspace_bytes, status_flags,
                                              cuda_stream);
    if (rc != INSTINFER_OK) return rc;
    if (cudaMemcpyAsync(out_host, out_dev, one, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    return INSTINFER_OK;
}

namespace {

struct SparfLayout {
    size_t scores, row_ids, stats, rows_state, row_hist, row_cand, chunk_count, chunk_sums, partials, total;
    size_t zeroed_bytes;      // rows_state and row_hist are adjacent and cleared before each call
    int32_t score_stride;
    SplitPlan plan;
};

size_t round256(size_t n) { return (n + 255) / 256 * 256; }

SparfLayout sparf_layout(int64_t pairs, int32_t max_seq_len, int32_t max_k)
{
    SparfLayout w;
    w.score_stride = (max_seq_len + 7) / 8 * 8;      // whole 8-token groups, 32-byte aligned rows
    w.plan = make_plan(pairs, max_k);
    w.scores = 0;
    w.row_ids = w.scores + round256((size_t)pairs * w.score_stride * sizeof(float));
    w.stats = w.row_ids + round256((size_t)pairs * max_k * sizeof(int32_t));
    const size_t chunks = (size_t)ceil_div(max_seq_len, kScoreChunk);
    w.rows_state = w.stats + round256((size_t)pairs * sizeof(float2));
    w.row_hist = w.rows_state + round256((size_t)pairs * sizeof(SelectRow));
    w.row_cand = w.row_hist + round256((size_t)pairs * (kLinearBins + 1) * sizeof(unsigned));
    w.zeroed_bytes = w.row_cand - w.rows_state;
    w.chunk_count = w.row_cand + round256((size_t)pairs * kRowCandidates * sizeof(uint2));
    w.chunk_sums = w.chunk_count + round256((size_t)pairs * chunks * sizeof(int32_t));
    w.partials = w.chunk_sums + round256((size_t)pairs * chunks * sizeof(float2));
    w.total = w.partials + workspace_for(pairs, w.plan);
    return w;
}

bool sparf_sizes_ok(int32_t batch, int32_t heads, int32_t head_dim, int32_t block_tokens,
                    int32_t max_blocks_per_seq, int64_t num_phys_blocks)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0 || block_tokens <= 0 || max_blocks_per_seq <= 0 ||
        num_phys_blocks <= 0 || (int64_t)batch * heads > (int64_t)1 << 24)
        return false;
    return true;
}

}  // namespace

int instinfer_sparf_append(void *k_pool, void *v_pool, void *kt_pool, float *v_sum,
                           const void *k_new, const void *v_new, const int32_t *seq_lens,
                           const int32_t *block_table, int32_t max_blocks_per_seq,
                           int32_t block_tokens, int64_t num_phys_blocks,
                           const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                           int32_t kt_block_tokens, int64_t num_kt_blocks, int32_t batch,
                           int32_t heads, int32_t head_dim, int32_t *status_flags,
                           void *cuda_stream)
{
    if (!sparf_sizes_ok(batch, heads, head_dim, block_tokens, max_blocks_per_seq, num_phys_blocks) ||
        kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0)
        return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || block_tokens % 8 != 0 || kt_block_tokens % 8 != 0)
        return INSTINFER_ERR_UNSUPPORTED;
    if (batch == 0) return INSTINFER_OK;
    if (!usable(k_pool) || !usable(v_pool) || !usable(kt_pool) || !usable(v_sum) || !usable(k_new) ||
        !usable(v_new) || seq_lens == nullptr || block_table == nullptr || kt_block_table == nullptr)
        return INSTINFER_ERR_INVALID_ARG;
    SparfParams p = {};
    p.k_pool = static_cast<__half *>(k_pool);
    p.v_pool = static_cast<__half *>(v_pool);
    p.kt_pool = static_cast<__half *>(kt_pool);
    p.v_sum = v_sum;
    p.k_new = static_cast<const __half *>(k_new);
    p.v_new = static_cast<const __half *>(v_new);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.status = status_flags;
    p.num_phys_blocks = num_phys_blocks;
    p.batch = batch;
    p.heads = heads;
    p.block_tokens = block_tokens;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.kt_block_table = kt_block_table;
    p.kt_block_tokens = kt_block_tokens;
    p.kt_max_blocks_per_seq = kt_max_blocks_per_seq;
    p.num_kt_blocks = num_kt_blocks;
    sparf_append_kernel<<<(unsigned)((int64_t)batch * heads), kSparfThreads, 0,
                          static_cast<cudaStream_t>(cuda_stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? INSTINFER_OK : INSTINFER_ERR_CUDA;
}

int instinfer_sparf_append_bulk(void *k_pool, void *v_pool, void *kt_pool, float *v_sum,
                                const void *k_new, const void *v_new, const int32_t *seq_lens,
                                const int32_t *new_lens, const int32_t *block_table,
                                int32_t max_blocks_per_seq, int32_t block_tokens,
                                int64_t num_phys_blocks, const int32_t *kt_block_table,
                                int32_t kt_max_blocks_per_seq, int32_t kt_block_tokens,
                                int64_t num_kt_blocks, int32_t batch, int32_t max_new,
                                int32_t heads, int32_t head_dim, int32_t *status_flags,
                                void *cuda_stream)
{
    if (!sparf_sizes_ok(batch, heads, head_dim, block_tokens, max_blocks_per_seq, num_phys_blocks) ||
        kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0 || max_new < 0)
        return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || block_tokens % 8 != 0 || kt_block_tokens % 8 != 0)
        return INSTINFER_ERR_UNSUPPORTED;
    if (batch == 0 || max_new == 0) return INSTINFER_OK;
    if (!usable(kt_pool) || !usable(v_sum) || block_table == nullptr || kt_block_table == nullptr)
        return INSTINFER_ERR_INVALID_ARG;
    // K and V rows: the ordinary bulk append on the paged pools.
    const int rc = instinfer_kv_append_bulk(k_pool, v_pool, k_new, v_new, seq_lens, new_lens, block_table,
                                            max_blocks_per_seq, block_tokens, num_phys_blocks, batch,
                                            max_new, heads, head_dim, 0, status_flags, cuda_stream);
    if (rc != INSTINFER_OK) return rc;
    SparfBulkParams q = {};
    SparfParams &p = q.base;
    p.kt_pool = static_cast<__half *>(kt_pool);
    p.v_sum = v_sum;
    p.k_new = static_cast<const __half *>(k_new);
    p.v_new = static_cast<const __half *>(v_new);
    p.seq_lens = seq_lens;
    p.block_table = block_table;
    p.kt_block_table = kt_block_table;
    p.status = status_flags;
    p.num_phys_blocks = num_phys_blocks;
    p.num_kt_blocks = num_kt_blocks;
    p.batch = batch;
    p.heads = heads;
    p.block_tokens = block_tokens;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.kt_block_tokens = kt_block_tokens;
    p.kt_max_blocks_per_seq = kt_max_blocks_per_seq;
    q.new_lens = new_lens;
    q.max_new = max_new;
    sparf_append_bulk_kernel<<<(unsigned)((int64_t)batch * heads), kSparfThreads, 0,
                               static_cast<cudaStream_t>(cuda_stream)>>>(q);
    return cudaGetLastError() == cudaSuccess ? INSTINFER_OK : INSTINFER_ERR_CUDA;
}

size_t instinfer_sparf_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim,
                                       int32_t max_seq_len, int32_t max_k)
{
    if (head_dim != kHeadDim || !sizes_ok(batch, heads, max_seq_len) || max_k <= 0 ||
        max_k > max_seq_len)
        return 0;
    if (batch == 0) return 256;
    return sparf_layout((int64_t)batch * heads, max_seq_len, max_k).total;
}

int instinfer_sparf_decode_attention(void *out, float *alpha, int32_t *selected, const void *q,
                                     const void *k_pool, const void *v_pool, const void *kt_pool,
                                     const float *v_sum, const int32_t *block_table,
                                     const int32_t *seq_lens, const int32_t *k_tokens,
                                     int32_t batch, int32_t heads, int32_t head_dim,
                                     int32_t block_tokens, int32_t max_blocks_per_seq,
                                     int64_t num_phys_blocks,
                                     const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                                     int32_t kt_block_tokens, int64_t num_kt_blocks,
                                     int32_t max_seq_len, int32_t max_k,
                                     int32_t r, int32_t local_window, float scale,
                                     void *workspace, size_t workspace_bytes,
                                     int32_t *status_flags, void *cuda_stream)
{
    if (!sparf_sizes_ok(batch, heads, head_dim, block_tokens, max_blocks_per_seq, num_phys_blocks) ||
        kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0 ||
        max_seq_len <= 0 || (int64_t)max_seq_len > (int64_t)max_blocks_per_seq * block_tokens ||
        (int64_t)max_seq_len > (int64_t)kt_max_blocks_per_seq * kt_block_tokens ||
        max_k <= 0 || max_k > max_seq_len || local_window < 0 || !std::isfinite(scale))
        return INSTINFER_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || block_tokens % 8 != 0 || kt_block_tokens % 8 != 0)
        return INSTINFER_ERR_UNSUPPORTED;
    if (r <= 0 || r > head_dim) return INSTINFER_ERR_INVALID_ARG;
    if (num_phys_blocks * heads * block_tokens >= (int64_t)1 << 31) return INSTINFER_ERR_UNSUPPORTED;
    if (batch == 0) return INSTINFER_OK;
    if (!usable(out) || !usable(q) || !usable(k_pool) || !usable(v_pool) || !usable(kt_pool) ||
        !usable(v_sum) || block_table == nullptr || kt_block_table == nullptr || seq_lens == nullptr ||
        k_tokens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;
    const int64_t pairs = (int64_t)batch * heads;
    const SparfLayout w = sparf_layout(pairs, max_seq_len, max_k);
    if (workspace == nullptr || !aligned16(workspace) || workspace_bytes < w.total)
        return INSTINFER_ERR_WORKSPACE;
    const int64_t score_chunks = ceil_div(max_seq_len, kScoreChunk);
    if (pairs * score_chunks >= (int64_t)1 << 31 || pairs * w.plan.n_splits >= (int64_t)1 << 31)
        return INSTINFER_ERR_INVALID_ARG;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    SparfParams sp = {};
    sp.k_pool = const_cast<__half *>(static_cast<const __half *>(k_pool));
    sp.v_pool = const_cast<__half *>(static_cast<const __half *>(v_pool));
    sp.kt_pool = const_cast<__half *>(static_cast<const __half *>(kt_pool));
    sp.v_sum = const_cast<float *>(v_sum);
    sp.q = static_cast<const __half *>(q);
    sp.seq_lens = seq_lens;
    sp.k_tokens = k_tokens;
    sp.block_table = block_table;
    sp.status = status_flags;
    sp.scores = reinterpret_cast<float *>(ws + w.scores);
    sp.row_ids = reinterpret_cast<int32_t *>(ws + w.row_ids);
    sp.stats = reinterpret_cast<float2 *>(ws + w.stats);
    sp.alpha_out = alpha;
    sp.selected = selected;
    sp.num_phys_blocks = num_phys_blocks;
    sp.batch = batch;
    sp.heads = heads;
    sp.block_tokens = block_tokens;
    sp.max_blocks_per_seq = max_blocks_per_seq;
    sp.kt_block_table = kt_block_table;
    sp.kt_block_tokens = kt_block_tokens;
    sp.kt_max_blocks_per_seq = kt_max_blocks_per_seq;
    sp.num_kt_blocks = num_kt_blocks;
    sp.max_seq_len = max_seq_len;
    sp.max_k = max_k;
    sp.score_stride = w.score_stride;
    sp.score_chunks = (int32_t)score_chunks;
    sp.score_blocks = (int32_t)ceil_div(max_seq_len, kScoreBlockTokens);
    sp.r = r;
    sp.window = local_window;
    sp.scale_log2e = scale * 1.44269504088896340736f;

    sp.rows_state = reinterpret_cast<SelectRow *>(ws + w.rows_state);
    sp.row_hist = reinterpret_cast<unsigned *>(ws + w.row_hist);
    sp.row_cand = reinterpret_cast<uint2 *>(ws + w.row_cand);
    sp.chunk_count = reinterpret_cast<int32_t *>(ws + w.chunk_count);
    sp.chunk_sums = reinterpret_cast<float2 *>(ws + w.chunk_sums);

    const unsigned chunk_grid = (unsigned)(pairs * ceil_div(score_chunks, kSubChunks)), row_grid = (unsigned)pairs;
    if (cudaMemsetAsync(ws + w.rows_state, 0, w.zeroed_bytes, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    launch_overlapped(sparf_scores_kernel, (unsigned)(pairs * sp.score_blocks), kSparfThreads, 0, stream, sp);
    // Steps 5-7, chunk-parallel; rows it cannot settle are redone by the single-block kernel.
    launch_overlapped(sparf_hist_kernel, chunk_grid, kChunkThreads, 0, stream, sp);
    launch_overlapped(sparf_locate_kernel, row_grid, 32, 0, stream, sp);
    launch_overlapped(sparf_collect_kernel, chunk_grid, kChunkThreads, 0, stream, sp);
    launch_overlapped(sparf_threshold_kernel, row_grid, kThresholdThreads, 0, stream, sp);
    launch_overlapped(sparf_compact_kernel, chunk_grid, kChunkThreads, 0, stream, sp);
    launch_overlapped(sparf_finish_kernel, row_grid, 64, 0, stream, sp);
    launch_overlapped(sparf_select_kernel, row_grid, kSelectThreads, 0, stream, sp);
    if (cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;

    SparfMergeParams mp = {};
    AttnParams &ap = mp.attn;
    ap.q = sp.q;
    ap.k = sp.k_pool;
    ap.v = sp.v_pool;
    ap.seq_lens = seq_lens;
    ap.out = static_cast<__half *>(out);
    ap.status = nullptr;                 // the select kernel has already reported
    ap.heads = heads;
    ap.pairs = (int32_t)pairs;
    ap.max_seq_len = max_seq_len;
    ap.scale_log2e = sp.scale_log2e;
    ap.chunk_tokens = w.plan.chunk_tokens;
    ap.n_big = w.plan.n_big;
    ap.tail_chunk = w.plan.tail_chunk;
    ap.n_splits = w.plan.n_splits;
    ap.part_o = reinterpret_cast<float *>(ws + w.partials);
    ap.part_lse = ap.part_o + (size_t)pairs * w.plan.n_splits * kHeadDim;
    ap.row_ids = sp.row_ids;
    ap.k_tokens = k_tokens;
    ap.row_stride = max_k;
    mp.stats = sp.stats;
    mp.v_sum = v_sum;

    static bool smem_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INSTINFER_ERR_CUDA;
    if (!smem_set[dev]) {
        if (cudaFuncSetAttribute(decode_attn_split_kernel<Rows::kGathered>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kSplitSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        smem_set[dev] = true;
    }
    if (launch_overlapped(decode_attn_split_kernel<Rows::kGathered>, (unsigned)(pairs * w.plan.n_splits),
                          kThreads, kSplitSmemBytes, stream, ap) != cudaSuccess ||
        cudaGetLastError() != cudaSuccess)
        return INSTINFER_ERR_CUDA;
    const cudaError_t err = launch_overlapped(sparf_merge_kernel, (unsigned)pairs, kHeadDim, 0, stream, mp);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? INSTINFER_OK : INSTINFER_ERR_CUDA;
}

size_t instinfer_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim, int32_t max_seq_len)
{
    if (head_dim != kHeadDim || !sizes_ok(batch, heads, max_seq_len)) return 0;
    const int64_t pairs = (int64_t)batch * heads;
    if (pairs == 0) return 256;
    return workspace_for(pairs, make_plan(pairs, max_seq_len));
}

int32_t instinfer_plan_chunk_tokens(int32_t batch, int32_t heads, int32_t max_seq_len)
{
    if (!sizes_ok(batch, heads, max_seq_len) || batch == 0) return 0;
    return make_plan((int64_t)batch * heads, max_seq_len).chunk_tokens;
}

int32_t instinfer_plan_num_splits(int32_t batch, int32_t heads, int32_t max_seq_len)
{
    if (!sizes_ok(batch, heads, max_seq_len) || batch == 0) return 0;
    return make_plan((int64_t)batch * heads, max_seq_len).n_splits;
}

int instinfer_set_chunk_tokens(int32_t chunk_tokens)
{
    if (chunk_tokens < 0 || chunk_tokens % kChunkGranule != 0) return INSTINFER_ERR_INVALID_ARG;
    g_forced_chunk = chunk_tokens;
    return INSTINFER_OK;
}

int instinfer_set_timing_events(void *before_split, void *after_split)
{
    if ((before_split == nullptr) != (after_split == nullptr)) return INSTINFER_ERR_INVALID_ARG;
    g_before_split = static_cast<cudaEvent_t>(before_split);
    g_after_split = static_cast<cudaEvent_t>(after_split);
    return INSTINFER_OK;
}

const char *instinfer_status_string(int status)
{
    switch (status) {
    case INSTINFER_OK: return "ok";
    case INSTINFER_ERR_INVALID_ARG: return "invalid argument";
    case INSTINFER_ERR_UNSUPPORTED: return "unsupported head_dim or block_tokens";
    case INSTINFER_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case INSTINFER_ERR_CUDA: return "CUDA launch failed";
    default: return "unknown status";
    }
}

}  // extern "C"
