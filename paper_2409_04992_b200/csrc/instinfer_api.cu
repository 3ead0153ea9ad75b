// C ABI of the decode-attention library, dense path: appends, one-row attention over
// contiguous and paged caches, the built-in-scratch and head-sharded variants, the host-buffer
// step, and the plan queries.  Nothing here allocates or synchronises; all work is enqueued on
// the caller's stream.
#include "api_common.cuh"

#include "allgather_merge_kernel.cuh"
#include "kv_append_kernel.cuh"

namespace {

using namespace instinfer;
using namespace instinfer::api;

// Shared-memory opt-in of the split kernels, once per device: [paged][cluster form].
int ensure_split_smem(bool paged, bool cluster)
{
    static bool done[kMaxDevices][2][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INSTINFER_ERR_CUDA;
    if (!done[dev][paged][cluster]) {
        const void *kernel = cluster
            ? (paged ? (const void *)decode_attn_split_kernel<Rows::kPaged, true>
                     : (const void *)decode_attn_split_kernel<Rows::kContiguous, true>)
            : (paged ? (const void *)decode_attn_split_kernel<Rows::kPaged, false>
                     : (const void *)decode_attn_split_kernel<Rows::kContiguous, false>);
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSplitSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        done[dev][paged][cluster] = true;
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
    // The head-sharded path ends in its own merge-and-gather kernel: it takes the same chunks
    // (so its rows equal the single-GPU ones bit for bit) but never the cluster form.
    SplitPlan plan = make_plan(pairs, p.max_seq_len);
    if (gather) plan.cluster = false;
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

    const int rc = ensure_split_smem(paged, plan.cluster);
    if (rc != INSTINFER_OK) return rc;
    const unsigned grid = (unsigned)(pairs * plan.n_splits);
    if (g_before_split) cudaEventRecord(g_before_split, stream);
    const bool timed = g_before_split != nullptr;          // event records break the overlap anyway
    cudaError_t err;
    if (plan.cluster)                  // pair-major grid, the chunks of a pair form a cluster and merge themselves
        err = paged ? launch_clustered(decode_attn_split_kernel<Rows::kPaged, true>, grid, (unsigned)plan.n_splits, kThreads, kSplitSmemBytes, stream, p)
                    : launch_clustered(decode_attn_split_kernel<Rows::kContiguous, true>, grid, (unsigned)plan.n_splits, kThreads, kSplitSmemBytes, stream, p);
    else
        err = paged ? launch_overlapped(decode_attn_split_kernel<Rows::kPaged, false>, grid, kThreads, kSplitSmemBytes, stream, p)
                    : launch_overlapped(decode_attn_split_kernel<Rows::kContiguous, false>, grid, kThreads, kSplitSmemBytes, stream, p);
    if (timed) cudaEventRecord(g_after_split, stream);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    if (gather) {
        err = launch_overlapped(lse_merge_allgather_kernel, (unsigned)pairs, kHeadDim, 0, stream, p, targets);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    } else if (plan.n_splits > 1 && !plan.cluster) {
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
    p.cache_rows = block_table ? num_phys_blocks * heads * block_tokens : (int64_t)batch * heads * s_max;
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
    const int64_t threads = (int64_t)batch * ceil_div(max_new, kBulkTokens) * heads * (head_dim / 8);
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
    p.cache_rows = block_table ? num_phys_blocks * heads * block_tokens : (int64_t)batch * heads * s_max;
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
    p.kv_bytes = (int64_t)batch * heads * s_max * kRowBytes;
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
    p.kv_bytes = num_phys_blocks * heads * block_tokens * kRowBytes;
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
    p.kv_bytes = (paged ? num_phys_blocks * heads * block_tokens : (int64_t)batch * heads * s_max) * kRowBytes;
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
// The host-vector step.  With `up` and `down` equal to the compute stream and no events this
// is one stream in order; otherwise the upload runs on `up`, the kernels on `compute` after
// `uploaded`, the download on `down` after `attended`.
static int host_step(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev, float *lse,
                     void *k_cache, void *v_cache, const int32_t *seq_lens, const int32_t *block_table,
                     int32_t max_blocks_per_seq, int32_t block_tokens, int64_t num_phys_blocks, int32_t batch,
                     int32_t heads, int32_t head_dim, int32_t s_max, int32_t max_seq_len, float scale,
                     void *workspace, size_t workspace_bytes, int32_t *status_flags, cudaStream_t compute,
                     cudaStream_t up, cudaStream_t down, cudaEvent_t uploaded, cudaEvent_t attended)
{
    // Everything the host can check is checked here, for all the calls this one is made of,
    // so that a refused call has put nothing on the stream (not even the upload).
    const bool paged = block_table != nullptr;
    if (head_dim <= 0 || !sizes_ok(batch, heads, max_seq_len) || !std::isfinite(scale))
        return INSTINFER_ERR_INVALID_ARG;
    if (paged) {
        if (block_tokens <= 0 || max_blocks_per_seq <= 0 || num_phys_blocks <= 0 ||
            (int64_t)max_seq_len > (int64_t)max_blocks_per_seq * block_tokens)
            return INSTINFER_ERR_INVALID_ARG;
    } else if (s_max <= 0 || max_seq_len > s_max) {
        return INSTINFER_ERR_INVALID_ARG;
    }
    if (head_dim != kHeadDim || (paged && block_tokens % 8 != 0)) return INSTINFER_ERR_UNSUPPORTED;
    if ((up != compute && uploaded == nullptr) || (down != compute && attended == nullptr))
        return INSTINFER_ERR_INVALID_ARG;
    if (batch == 0) return INSTINFER_OK;
    if (out_host == nullptr || qkv_host == nullptr || !usable(qkv_dev) || !usable(out_dev) ||
        !usable(k_cache) || !usable(v_cache) || seq_lens == nullptr)
        return INSTINFER_ERR_INVALID_ARG;
    {
        const int64_t pairs = (int64_t)batch * heads;
        if (workspace == nullptr || !aligned16(workspace) ||
            workspace_bytes < workspace_for(pairs, make_plan(pairs, max_seq_len)))
            return INSTINFER_ERR_WORKSPACE;
    }
    const size_t one = (size_t)batch * heads * head_dim * sizeof(__half);
    bool fine = cudaMemcpyAsync(qkv_dev, qkv_host, 3 * one, cudaMemcpyHostToDevice, up) == cudaSuccess;
    if (fine && up != compute)
        fine = cudaEventRecord(uploaded, up) == cudaSuccess && cudaStreamWaitEvent(compute, uploaded, 0) == cudaSuccess;
    if (!fine) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    const unsigned char *staged = static_cast<const unsigned char *>(qkv_dev);
    int rc = instinfer_kv_append(k_cache, v_cache, staged + one, staged + 2 * one, seq_lens, block_table,
                                 max_blocks_per_seq, block_tokens, num_phys_blocks, batch, heads,
                                 head_dim, s_max, status_flags, compute);
    if (rc != INSTINFER_OK) return rc;
    if (block_table == nullptr)
        rc = instinfer_decode_attention(out_dev, lse, staged, k_cache, v_cache, seq_lens, batch, heads,
                                        head_dim, s_max, max_seq_len, scale, workspace,
                                        workspace_bytes, status_flags, compute);
    else
        rc = instinfer_decode_attention_paged(out_dev, lse, staged, k_cache, v_cache, block_table,
                                              seq_lens, batch, heads, head_dim, block_tokens,
                                              max_blocks_per_seq, num_phys_blocks, max_seq_len,
                                              scale, workspace, workspace_bytes, status_flags,
                                              compute);
    if (rc != INSTINFER_OK) return rc;
    if (down != compute)
        fine = cudaEventRecord(attended, compute) == cudaSuccess && cudaStreamWaitEvent(down, attended, 0) == cudaSuccess;
    fine = fine && cudaMemcpyAsync(out_host, out_dev, one, cudaMemcpyDeviceToHost, down) == cudaSuccess;
    if (!fine) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    return INSTINFER_OK;
}

int instinfer_decode_step_host(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev,
                               float *lse, void *k_cache, void *v_cache, const int32_t *seq_lens,
                               const int32_t *block_table, int32_t max_blocks_per_seq,
                               int32_t block_tokens, int64_t num_phys_blocks, int32_t batch,
                               int32_t heads, int32_t head_dim, int32_t s_max, int32_t max_seq_len,
                               float scale, void *workspace, size_t workspace_bytes,
                               int32_t *status_flags, void *cuda_stream)
{
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    return host_step(out_host, qkv_host, qkv_dev, out_dev, lse, k_cache, v_cache, seq_lens, block_table,
                     max_blocks_per_seq, block_tokens, num_phys_blocks, batch, heads, head_dim, s_max,
                     max_seq_len, scale, workspace, workspace_bytes, status_flags, stream, stream, stream,
                     nullptr, nullptr);
}

int instinfer_decode_step_host_overlapped(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev,
                                          float *lse, void *k_cache, void *v_cache, const int32_t *seq_lens,
                                          const int32_t *block_table, int32_t max_blocks_per_seq,
                                          int32_t block_tokens, int64_t num_phys_blocks, int32_t batch,
                                          int32_t heads, int32_t head_dim, int32_t s_max, int32_t max_seq_len,
                                          float scale, void *workspace, size_t workspace_bytes,
                                          int32_t *status_flags, void *compute_stream, void *upload_stream,
                                          void *download_stream, void *uploaded_event, void *attended_event)
{
    return host_step(out_host, qkv_host, qkv_dev, out_dev, lse, k_cache, v_cache, seq_lens, block_table,
                     max_blocks_per_seq, block_tokens, num_phys_blocks, batch, heads, head_dim, s_max,
                     max_seq_len, scale, workspace, workspace_bytes, status_flags,
                     static_cast<cudaStream_t>(compute_stream), static_cast<cudaStream_t>(upload_stream),
                     static_cast<cudaStream_t>(download_stream), static_cast<cudaEvent_t>(uploaded_event),
                     static_cast<cudaEvent_t>(attended_event));
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

int32_t instinfer_plan_merges_in_cluster(int32_t batch, int32_t heads, int32_t max_seq_len)
{
    if (!sizes_ok(batch, heads, max_seq_len) || batch == 0) return 0;
    return make_plan((int64_t)batch * heads, max_seq_len).cluster ? 1 : 0;
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

#include "api_grouped.inl"
#include "api_sparf.inl"
