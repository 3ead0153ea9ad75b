// C ABI, grouped-head / multi-token / other-head-size attention: checks, plan and launches.
// Included by instinfer_api.cu (one translation unit: the kernels' headers define
// non-template kernels, which must not be compiled twice).
#include "grouped_attention_kernels.cuh"

namespace {

// The grouped kernel's blocks are heavier (query fragments to load, 16 rows to merge at the
// end: about the cost of 20 tiles) and its warps are latency-bound, so a launch takes whole
// waves of blocks: the chunk count is chosen by that model, chunks up to 4096 tokens, and
// 1024-token chunks at the end of the longest sequences (+3 % on ragged batches, neutral on
// uniform ones; 256-token ones cost more in per-block work than they save in the tail).
PlanRules grouped_rules(int32_t head_dim)
{
    const int ctas = head_dim == 64 ? GroupedGeometry<64>::kCtasPerSm
                   : head_dim == 128 ? GroupedGeometry<128>::kCtasPerSm : GroupedGeometry<256>::kCtasPerSm;
    return PlanRules{ctas, 2, 4096, 1024, 320, false};
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

extern "C" {

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
    p.a.kv_bytes = (paged ? num_phys_blocks * kv_heads * block_tokens : (int64_t)batch * kv_heads * s_max) * head_dim * 2;
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

}  // extern "C"
