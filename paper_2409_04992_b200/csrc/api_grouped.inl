// C ABI, grouped-head / multi-token / other-head-size attention: checks, plan and launches.
// Included by instinfer_api.cu (one translation unit: the kernels' headers define
// non-template kernels, which must not be compiled twice).
#include "grouped_umma_kernels.cuh"

namespace {

int g_grouped_path = 0;     // 0 automatic, 1 warp-level MMAs, 2 tcgen05 where the shape allows (see instinfer_set_grouped_path)

// The grouped kernel's blocks are heavier (query fragments to load, 16 rows to merge at the
// end: about the cost of 20 tiles) and its warps are latency-bound, so a launch takes whole
// waves of blocks: the chunk count is chosen by that model, chunks up to 4096 tokens, and
// 1024-token chunks at the end of the longest sequences (+3 % on ragged batches, neutral on
// uniform ones; 256-token ones cost more in per-block work than they save in the tail).
PlanRules grouped_rules(int32_t head_dim)
{
    const int ctas = head_dim == 64 ? GroupedGeometry<64>::kCtasPerSm
                   : head_dim == 128 ? GroupedGeometry<128>::kCtasPerSm : GroupedGeometry<256>::kCtasPerSm;
    return PlanRules{ctas, 2, 4096, 1024, 320, false, 0};
}

// The tcgen05 form is persistent (one block per SM draws chunks from a counter), so waves do not
// matter; chunks are whole 128-token tiles, long enough (up to 4096 tokens) that the per-chunk
// epilogue is small, with 1024-token chunks drawn last to even out the end of the launch.
PlanRules umma_rules() { return PlanRules{1, 8, 4096, 1024, 0, false, 128}; }

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

// ---- the tcgen05 form (head sizes 128 and 256; contiguous, or paged in blocks of 16, 32, 64 or a multiple of 128 tokens) ----

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link libcuda).
EncodeTiledFn tensor_map_encoder()
{
    static EncodeTiledFn fn = [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &found) != cudaSuccess ||
            found != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            f = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// A K or V cache as a 2-D fp16 tensor [rows][head_dim] (a row is one token of one head);
// a box is 64 dims (128 bytes, the swizzle span) by `box_rows` tokens.
bool make_cache_map(CUtensorMap *map, const void *cache, int64_t rows, int32_t head_dim, int32_t box_rows)
{
    EncodeTiledFn encode = tensor_map_encoder();
    if (encode == nullptr || rows <= 0 || rows >= ((int64_t)1 << 31)) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(cache), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool umma_shape(int32_t head_dim, bool paged, int32_t block_tokens)
{
    // blocks of 16, 32 or 64 tokens, or of a multiple of 128 (then a forced chunk length must be one too,
    // so that no 128-token tile straddles two blocks)
    return (head_dim == 128 || head_dim == 256) &&
           (!paged || block_tokens == 16 || block_tokens == 32 || block_tokens == 64 ||
            (block_tokens % kUmmaTile == 0 && g_forced_chunk % kUmmaTile == 0));
}

// The query tensor [B, Tq, Hq, head_dim] as the copy engine sees it: a box is 64 dims of the `group`
// heads of one KV head for all Tq new tokens, i.e. the chunk's rows t * group + g in order.
bool make_query_map(CUtensorMap *map, const void *q, int32_t batch, int32_t q_tokens, int32_t q_heads, int32_t group,
                    int32_t head_dim)
{
    EncodeTiledFn encode = tensor_map_encoder();
    if (encode == nullptr) return false;
    const cuuint64_t row = (cuuint64_t)head_dim * 2;
    const cuuint64_t dims[4] = {(cuuint64_t)head_dim, (cuuint64_t)q_heads, (cuuint64_t)q_tokens, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {row, (cuuint64_t)q_heads * row, (cuuint64_t)q_tokens * q_heads * row};
    const cuuint32_t box[4] = {64, (cuuint32_t)group, (cuuint32_t)q_tokens, 1};
    const cuuint32_t elem[4] = {1, 1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void *>(q), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool kPaged, int R>
int launch_grouped_umma(const GroupedParams &p, unsigned *ticket, const CUtensorMap &map_q, const CUtensorMap &map_k,
                        const CUtensorMap &map_v, cudaStream_t stream)
{
    static bool done[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INSTINFER_ERR_CUDA;
    if (!done[dev]) {
        if (cudaFuncSetAttribute(grouped_attn_umma_kernel<D, kPaged, R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 UmmaGeometry<D>::kSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        done[dev] = true;
    }
    // One block per SM draws chunks from the ticket counter, which starts at zero.
    if (cudaMemsetAsync(ticket, 0, sizeof(unsigned), stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return INSTINFER_ERR_CUDA;
    }
    const int64_t chunks = (int64_t)p.a.pairs * p.a.n_splits;
    const unsigned grid = (unsigned)(chunks < sm_count() ? chunks : sm_count());
    cudaError_t err = launch_overlapped(grouped_attn_umma_kernel<D, kPaged, R>, grid, kUmmaThreads,
                                        UmmaGeometry<D>::kSmemBytes, stream, p, ticket, map_q, map_k, map_v);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    if (p.a.n_splits > 1) {
        err = launch_overlapped(grouped_merge_kernel<D>, (unsigned)(p.a.pairs * p.rows), D, 0, stream, p);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return INSTINFER_ERR_CUDA;
    }
    return INSTINFER_OK;
}

// The instance for the cache layout and for the number of query rows per KV head (4, 8 or 16
// rows of softmax work per token).
template <int D>
int launch_grouped_umma_rows(bool paged, const GroupedParams &p, unsigned *ticket, const CUtensorMap &map_q,
                             const CUtensorMap &map_k, const CUtensorMap &map_v, cudaStream_t stream)
{
    if (p.rows <= 4)
        return paged ? launch_grouped_umma<D, true, 4>(p, ticket, map_q, map_k, map_v, stream)
                     : launch_grouped_umma<D, false, 4>(p, ticket, map_q, map_k, map_v, stream);
    if (p.rows <= 8)
        return paged ? launch_grouped_umma<D, true, 8>(p, ticket, map_q, map_k, map_v, stream)
                     : launch_grouped_umma<D, false, 8>(p, ticket, map_q, map_k, map_v, stream);
    return paged ? launch_grouped_umma<D, true, 16>(p, ticket, map_q, map_k, map_v, stream)
                 : launch_grouped_umma<D, false, 16>(p, ticket, map_q, map_k, map_v, stream);
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
    GroupedParams p = {};
    p.group = q_heads / kv_heads;
    p.q_tokens = q_tokens;
    p.rows = p.group * q_tokens;
    const int64_t kv_bytes = (paged ? num_phys_blocks * kv_heads * block_tokens : (int64_t)batch * kv_heads * s_max) * head_dim * 2;
    // The tcgen05 form needs the caches and the query as the copy engine sees them; a cache of
    // 2^31 rows or more, or a driver without the encoder, takes the warp-level form.
    CUtensorMap map_q, map_k, map_v;
    const bool umma = g_grouped_path != 1 && umma_shape(head_dim, paged, block_tokens) &&
                      make_query_map(&map_q, q, batch, q_tokens, q_heads, p.group, head_dim) &&
                      make_cache_map(&map_k, k_cache, kv_bytes / (2 * head_dim), head_dim,
                                     paged && block_tokens < kUmmaTile ? block_tokens : kUmmaTile) &&
                      make_cache_map(&map_v, v_cache, kv_bytes / (2 * head_dim), head_dim,
                                     paged && block_tokens < kUmmaTile ? block_tokens : kUmmaTile);
    const SplitPlan plan = make_plan(pairs, max_seq_len, umma ? umma_rules() : grouped_rules(head_dim));
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
    p.a.kv_bytes = kv_bytes;
    p.a.scale_log2e = scale * 1.44269504088896340736f;
    p.a.part_o = static_cast<float *>(workspace);
    p.a.part_lse = p.a.part_o + (size_t)pairs * plan.n_splits * p.rows * head_dim;

    const unsigned grid = (unsigned)(pairs * plan.n_splits);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (umma) {
        // the ticket counter sits in the last 256 bytes of the workspace, behind the partials
        unsigned *ticket = reinterpret_cast<unsigned *>(
            static_cast<unsigned char *>(workspace) + grouped_workspace_for(pairs, p.rows, head_dim, plan) - 256);
        return head_dim == 128 ? launch_grouped_umma_rows<128>(paged, p, ticket, map_q, map_k, map_v, stream)
                               : launch_grouped_umma_rows<256>(paged, p, ticket, map_q, map_k, map_v, stream);
    }
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
    // enough for either implementation: which one runs also depends on the cache layout
    const int32_t rows = q_heads / kv_heads * q_tokens;
    size_t bytes = grouped_workspace_for(pairs, rows, head_dim, make_plan(pairs, max_seq_len, grouped_rules(head_dim)));
    if (head_dim != 64) {
        const size_t other = grouped_workspace_for(pairs, rows, head_dim, make_plan(pairs, max_seq_len, umma_rules()));
        if (other > bytes) bytes = other;
    }
    return bytes;
}

int32_t instinfer_grouped_path_for(int32_t head_dim, int32_t block_tokens)
{
    if (head_dim != 64 && head_dim != 128 && head_dim != 256) return 0;
    if (block_tokens < 0 || (block_tokens > 0 && block_tokens % kGroupTile != 0)) return 0;
    const bool paged = block_tokens > 0;
    return g_grouped_path != 1 && umma_shape(head_dim, paged, block_tokens) && tensor_map_encoder() != nullptr ? 2 : 1;
}

int instinfer_set_grouped_path(int32_t path)
{
    if (path < 0 || path > 2) return INSTINFER_ERR_INVALID_ARG;
    g_grouped_path = path;
    return INSTINFER_OK;
}

}  // extern "C"
