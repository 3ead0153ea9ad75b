// C ABI, sparse attention (Algorithm 1): appends that maintain the transposed K copy and the
// running V sum, workspace layout, and the launch chain of the attention call.
// Included by instinfer_api.cu (one translation unit: the kernels' headers define
// non-template kernels, which must not be compiled twice).
#include "sparf_staged_select.cuh"

namespace {

int g_sparse_path = 0;      // 0 automatic, 1 chunk-parallel, 2 one block per row (see instinfer_set_sparse_path)

struct SparfLayout {
    size_t scores, stage_pos, row_ids, stats, rows_state, row_cand, seg_count, seg_final, blk_z, seg_mass,
        partials, total;
    size_t zeroed_bytes;      // rows_state is cleared before each call of the staged chain
    int32_t score_stride, segments, score_blocks, cand_capacity;
    SplitPlan plan;
};

size_t round256(size_t n) { return (n + 255) / 256 * 256; }

SparfLayout sparf_layout(int64_t pairs, int32_t max_seq_len, int32_t max_k)
{
    SparfLayout w;
    w.score_stride = (max_seq_len + 7) / 8 * 8;      // whole 8-token groups, 32-byte aligned rows
    w.segments = (int32_t)ceil_div(max_seq_len, kSegmentTokens);
    w.score_blocks = (int32_t)ceil_div(max_seq_len, kScoreBlockTokens);
    // candidates per row: the bracket of the sampled pre-pass holds a few per cent of the row
    int64_t cand = max_seq_len / 4;
    w.cand_capacity = (int32_t)(cand < 1024 ? 1024 : cand > kCandidates ? kCandidates : cand);
    w.plan = make_plan(pairs, max_k, kNoClusterRules);       // the row-list kernel has no cluster form
    w.scores = 0;
    w.stage_pos = w.scores + round256((size_t)pairs * w.score_stride * sizeof(float));
    w.row_ids = w.stage_pos + round256((size_t)pairs * w.score_stride * sizeof(int32_t));
    w.stats = w.row_ids + round256((size_t)pairs * max_k * sizeof(int32_t));
    w.rows_state = w.stats + round256((size_t)pairs * sizeof(float2));
    // (+ one counter behind the rows: how many rows the chain left unsolved)
    w.row_cand = w.rows_state + round256(((size_t)pairs + 1) * sizeof(SelectRow));
    w.zeroed_bytes = w.row_cand - w.rows_state;
    w.seg_count = w.row_cand + round256((size_t)pairs * w.cand_capacity * sizeof(uint2));
    w.seg_final = w.seg_count + round256((size_t)pairs * w.segments * sizeof(int32_t));
    w.blk_z = w.seg_final + round256((size_t)pairs * w.segments * sizeof(int32_t));
    w.seg_mass = w.blk_z + round256((size_t)pairs * w.score_blocks * sizeof(float));
    w.partials = w.seg_mass + round256((size_t)pairs * w.segments * sizeof(float));
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

extern "C" {

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
    if (pairs * w.score_blocks >= (int64_t)1 << 31 || pairs * w.plan.n_splits >= (int64_t)1 << 31)
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
    sp.stage_pos = reinterpret_cast<int32_t *>(ws + w.stage_pos);
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
    sp.kt_elems = num_kt_blocks * heads * kHeadDim * kt_block_tokens;
    sp.max_seq_len = max_seq_len;
    sp.max_k = max_k;
    sp.score_stride = w.score_stride;
    sp.segments = w.segments;
    sp.score_blocks = w.score_blocks;
    sp.cand_capacity = w.cand_capacity;
    sp.r = r;
    sp.window = local_window;
    sp.scale_log2e = scale * 1.44269504088896340736f;

    sp.rows_state = reinterpret_cast<SelectRow *>(ws + w.rows_state);
    sp.unsolved = reinterpret_cast<int *>(sp.rows_state + pairs);
    sp.row_cand = reinterpret_cast<uint2 *>(ws + w.row_cand);
    sp.seg_count = reinterpret_cast<int32_t *>(ws + w.seg_count);
    sp.seg_final = reinterpret_cast<int32_t *>(ws + w.seg_final);
    sp.blk_z = reinterpret_cast<float *>(ws + w.blk_z);
    sp.seg_mass = reinterpret_cast<float *>(ws + w.seg_mass);

    const unsigned block_grid = (unsigned)(pairs * w.score_blocks), row_grid = (unsigned)pairs;
    // Two ways through steps 1-7, neither of which writes the logits to HBM.  One block per row
    // computes the row's logits into shared memory and selects from there (rows of at most
    // kFusedMaxTokens tokens); the staged chain brackets the threshold on a sample and keeps
    // only the tokens that can still be selected.  Measured on one B200: the chain wins for
    // long rows with enough work to fill the GPU (2560 rows of 16k tokens: 0.86 against
    // 0.97 ms a step; 320 rows of 128k only fit the chain), the single kernel for short rows,
    // where the chain's nine launches are mostly latency (640 rows of 4k-8k tokens: 0.13
    // against 0.17 ms).
    const bool fits = max_seq_len <= kFusedMaxTokens;
    const bool long_rows = max_seq_len > 8192 && pairs * (int64_t)max_seq_len >= (int64_t)1 << 24;
    const bool fused = g_sparse_path == 1 ? false : g_sparse_path == 2 ? fits : fits && !long_rows;
    if (fused) {
        static bool fused_smem_set[kMaxDevices] = {};
        int device = 0;
        if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return INSTINFER_ERR_CUDA;
        if (!fused_smem_set[device]) {
            if (cudaFuncSetAttribute(sparf_fused_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kFusedSmemBytes) != cudaSuccess) {
                (void)cudaGetLastError();
                return INSTINFER_ERR_CUDA;
            }
            fused_smem_set[device] = true;
        }
        if (launch_overlapped(sparf_fused_select_kernel, row_grid, kFusedThreads,
                              (size_t)w.score_stride * sizeof(float), stream, sp) != cudaSuccess)
            return INSTINFER_ERR_CUDA;
    } else {
        static bool staged_smem_set[kMaxDevices] = {};
        int device = 0;
        if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return INSTINFER_ERR_CUDA;
        if (!staged_smem_set[device]) {
            if (cudaFuncSetAttribute(sparf_sample_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kMaxSamples * (int)sizeof(float)) != cudaSuccess ||
                cudaFuncSetAttribute(sparf_sample_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kMaxSamples * (int)sizeof(float)) != cudaSuccess ||
                cudaFuncSetAttribute(sparf_resolve_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kCandidates * (int)sizeof(int)) != cudaSuccess ||
                cudaFuncSetAttribute(sparf_resolve_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kCandidates * (int)sizeof(int)) != cudaSuccess) {
                (void)cudaGetLastError();
                return INSTINFER_ERR_CUDA;
            }
            staged_smem_set[device] = true;
        }
        if (cudaMemsetAsync(ws + w.rows_state, 0, w.zeroed_bytes, stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
        const size_t sample_bytes = (size_t)sample_capacity(max_seq_len) * sizeof(float);
        bool ok = max_seq_len > 32768
            ? launch_overlapped(sparf_sample_kernel<512>, row_grid, 512, sample_bytes, stream, sp) == cudaSuccess
            : launch_overlapped(sparf_sample_kernel<256>, row_grid, 256, sample_bytes, stream, sp) == cudaSuccess;
        ok = ok && launch_overlapped(sparf_stage_kernel, block_grid, kSparfThreads, 0, stream, sp) == cudaSuccess;
        const size_t where_bytes = (size_t)w.cand_capacity * sizeof(int);
        ok = ok && (w.cand_capacity > 4096
            ? launch_overlapped(sparf_resolve_kernel<512>, row_grid, 512, where_bytes, stream, sp)
            : launch_overlapped(sparf_resolve_kernel<256>, row_grid, 256, where_bytes, stream, sp)) == cudaSuccess;
        ok = ok && launch_overlapped(sparf_emit_kernel, block_grid, kEmitThreads, 0, stream, sp) == cudaSuccess;
        ok = ok && launch_overlapped(sparf_finish_kernel, row_grid, 64, 0, stream, sp) == cudaSuccess;
        // rows the chain could not settle: all their logits to the workspace, one block per row selects
        const unsigned few = (unsigned)(2 * sm_count());
        ok = ok && launch_overlapped(sparf_scores_kernel, block_grid < 4 * few ? block_grid : 4 * few, kSparfThreads, 0, stream, sp) == cudaSuccess;
        ok = ok && launch_overlapped(sparf_select_kernel, row_grid < few ? row_grid : few, kSelectThreads, 0, stream, sp) == cudaSuccess;
        if (!ok) {
            (void)cudaGetLastError();
            return INSTINFER_ERR_CUDA;
        }
    }
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
    ap.kv_bytes = num_phys_blocks * heads * block_tokens * kRowBytes;
    ap.row_limit = (int32_t)(num_phys_blocks * heads * block_tokens);      // below 2^31, checked above
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

int instinfer_set_sparse_path(int32_t path)
{
    if (path < 0 || path > 2) return INSTINFER_ERR_INVALID_ARG;
    g_sparse_path = path;
    return INSTINFER_OK;
}

}  // extern "C"
