/*
 * instinfer.h -- C ABI of the decode-attention library (sm_100a).
 *
 * One decode step of one transformer layer, per (sequence, head): the newest token's k,v
 * are appended to that sequence's fp16 KV cache, then its single query row computes
 * q.K^T over every cached key, a softmax scaled by `scale`, and the weighted sum of V.
 * This is the work the paper moves into the storage drive together with the KV cache:
 * the decode-phase "Logit" and "Attend" operators (Sec. III-B) of
 * Attention(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V (Sec. II-A) with a KV cache (Sec. II-B).
 *
 * Conventions common to every entry point
 * ---------------------------------------
 * - Every pointer is a DEVICE pointer unless a comment says "host".  Data pointers must be
 *   16-byte aligned.  The library allocates nothing, never synchronises, and only enqueues
 *   work on `cuda_stream` (a cudaStream_t passed as void*; NULL = the default stream).  The
 *   caller owns every buffer, the workspace included, and must keep it alive until the
 *   enqueued work has run.
 * - fp16 = IEEE binary16.  heads = number of attention heads (query heads == KV heads,
 *   multi-head attention, Sec. II-A).  head_dim must be 128 (the paper's head size,
 *   Sec. IV-C); the two appends and instinfer_decode_attention_grouped also take 64 and 256.
 * - seq_lens[b] (int32, device, [batch]) is the length of sequence b AFTER this step's
 *   append: the append writes logical position seq_lens[b]-1, attention covers positions
 *   [0, seq_lens[b]) -- the new token attends to itself (Sec. II-B).  seq_lens[b] == 0
 *   marks an inactive slot: nothing is appended, its output rows are 0 and its lse -inf.
 * - Contiguous layout: K and V caches are [batch, heads, s_max, head_dim], row-major.
 * - Paged layout (the counterpart of the paper's token-indexed page groups, Sec. IV-C):
 *   K pool and V pool are each [num_phys_blocks, heads, block_tokens, head_dim]; logical
 *   token i of sequence b lives in physical block block_table[b][i / block_tokens] at slot
 *   i % block_tokens; block_table is int32 [batch, max_blocks_per_seq], shared by K and V.
 *   Entries past a sequence's last block are never read.  block_tokens must be a positive
 *   multiple of 8.
 * - Cache slots outside [0, seq_lens[b]) are never read and never influence a result.
 * - Return value: an instinfer_status.  Everything the host can check (null or misaligned
 *   pointers, non-positive sizes, unsupported head_dim or block_tokens, a workspace that is
 *   too small) fails before anything is enqueued.  A failed launch gives INSTINFER_ERR_CUDA.
 * - Data-dependent violations are found on the device and never fault it: a bit is OR-ed
 *   into *status_flags (int32, device, nullable; the caller zeroes it and reads it back
 *   when it wants to know).  A sequence whose length is out of range is treated as
 *   inactive (nothing appended, zero output).  A block-table entry outside
 *   [0, num_phys_blocks) is not dereferenced: the append skips that sequence, attention
 *   reads that block's rows as zeros (the sequence's output is then meaningless but finite).
 *   No kernel traps, asserts or waits on another kernel; the only waits inside a kernel are
 *   for its own asynchronous copies, and those give up after a time limit (see
 *   INSTINFER_FLAG_COPY_TIMEOUT).
 * - Stream order is kept: each kernel sees everything enqueued before it on the stream as
 *   complete.  Internally the launches use programmatic dependent launch, so a kernel's
 *   blocks may already be resident while the previous kernel drains; they touch no memory
 *   before that kernel has completed.
 * - batch == 0 is a valid empty call: INSTINFER_OK, nothing enqueued.
 */
#ifndef INSTINFER_H_
#define INSTINFER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    INSTINFER_OK = 0,
    INSTINFER_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, non-positive size, bad bound */
    INSTINFER_ERR_UNSUPPORTED = 2,   /* head_dim or block_tokens outside the supported set     */
    INSTINFER_ERR_WORKSPACE = 3,     /* workspace null or smaller than instinfer_workspace_bytes */
    INSTINFER_ERR_CUDA = 4           /* the CUDA runtime refused a launch                        */
} instinfer_status;

/* Bits OR-ed into *status_flags by the kernels. */
#define INSTINFER_FLAG_SEQ_LEN_RANGE 1  /* seq_lens[b] < 0, beyond the cache capacity, or beyond max_seq_len */
#define INSTINFER_FLAG_BLOCK_RANGE   2  /* a block_table entry that had to be read lies outside [0, num_phys_blocks) */
#define INSTINFER_FLAG_BOUNDS_CHECK  8  /* only in the bounds-checking build of the library (compiled with
                                           -DINSTINFER_BOUNDS_CHECK): a kernel computed a global offset outside the
                                           extent that the call's shapes imply and skipped that access; a defect of
                                           the library, never of the caller's data */
#define INSTINFER_FLAG_COPY_TIMEOUT  4  /* an asynchronous copy inside a kernel did not complete within about two
                                           seconds (a hardware problem, never a data problem); the kernel ended
                                           instead of waiting on and the outputs of that call are undefined */

/*
 * Append (Sec. II-B: the new token's k,v join the cache; Sec. IV-C, batch writing of the
 * decode phase's new vectors).  Copies the bit patterns of k_new[b][h][:] and v_new[b][h][:]
 * (fp16 [batch, heads, head_dim]) into logical position seq_lens[b]-1 of the caches.
 *   block_table == NULL : contiguous caches [batch, heads, s_max, head_dim];
 *                         max_blocks_per_seq, block_tokens, num_phys_blocks are ignored.
 *   block_table != NULL : paged pools; s_max is ignored.
 * k_cache / v_cache are the only buffers this call mutates, and only those rows.
 */
int instinfer_kv_append(void *k_cache, void *v_cache,
                        const void *k_new, const void *v_new,
                        const int32_t *seq_lens,
                        const int32_t *block_table, int32_t max_blocks_per_seq,
                        int32_t block_tokens, int64_t num_phys_blocks,
                        int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max,
                        int32_t *status_flags, void *cuda_stream);

/*
 * Bulk append (the prefill phase hands a layer's K,V of all prompt tokens to the cache at
 * once, Sec. IV-D).  Sequence b receives new_lens[b] tokens (0 <= new_lens[b] <= max_new,
 * new_lens[b] <= seq_lens[b]) from k_new / v_new, fp16 [batch, max_new, heads, head_dim]
 * (token-major, as a projection produces them), at logical positions
 * seq_lens[b]-new_lens[b] .. seq_lens[b]-1; seq_lens are the lengths AFTER the append.
 * Layout selection and the other arguments as in instinfer_kv_append.  A sequence whose
 * lengths are out of range is skipped and flagged.
 */
int instinfer_kv_append_bulk(void *k_cache, void *v_cache,
                             const void *k_new, const void *v_new,
                             const int32_t *seq_lens, const int32_t *new_lens,
                             const int32_t *block_table, int32_t max_blocks_per_seq,
                             int32_t block_tokens, int64_t num_phys_blocks,
                             int32_t batch, int32_t max_new, int32_t heads, int32_t head_dim,
                             int32_t s_max, int32_t *status_flags, void *cuda_stream);

/*
 * Decode attention over a contiguous cache (Sec. II-A definition, Sec. II-B/III-B decode
 * form): out[b][h][:] = softmax_i(scale * q[b][h].K[b][h][i]) . V[b][h][i], i < seq_lens[b].
 *   out          fp16 [batch, heads, head_dim]; fp32 accumulation, rounded once (nearest even)
 *   lse          fp32 [batch, heads], nullable: max_i s_i + ln sum_i exp(s_i - max), s = scale*q.k
 *   q            fp16 [batch, heads, head_dim]
 *   max_seq_len  host upper bound on every seq_lens[b], 1 <= max_seq_len <= s_max; a longer
 *                sequence is treated as inactive and flagged
 *   workspace    at least instinfer_workspace_bytes(batch, heads, head_dim, max_seq_len) bytes;
 *                holds the per-split partial outputs between the two kernels; contents are
 *                scratch before and after the call
 */
int instinfer_decode_attention(void *out, float *lse, const void *q,
                               const void *k_cache, const void *v_cache,
                               const int32_t *seq_lens,
                               int32_t batch, int32_t heads, int32_t head_dim,
                               int32_t s_max, int32_t max_seq_len, float scale,
                               void *workspace, size_t workspace_bytes,
                               int32_t *status_flags, void *cuda_stream);

/*
 * The same over block-paged pools with a block table (Sec. IV-C token-indexed groups).
 * max_seq_len <= max_blocks_per_seq * block_tokens.  The split of a sequence into partial
 * results follows logical token positions only, so the result does not depend on which
 * physical blocks hold the tokens.
 */
int instinfer_decode_attention_paged(void *out, float *lse, const void *q,
                                     const void *k_pool, const void *v_pool,
                                     const int32_t *block_table, const int32_t *seq_lens,
                                     int32_t batch, int32_t heads, int32_t head_dim,
                                     int32_t block_tokens, int32_t max_blocks_per_seq,
                                     int64_t num_phys_blocks, int32_t max_seq_len, float scale,
                                     void *workspace, size_t workspace_bytes,
                                     int32_t *status_flags, void *cuda_stream);

/*
 * Decode attention without a caller-supplied workspace (the paper has no counterpart: its
 * engine has no split partials to park).  For callers that have no device memory of their
 * own to hand over and may not ask the driver for any: a serving engine that gave its whole
 * memory budget to the KV pool at start-up, a plug-in that runs under someone else's
 * allocator, a latency-critical loop in which an allocation's implicit device
 * synchronisation is not acceptable.  The partial results live in a 16 MiB array that is
 * part of the library image, so every GPU context that loads the library carries those
 * 16 MiB until it exits.
 *   block_table == NULL : contiguous caches, arguments as instinfer_decode_attention
 *                         (block_tokens, max_blocks_per_seq, num_phys_blocks ignored);
 *   block_table != NULL : paged pools, arguments as instinfer_decode_attention_paged
 *                         (s_max ignored).
 * Results are those of the two entry points above, bit for bit.
 * Limits and rules:
 * - instinfer_workspace_bytes(batch, heads, head_dim, max_seq_len) must not exceed
 *   INSTINFER_STATIC_WORKSPACE_BYTES; otherwise INSTINFER_ERR_WORKSPACE, nothing enqueued.
 * - The first call on each device looks up the array's device address (the device must be
 *   current); make that first call outside any stream capture.  No call allocates or frees.
 * - All calls on a device share the one array, which keeps whatever the last call left in
 *   it.  Nothing in it needs to start at zero: a call only reads back the slots it has
 *   itself just written.  Two calls that can run at the same time on the GPU (different
 *   streams, no dependency between them) race on it and corrupt each other's results:
 *   order them on one stream or with events.
 */
#define INSTINFER_STATIC_WORKSPACE_BYTES ((size_t)16 << 20)
int instinfer_decode_attention_static(void *out, float *lse, const void *q,
                                      const void *k_cache, const void *v_cache,
                                      const int32_t *block_table, const int32_t *seq_lens,
                                      int32_t batch, int32_t heads, int32_t head_dim,
                                      int32_t s_max, int32_t block_tokens,
                                      int32_t max_blocks_per_seq, int64_t num_phys_blocks,
                                      int32_t max_seq_len, float scale,
                                      int32_t *status_flags, void *cuda_stream);

/*
 * Decode attention on one head shard of a multi-GPU deployment, with the all-gather of the
 * outputs fused into the last kernel (Sec. IV-D, "Scale to CSD array": heads are independent,
 * each device keeps the KV cache of its own heads and computes them locally; only the small
 * output vectors are exchanged).  This GPU holds `heads` consecutive heads, global heads
 * head_offset .. head_offset + heads - 1 of total_heads, in caches shaped as for the two
 * single-GPU entry points with H = heads (block_table == NULL: contiguous, else paged).  The
 * kernel that finishes a (sequence, head) writes its output row into EVERY rank's full
 * output buffer at [b, head_offset + h, :], with plain 16-byte stores:
 *   out_all   HOST array of n_ranks DEVICE pointers; entry r is rank r's fp16
 *             [batch, total_heads, head_dim] buffer as addressable from THIS GPU (its own
 *             allocation, or a peer mapping: CUDA IPC, symmetric memory).  The array is read
 *             during the call only.  1 <= n_ranks <= INSTINFER_MAX_RANKS.
 *   lse       nullable, this shard's own [batch, heads] (not exchanged).
 *   workspace at least instinfer_allgather_workspace_bytes(batch, heads, head_dim, max_seq_len).
 * Every other argument as in instinfer_decode_attention / instinfer_decode_attention_paged.
 * No rank waits for another inside the kernels and nothing here synchronises GPUs: when every
 * rank's call has completed, every buffer holds all heads.  Ordering a reader on rank r after
 * the other ranks' calls is the caller's job (an event exchange, or a barrier collective
 * enqueued after the call on each rank's stream).  Errors as for the single-GPU entry points;
 * head_offset < 0 or head_offset + heads > total_heads: INSTINFER_ERR_INVALID_ARG.
 */
#define INSTINFER_MAX_RANKS 16
int instinfer_decode_attention_allgather(void *const *out_all, int32_t n_ranks, float *lse,
                                         const void *q, const void *k_cache, const void *v_cache,
                                         const int32_t *block_table, const int32_t *seq_lens,
                                         int32_t batch, int32_t heads, int32_t head_offset,
                                         int32_t total_heads, int32_t head_dim, int32_t s_max,
                                         int32_t block_tokens, int32_t max_blocks_per_seq,
                                         int64_t num_phys_blocks, int32_t max_seq_len, float scale,
                                         void *workspace, size_t workspace_bytes,
                                         int32_t *status_flags, void *cuda_stream);

size_t instinfer_allgather_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim,
                                           int32_t max_seq_len);

/*
 * Decode attention for configurations other than the paper's one query head per KV head and
 * one new token per step (Sec. II-A, II-B; Sec. IV-C only notes that other configurations
 * exist): grouped heads, several new tokens per step, head sizes 64 / 128 / 256.
 *   q, out   fp16 [batch, q_tokens, q_heads, head_dim]
 *   lse      nullable fp32 [batch, q_tokens, q_heads]
 *   caches   as for the entry points above with `kv_heads` heads (block_table == NULL:
 *            contiguous [batch, kv_heads, s_max, head_dim], else paged pools
 *            [num_phys_blocks, kv_heads, block_tokens, head_dim])
 * Query head hq reads KV head hq / (q_heads / kv_heads); q_heads must be a multiple of
 * kv_heads.  The caches already hold all q_tokens new tokens (append them with
 * instinfer_kv_append, or instinfer_kv_append_bulk for q_tokens > 1) and seq_lens[b] counts
 * them; new token t (0 = oldest) attends causally to positions
 * [0, seq_lens[b] - (q_tokens - 1 - t)).  A token whose range is empty gives a zero row and
 * lse = -inf.  With q_tokens = 1 and q_heads = kv_heads the result is that of the entry points
 * above within the same tolerance (not bit for bit: the contractions run on the tensor cores).
 * Limits (INSTINFER_ERR_UNSUPPORTED otherwise): (q_heads / kv_heads) * q_tokens <= 16;
 * head_dim in {64, 128, 256}; paged block_tokens a multiple of 16.
 *   workspace at least instinfer_grouped_workspace_bytes(...) bytes.
 */
int instinfer_decode_attention_grouped(void *out, float *lse, const void *q, const void *k_cache,
                                       const void *v_cache, const int32_t *block_table,
                                       const int32_t *seq_lens, int32_t batch, int32_t q_tokens,
                                       int32_t q_heads, int32_t kv_heads, int32_t head_dim,
                                       int32_t s_max, int32_t block_tokens,
                                       int32_t max_blocks_per_seq, int64_t num_phys_blocks,
                                       int32_t max_seq_len, float scale, void *workspace,
                                       size_t workspace_bytes, int32_t *status_flags,
                                       void *cuda_stream);

size_t instinfer_grouped_workspace_bytes(int32_t batch, int32_t q_tokens, int32_t q_heads,
                                         int32_t kv_heads, int32_t head_dim, int32_t max_seq_len);

/*
 * One whole decode step for a caller whose new vectors live in host memory (the paper's
 * decode flow, Sec. IV-D: only q, k, v travel to the device that owns the KV cache and only
 * the attention output travels back; the cache never moves).
 *   qkv_host  HOST (pinned for an asynchronous copy) fp16 [3, batch, heads, head_dim]:
 *             q, k_new, v_new packed in this order
 *   out_host  HOST fp16 [batch, heads, head_dim]
 *   qkv_dev, out_dev  DEVICE staging buffers of the same shapes, owned by the caller
 *   lse       DEVICE fp32 [batch, heads], nullable
 * Enqueued on the stream, in order: copy qkv_host -> qkv_dev, instinfer_kv_append,
 * instinfer_decode_attention (block_table == NULL) or instinfer_decode_attention_paged,
 * copy out_dev -> out_host.  out_host holds the result once the stream has reached that
 * point; the call itself does not synchronise.  Other arguments and errors as in the calls
 * it is made of.
 */
int instinfer_decode_step_host(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev,
                               float *lse, void *k_cache, void *v_cache, const int32_t *seq_lens,
                               const int32_t *block_table, int32_t max_blocks_per_seq,
                               int32_t block_tokens, int64_t num_phys_blocks,
                               int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max,
                               int32_t max_seq_len, float scale,
                               void *workspace, size_t workspace_bytes,
                               int32_t *status_flags, void *cuda_stream);

/*
 * The same step with the two copies taken off the compute stream, so that a caller with
 * several independent steps in flight (the paper's mini-batches, Sec. IV-D: one mini-batch's
 * vectors travel while another's attention runs) overlaps the next step's upload and the
 * previous step's download with this step's kernels.  Streams and events are the caller's (cudaStream_t / cudaEvent_t as void*):
 *   upload_stream:    copy qkv_host -> qkv_dev, then record uploaded_event
 *   compute_stream:   wait for uploaded_event, instinfer_kv_append, attention, record attended_event
 *   download_stream:  wait for attended_event, copy out_dev -> out_host
 * A copy stream may be the compute stream itself (then its event is not used and may be
 * NULL); otherwise its event must not be NULL.  Nothing else orders the three streams: the
 * caller keeps qkv_dev, out_dev, the workspace and the events of a call untouched until that
 * call's part of each stream has run (one set per call in flight), and if the streams are
 * being captured into a graph it forks the copy streams from the capturing stream before the
 * first call and joins them after the last.  out_host holds the result once download_stream
 * has reached that point.  Arguments and errors otherwise as instinfer_decode_step_host.
 */
int instinfer_decode_step_host_overlapped(void *out_host, const void *qkv_host, void *qkv_dev, void *out_dev,
                                          float *lse, void *k_cache, void *v_cache, const int32_t *seq_lens,
                                          const int32_t *block_table, int32_t max_blocks_per_seq,
                                          int32_t block_tokens, int64_t num_phys_blocks,
                                          int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max,
                                          int32_t max_seq_len, float scale,
                                          void *workspace, size_t workspace_bytes, int32_t *status_flags,
                                          void *compute_stream, void *upload_stream, void *download_stream,
                                          void *uploaded_event, void *attended_event);

/*
 * ---- Sparse decode attention (the paper's Algorithm 1, SparF; SparQ's arithmetic) ----
 * Paged layout only.  Besides the K and V pools the cache keeps
 *   kt_pool  fp16 [num_kt_blocks, heads, head_dim, kt_block_tokens]: K a second time,
 *            embedding-major inside each block (Sec. IV-C, hidden-embedding-indexed copy).
 *            It has its own block size and its own table kt_block_table
 *            [batch, kt_max_blocks_per_seq]: token i of sequence b is column
 *            i % kt_block_tokens of block kt_block_table[b][i / kt_block_tokens].  As in the
 *            paper, where this mapping uses far larger token groups than the 16-token pages
 *            of K and V, a larger kt_block_tokens (a positive multiple of 8; 128-512 is a good
 *            choice) makes the r selected rows of a block long contiguous runs.  Slots past a
 *            sequence's end inside its last block may be read (in groups of 8 tokens) but
 *            never influence a result;
 *   v_sum    fp32 [batch, heads, head_dim]: the sum of all cached V rows of each sequence;
 *            Algorithm 1's mean value vector is v_sum / seq_lens[b].
 *
 * instinfer_sparf_append does what instinfer_kv_append does on the paged pools and also
 * writes k_new into kt_pool and adds v_new to v_sum (one fp32 rounding per element).
 * seq_lens[b] must fit both tables (max_blocks_per_seq * block_tokens and
 * kt_max_blocks_per_seq * kt_block_tokens); a longer one is flagged and that sequence is left
 * untouched, as is one whose block id in either table is out of range.
 * Unlike the plain append this call is not idempotent: v_sum grows by v_new every time, so
 * replaying a step (a retried request, a benchmark loop) adds the token's value again.
 */
int instinfer_sparf_append(void *k_pool, void *v_pool, void *kt_pool, float *v_sum,
                           const void *k_new, const void *v_new, const int32_t *seq_lens,
                           const int32_t *block_table, int32_t max_blocks_per_seq,
                           int32_t block_tokens, int64_t num_phys_blocks,
                           const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                           int32_t kt_block_tokens, int64_t num_kt_blocks,
                           int32_t batch, int32_t heads, int32_t head_dim,
                           int32_t *status_flags, void *cuda_stream);

/*
 * Bulk form of instinfer_sparf_append for the prefill phase (Sec. IV-D): new_lens[b] tokens
 * per sequence from token-major k_new / v_new [batch, max_new, heads, head_dim], as in
 * instinfer_kv_append_bulk; v_sum receives the tokens in order, one fp32 rounding each, so
 * the result equals that of appending them one by one.  A sequence with a block id out of
 * range among the blocks its new tokens need keeps its transposed copy and its v_sum, but its
 * K and V rows in valid blocks may already have been written: after a flagged call the cache
 * state of the flagged sequence is undefined and the caller should rebuild or drop it.
 */
int instinfer_sparf_append_bulk(void *k_pool, void *v_pool, void *kt_pool, float *v_sum,
                                const void *k_new, const void *v_new, const int32_t *seq_lens,
                                const int32_t *new_lens,
                                const int32_t *block_table, int32_t max_blocks_per_seq,
                                int32_t block_tokens, int64_t num_phys_blocks,
                                const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                                int32_t kt_block_tokens, int64_t num_kt_blocks,
                                int32_t batch, int32_t max_new, int32_t heads, int32_t head_dim,
                                int32_t *status_flags, void *cuda_stream);

/*
 * Algorithm 1 per (sequence, head), S = seq_lens[b]:
 *   1     I = the r dims of largest |q_d| (ties: lower d)
 *   2-4   approximate weights s^ = softmax_i(q_I . K^T[I, i] * scale / sqrt(|q_I|_1 / |q|_1)),
 *         read from kt_pool (scale = 1/sqrt(head_dim) gives the printed temperature)
 *   5-6   J = the k positions of largest s^, the last `local_window` positions always kept
 *         (ties: lower position); k = k_tokens[b] clipped to S, local_window clipped to k
 *   7     alpha = sum of s^ over J
 *   8-10  exact softmax over J of scale * q . K[j]
 *   11    out = alpha * (weights . V[J]) + (1 - alpha) * v_sum / S
 * The page-then-filter loading of steps 2-3 and 8-9 is a property of flash pages; here rows
 * are gathered directly, which gives the same values.
 *   out       fp16 [batch, heads, head_dim]
 *   alpha     fp32 [batch, heads], nullable
 *   selected  int32 [batch, heads, max_k], nullable: J in ascending order, -1 padded
 *   k_tokens  int32 [batch], device; max_k is a host upper bound (1 <= max_k <= max_seq_len);
 *             a larger k_tokens[b] is clipped to max_k
 *   r         1 <= r <= head_dim
 *   workspace at least instinfer_sparf_workspace_bytes(batch, heads, head_dim, max_seq_len, max_k)
 * Scores and the selection are computed in fp32; two scores closer than fp32 rounding may be
 * ordered differently than in exact arithmetic.  num_phys_blocks * heads * block_tokens must
 * be below 2^31.  S == 0 gives a zero row.
 */
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
                                     int32_t *status_flags, void *cuda_stream);

size_t instinfer_sparf_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim,
                                       int32_t max_seq_len, int32_t max_k);


/*
 * Workspace size (bytes, host computation only) for a call with these sizes under the
 * current split plan; 0 if an argument is invalid.
 */
size_t instinfer_workspace_bytes(int32_t batch, int32_t heads, int32_t head_dim,
                                 int32_t max_seq_len);

/*
 * Split plan.  A sequence is cut at fixed logical token positions, the same for every
 * sequence: first a few short chunks (they are scheduled last: every sequence of a ragged
 * batch has its first tokens, so every launch ends on short blocks and its tail stays short),
 * then long chunks of `chunk_tokens`.  Each chunk of each (sequence, head) is reduced by one
 * thread block and the partial results are merged by log-sum-exp in position order (no
 * counterpart in the paper, whose engine streams token groups through parallel GeMV units,
 * Sec. IV-B).  instinfer_plan_chunk_tokens returns the long chunk size the library would use
 * for these sizes and instinfer_plan_num_splits the number of chunks per sequence, short ones
 * included (0 if an argument is invalid).
 * instinfer_set_chunk_tokens(n) forces uniform chunks of n tokens for later calls of this
 * process (n > 0, a multiple of 64), n == 0 restores the automatic choice; it returns
 * INSTINFER_OK or INSTINFER_ERR_INVALID_ARG.  Not thread-safe against concurrent calls.
 */
int32_t instinfer_plan_chunk_tokens(int32_t batch, int32_t heads, int32_t max_seq_len);
int32_t instinfer_plan_num_splits(int32_t batch, int32_t heads, int32_t max_seq_len);
/*
 * Small problems (at most 8 chunks of at most 512 tokens per sequence and about two waves of
 * thread blocks in all) are bound by launch and memory latency: there the chunks of one
 * (sequence, head) run as one thread-block cluster, leave their partials in shared memory and
 * are merged inside the same kernel, so the call is one launch instead of two and the
 * workspace is not touched.  Returns 1 if the single-GPU attention entry points would do
 * that for these sizes under the current plan, else 0.
 */
int32_t instinfer_plan_merges_in_cluster(int32_t batch, int32_t heads, int32_t max_seq_len);

/*
 * ======================= Tuning, test and measurement aids =======================
 * The three calls below set process-global state that later calls of the entry points above
 * read.  They exist so that tests can drive every split plan and both forms of the sparse
 * selection, and so that a benchmark can time one kernel where it runs; a serving process
 * never needs them.  None is thread-safe against calls that run at the same time, and none
 * changes a result beyond what its comment says.
 */
int instinfer_set_chunk_tokens(int32_t chunk_tokens);

/*
 * Steps 1-7 of Algorithm 1 have two implementations: one thread block per (sequence, head)
 * that keeps the row's approximate logits in shared memory (rows of at most 16384 tokens), and
 * a chain of kernels for long rows that first brackets the k-th largest score on a sample of
 * the row and then keeps only the tokens that can still be selected (any length; rows it
 * cannot settle, e.g. thousands of equal scores, are redone by one block per row).  Both
 * compute the same fp32 scores and cut ties by position, so they select the same tokens.
 * The library picks by the sizes; instinfer_set_sparse_path forces the choice for later calls
 * of this process: 0 automatic, 1 the chain, 2 one block per row where the rows fit (a tuning
 * and test aid; returns INSTINFER_OK or INSTINFER_ERR_INVALID_ARG; not thread-safe against
 * concurrent calls).
 */
int instinfer_set_sparse_path(int32_t path);

/*
 * instinfer_decode_attention_grouped has two implementations of the same arithmetic: warp-level
 * tensor-core MMAs (every head size and block size the entry point takes) and, for head size
 * 128 or 256 with a contiguous cache or blocks of 16, 32, 64 or a multiple of 128 tokens,
 * asynchronous tcgen05 MMAs that take 128-token tiles as the long side, with accumulators in
 * tensor memory and tiles moved by tensor-map copies.  The library picks the second where the shape allows;
 * instinfer_set_grouped_path forces the choice for later calls of this process: 0 automatic,
 * 1 warp-level, 2 tcgen05 where the shape allows (a tuning and test aid; returns INSTINFER_OK
 * or INSTINFER_ERR_INVALID_ARG; not thread-safe against concurrent calls).  Both meet the
 * entry point's tolerances; their results are not bit-identical to each other.
 */
int instinfer_set_grouped_path(int32_t path);

/*
 * Which of the two implementations instinfer_decode_attention_grouped takes for a head size
 * and a cache layout (block_tokens = 0: contiguous), under the current setting of
 * instinfer_set_grouped_path: 1 warp-level, 2 tcgen05, 0 for a shape the entry point refuses.
 * (A cache of 2^31 rows or more still takes the warp-level form at call time.)  Host only.
 */
int32_t instinfer_grouped_path_for(int32_t head_dim, int32_t block_tokens);


/*
 * Measurement aid (no counterpart in the paper).  Given two cudaEvent_t (as void*, owned by
 * the caller), later attention calls of this process record `before_split` on the stream
 * just before the split-KV kernel and `after_split` just after it, so that the caller can
 * time that one kernel where it runs; (NULL, NULL) switches this off, one NULL is invalid.
 * Each call overwrites the previous recording of the same events.  Not thread-safe.
 */
int instinfer_set_timing_events(void *before_split, void *after_split);

/* Static, human-readable text for a status value (host pointer, never NULL). */
const char *instinfer_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* INSTINFER_H_ */
