/*
 * decode_attention_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of what decode-phase attention over a
 * per-sequence fp16 KV cache computes.  It exists only so that tests, the smoke check
 * and the benchmark's cpu_baseline leg have something independent to compare the CUDA
 * library with.  It shares no source, header, table or helper with that library, and
 * the library never calls it.
 *
 * Arithmetic: every fp16 input is widened exactly to fp64, every sum, exp and division
 * is fp64, and nothing is blocked, split, fused or reordered: the loops below are the
 * definition written out.
 *
 * What it follows (paper sections):
 *   - Sec. II-A  Attention(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V, heads independent (MHA).
 *   - Sec. II-B  decode with a KV cache: only the newest token's q,k,v are computed, its
 *                k,v join the cache, and its single query attends to the whole sequence
 *                (itself included) -- a GeMV per head, O(s).
 *   - Sec. III-B the "Logit" (q.K^T) and "Attend" (weights.V) operators of the decode phase.
 *   - Sec. IV-C  token-indexed storage: K (or V) of consecutive tokens of one head form a
 *                fixed-size group (16 tokens x 128 x fp16 = one 4 KB page); the decode
 *                phase appends the new token's k,v ("batch writing").  A block table plays
 *                the role of the drive's logical-to-physical map.
 *
 * Layouts (row = one token's D fp16 values of one head):
 *   contiguous: cache[b][h][i][:]           , i < s_max
 *   paged     : pool[table[b][i / T]][h][i % T][:], one table for K and V, T tokens/block
 *
 * seq_lens[b] is the sequence length AFTER this step's append: the append writes logical
 * position seq_lens[b]-1 and attention covers positions [0, seq_lens[b]).
 *
 * Return value of every function: 0 on success, otherwise a negative code and nothing is
 * guaranteed about the outputs:  -1 bad argument, -2 seq_len out of range, -3 block id out
 * of range.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE 754 binary16 -> binary64, exact (every binary16 value is a binary64 value). */
static double widen_half(uint16_t bits)
{
    const int sign = (bits >> 15) & 1;
    const int expo = (bits >> 10) & 0x1f;
    const int frac = bits & 0x3ff;
    double mag;
    if (expo == 0) {
        mag = ldexp((double)frac, -24);              /* zero and subnormals */
    } else if (expo == 31) {
        mag = frac ? NAN : INFINITY;
    } else {
        mag = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    }
    return sign ? -mag : mag;
}

/* Describes where the rows of the cache live; block_table == NULL means contiguous. */
typedef struct {
    const int32_t *block_table;
    int32_t max_blocks_per_seq;
    int32_t block_tokens;
    int64_t num_phys_blocks;
    int32_t heads;
    int32_t head_dim;
    int32_t s_max;
} cache_geometry;

/* Element offset of row (b, h, token i); -1 when the block id is out of range. */
static int64_t row_offset(const cache_geometry *g, int32_t b, int32_t h, int32_t i)
{
    const int64_t D = g->head_dim, H = g->heads;
    if (g->block_table == NULL) {
        return (((int64_t)b * H + h) * g->s_max + i) * D;
    }
    const int64_t T = g->block_tokens;
    const int32_t phys = g->block_table[(int64_t)b * g->max_blocks_per_seq + i / T];
    if (phys < 0 || (int64_t)phys >= g->num_phys_blocks) return -1;
    return (((int64_t)phys * H + h) * T + (i % T)) * D;
}

static int check_geometry(const cache_geometry *g, int32_t batch)
{
    if (batch < 0 || g->heads <= 0 || g->head_dim <= 0) return -1;
    if (g->block_table == NULL) return g->s_max > 0 ? 0 : -1;
    if (g->block_tokens <= 0 || g->max_blocks_per_seq <= 0 || g->num_phys_blocks <= 0) return -1;
    return 0;
}

static int64_t capacity_tokens(const cache_geometry *g)
{
    return g->block_table == NULL ? (int64_t)g->s_max
                                  : (int64_t)g->max_blocks_per_seq * g->block_tokens;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Append (Sec. II-B: the new token's k,v join the cache; Sec. IV-C "batch writing").
 * Copies the 16-bit patterns of k_new[b][h][:], v_new[b][h][:] to logical position
 * seq_lens[b]-1.  A sequence with seq_lens[b] == 0 is an inactive slot: nothing is
 * written for it.  Bit copy, no arithmetic: there is exactly one correct result.
 */
int oracle_kv_append(uint16_t *k_cache, uint16_t *v_cache,
                     const uint16_t *k_new, const uint16_t *v_new,
                     const int32_t *seq_lens,
                     const int32_t *block_table, int32_t max_blocks_per_seq,
                     int32_t block_tokens, int64_t num_phys_blocks,
                     int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max)
{
    const cache_geometry g = {block_table, max_blocks_per_seq, block_tokens,
                              num_phys_blocks, heads, head_dim, s_max};
    int rc = check_geometry(&g, batch);
    if (rc) return rc;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = seq_lens[b];
        if (L == 0) continue;
        if (L < 0 || (int64_t)L > capacity_tokens(&g)) return -2;
        for (int32_t h = 0; h < heads; ++h) {
            const int64_t dst = row_offset(&g, b, h, L - 1);
            if (dst < 0) return -3;
            const int64_t src = ((int64_t)b * heads + h) * head_dim;
            memcpy(k_cache + dst, k_new + src, sizeof(uint16_t) * (size_t)head_dim);
            memcpy(v_cache + dst, v_new + src, sizeof(uint16_t) * (size_t)head_dim);
        }
    }
    return 0;
}

/*
 * Bulk append (Sec. IV-D: in the prefill phase the K,V of all prompt tokens of a layer are
 * produced at once and handed to the cache layer by layer).  Sequence b receives
 * new_lens[b] tokens, taken from k_new / v_new [batch][max_new][heads][head_dim] (token-major,
 * as a projection produces them), at logical positions seq_lens[b]-new_lens[b] ..
 * seq_lens[b]-1.  Bit copy.
 */
int oracle_kv_append_bulk(uint16_t *k_cache, uint16_t *v_cache,
                          const uint16_t *k_new, const uint16_t *v_new,
                          const int32_t *seq_lens, const int32_t *new_lens,
                          const int32_t *block_table, int32_t max_blocks_per_seq,
                          int32_t block_tokens, int64_t num_phys_blocks,
                          int32_t batch, int32_t max_new, int32_t heads, int32_t head_dim,
                          int32_t s_max)
{
    const cache_geometry g = {block_table, max_blocks_per_seq, block_tokens,
                              num_phys_blocks, heads, head_dim, s_max};
    int rc = check_geometry(&g, batch);
    if (rc) return rc;
    if (max_new < 0) return -1;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = seq_lens[b], n = new_lens[b];
        if (L < 0 || (int64_t)L > capacity_tokens(&g) || n < 0 || n > max_new || n > L) return -2;
        for (int32_t t = 0; t < n; ++t) {
            for (int32_t h = 0; h < heads; ++h) {
                const int64_t dst = row_offset(&g, b, h, L - n + t);
                if (dst < 0) return -3;
                const int64_t src = ((((int64_t)b * max_new + t) * heads) + h) * head_dim;
                memcpy(k_cache + dst, k_new + src, sizeof(uint16_t) * (size_t)head_dim);
                memcpy(v_cache + dst, v_new + src, sizeof(uint16_t) * (size_t)head_dim);
            }
        }
    }
    return 0;
}

/*
 * One (sequence, head): the definition of Sec. II-A with a single query row.
 *   s_i = scale * sum_d q[d] K[i][d]          ("Logit", Sec. III-B)
 *   w_i = exp(s_i - max_j s_j) / sum_j exp(s_j - max_j s_j)
 *   out[d] = sum_i w_i V[i][d]                ("Attend", Sec. III-B)
 *   lse = max_j s_j + log sum_j exp(s_j - max_j s_j)
 * `scores` is caller scratch of length >= L.  weights (nullable) receives w_i.
 */
static int attend_one(const cache_geometry *g, int32_t b, int32_t h, int32_t L,
                      const uint16_t *q_row, const uint16_t *k_cache, const uint16_t *v_cache,
                      double scale, double *scores, double *out_row, double *lse_out,
                      double *weights)
{
    const int32_t D = g->head_dim;
    for (int32_t d = 0; d < D; ++d) out_row[d] = 0.0;
    if (L == 0) {                       /* inactive slot: no keys, zero output */
        *lse_out = -INFINITY;
        return 0;
    }
    double s_max_val = -INFINITY;
    for (int32_t i = 0; i < L; ++i) {
        const int64_t off = row_offset(g, b, h, i);
        if (off < 0) return -3;
        double dot = 0.0;
        for (int32_t d = 0; d < D; ++d) dot += widen_half(q_row[d]) * widen_half(k_cache[off + d]);
        scores[i] = scale * dot;
        if (scores[i] > s_max_val) s_max_val = scores[i];
    }
    double z = 0.0;
    for (int32_t i = 0; i < L; ++i) {
        scores[i] = exp(scores[i] - s_max_val);
        z += scores[i];
    }
    for (int32_t i = 0; i < L; ++i) {
        const int64_t off = row_offset(g, b, h, i);
        const double p = scores[i];
        for (int32_t d = 0; d < D; ++d) out_row[d] += p * widen_half(v_cache[off + d]);
    }
    for (int32_t d = 0; d < D; ++d) out_row[d] /= z;
    *lse_out = s_max_val + log(z);
    if (weights) for (int32_t i = 0; i < L; ++i) weights[i] = scores[i] / z;
    return 0;
}

/*
 * Decode attention for every (sequence, head) of a batch, contiguous or paged
 * (block_table == NULL selects contiguous).
 *   out     fp64 [batch][heads][head_dim]
 *   lse     fp64 [batch][heads]                    (nullable)
 *   weights fp64 [batch][heads][weights_stride]    (nullable; first seq_lens[b] filled)
 *   scale   the float the ABI carries, used at its exact value.
 */
int oracle_decode_attention(double *out, double *lse, double *weights, int64_t weights_stride,
                            const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                            const int32_t *seq_lens,
                            const int32_t *block_table, int32_t max_blocks_per_seq,
                            int32_t block_tokens, int64_t num_phys_blocks,
                            int32_t batch, int32_t heads, int32_t head_dim, int32_t s_max,
                            float scale)
{
    const cache_geometry g = {block_table, max_blocks_per_seq, block_tokens,
                              num_phys_blocks, heads, head_dim, s_max};
    int rc = check_geometry(&g, batch);
    if (rc) return rc;
    int32_t longest = 0;
    for (int32_t b = 0; b < batch; ++b) {
        if (seq_lens[b] < 0 || (int64_t)seq_lens[b] > capacity_tokens(&g)) return -2;
        if (weights && seq_lens[b] > weights_stride) return -1;
        if (seq_lens[b] > longest) longest = seq_lens[b];
    }
    int failure = 0;
    const int64_t pairs = (int64_t)batch * heads;
#pragma omp parallel
    {
        double scores_small[1];
        double *scores = scores_small;
        if (longest > 0) scores = (double *)malloc(sizeof(double) * (size_t)longest);
#pragma omp for schedule(dynamic, 1)
        for (int64_t pair = 0; pair < pairs; ++pair) {
            const int32_t b = (int32_t)(pair / heads), h = (int32_t)(pair % heads);
            double lse_val = 0.0;
            const int err = attend_one(&g, b, h, seq_lens[b], q + pair * head_dim,
                                       k_cache, v_cache, (double)scale, scores,
                                       out + pair * head_dim, &lse_val,
                                       weights ? weights + pair * weights_stride : NULL);
            if (lse) lse[pair] = lse_val;
            if (err) {
#pragma omp atomic write
                failure = err;
            }
        }
        if (longest > 0) free(scores);
    }
    return failure;
}

/*
 * Grouped / multi-token variant.  The paper's models use one KV head per query head and one
 * new token per step (Sec. II-A, II-B); it only notes that other configurations exist
 * (Sec. IV-C).  This is the same definition applied row by row to the two common ones:
 *   - grouped heads: query head hq reads the cache of KV head hq / group, group = q_heads /
 *     kv_heads (group == 1 is the paper's case);
 *   - several new tokens per sequence in one step: the cache already holds all q_tokens new
 *     tokens, seq_lens[b] counts them, and new token t (0 = oldest) attends causally to
 *     positions [0, seq_lens[b] - (q_tokens - 1 - t)), i.e. to itself and everything before.
 *     A token whose range is empty (sequence shorter than q_tokens) gives zero output, lse -inf.
 *   q, out  [batch][q_tokens][q_heads][head_dim]   (fp16 bits / fp64)
 *   lse     [batch][q_tokens][q_heads]             (nullable)
 *   caches  as above with kv_heads heads.
 */
int oracle_decode_attention_grouped(double *out, double *lse, const uint16_t *q,
                                    const uint16_t *k_cache, const uint16_t *v_cache,
                                    const int32_t *seq_lens,
                                    const int32_t *block_table, int32_t max_blocks_per_seq,
                                    int32_t block_tokens, int64_t num_phys_blocks,
                                    int32_t batch, int32_t q_tokens, int32_t q_heads,
                                    int32_t kv_heads, int32_t head_dim, int32_t s_max, float scale)
{
    const cache_geometry g = {block_table, max_blocks_per_seq, block_tokens,
                              num_phys_blocks, kv_heads, head_dim, s_max};
    int rc = check_geometry(&g, batch);
    if (rc) return rc;
    if (q_tokens <= 0 || q_heads <= 0 || q_heads % kv_heads != 0) return -1;
    const int32_t group = q_heads / kv_heads;
    int32_t longest = 0;
    for (int32_t b = 0; b < batch; ++b) {
        if (seq_lens[b] < 0 || (int64_t)seq_lens[b] > capacity_tokens(&g)) return -2;
        if (seq_lens[b] > longest) longest = seq_lens[b];
    }
    int failure = 0;
    const int64_t rows = (int64_t)batch * q_tokens * q_heads;
#pragma omp parallel
    {
        double scores_small[1];
        double *scores = scores_small;
        if (longest > 0) scores = (double *)malloc(sizeof(double) * (size_t)longest);
#pragma omp for schedule(dynamic, 1)
        for (int64_t row = 0; row < rows; ++row) {
            const int32_t hq = (int32_t)(row % q_heads);
            const int32_t t = (int32_t)((row / q_heads) % q_tokens);
            const int32_t b = (int32_t)(row / ((int64_t)q_heads * q_tokens));
            int32_t visible = seq_lens[b] - (q_tokens - 1 - t);
            if (visible < 0) visible = 0;
            double lse_val = 0.0;
            const int err = attend_one(&g, b, hq / group, visible, q + row * head_dim,
                                       k_cache, v_cache, (double)scale, scores,
                                       out + row * head_dim, &lse_val, NULL);
            if (lse) lse[row] = lse_val;
            if (err) {
#pragma omp atomic write
                failure = err;
            }
        }
        if (longest > 0) free(scores);
    }
    return failure;
}
