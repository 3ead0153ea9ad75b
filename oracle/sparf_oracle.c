/*
 * sparf_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain CPU statement of SparF attention (the paper's Algorithm 1, "flash-aware sparse
 * q-attention", which keeps SparQ attention's arithmetic, Sec. II-B and IV-A) for one decode
 * step over a block-paged fp16 KV cache, in fp64 after exact fp16 widening.  The steps are
 * taken in the algorithm's order and notation; the page/filter steps (loading whole groups,
 * then dropping the unwanted units) move data only and do not change any value, so they
 * appear here as plain indexing.  Shares no code with the CUDA library.
 *
 * Per (sequence b, head h), with S = seq_lens[b] cached tokens (the new one included):
 *   step 1      I  = the r dims of largest |q_d|               (ties: lower d first)
 *   steps 2-4   a_i = q_I . K^T[I, i] * scale / sqrt(|q_I|_1 / |q|_1),  s^ = softmax(a)
 *               (scale = 1/sqrt(d_h) gives the printed temperature sqrt(d_h |q_I|_1/|q|_1);
 *                the K^T values are read from the embedding-major copy of K)
 *   step 5      m_i = 1 for the last l positions, else 0        (the local window)
 *   step 6      J  = the k positions of largest s^_i + m_i      (ties: lower i first)
 *   step 7      alpha = sum of s^_j over J
 *   steps 8-10  s = softmax over J of scale * q . K[j, :]
 *   step 11     out = alpha * sum_j s_j V[j, :] + (1 - alpha) * vbar,  vbar = v_sum / S
 * k is clipped to S and l to k.  S == 0 gives out = 0 and alpha = 0.  If |q|_1 == 0 the
 * ratio is taken as 1.
 *
 * The two selections.  Step 1 compares fp16 magnitudes, which is exact.  Step 6 ranks the
 * fp64 values s^_i + m_i.  Every s^_i is positive and they sum to 1, so in exact arithmetic
 * s^_i + 1 exceeds every s^_j: the ranking of the sums is the ranking of the pairs
 * (m_i, s^_i), and it is taken on the pairs so that rounding 1 + s^_i to 1 cannot push a
 * window position below a dominant token.  Ties go to the lower position.
 *
 * Layouts: K, V pools [P][H][T][D] with block_table [B][M].  The K^T copy has its own
 * granularity (Sec. IV-C gives the embedding-indexed mapping much larger token groups than
 * the token-indexed one): pool [Pk][H][D][Tk] with kt_block_table [B][Mk]; token i of sequence b
 * sits in K^T block kt_block_table[b][i / Tk] at column i % Tk.  v_sum is float [B][H][D],
 * the running sum of all V rows of the sequence kept by the append.
 *
 * Return: 0, or -1 bad argument, -2 seq_len out of range, -3 block id out of range.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double widen(uint16_t bits)
{
    const int sign = (bits >> 15) & 1, expo = (bits >> 10) & 0x1f, frac = bits & 0x3ff;
    double mag;
    if (expo == 0) mag = ldexp((double)frac, -24);
    else if (expo == 31) mag = frac ? NAN : INFINITY;
    else mag = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    return sign ? -mag : mag;
}

typedef struct {
    const int32_t *table;
    int32_t max_blocks, tokens, heads, dim;
    int64_t phys_blocks;
} paged_geometry;

/* first element of physical block (b, logical block) for head h, in units of T*D elements */
static int64_t block_base(const paged_geometry *g, int32_t b, int32_t h, int32_t i)
{
    const int32_t phys = g->table[(int64_t)b * g->max_blocks + i / g->tokens];
    if (phys < 0 || (int64_t)phys >= g->phys_blocks) return -1;
    return ((int64_t)phys * g->heads + h) * g->tokens * g->dim;
}

/* element offset of K^T[dim d][token i] of (b, h) in the embedding-major pool; -1 if the block id is bad */
static int64_t kt_offset(const paged_geometry *g, int32_t b, int32_t h, int32_t d, int32_t i)
{
    const int32_t phys = g->table[(int64_t)b * g->max_blocks + i / g->tokens];
    if (phys < 0 || (int64_t)phys >= g->phys_blocks) return -1;
    return (((int64_t)phys * g->heads + h) * g->dim + d) * g->tokens + i % g->tokens;
}

/*
 * Append for the SparF state (Sec. IV-C: K is stored twice, token-indexed and hidden-
 * embedding-indexed; Algorithm 1's vbar needs the mean of V).  Position seq_lens[b]-1 gets
 * k_new, v_new in the token-major pools, k_new transposed in the embedding-major pool, and
 * v_sum += v_new with one fp32 rounding per element (the sum is carried in fp32).
 */
int oracle_sparf_append(uint16_t *k_pool, uint16_t *v_pool, uint16_t *kt_pool, float *v_sum,
                        const uint16_t *k_new, const uint16_t *v_new, const int32_t *seq_lens,
                        const int32_t *block_table, int32_t max_blocks_per_seq,
                        int32_t block_tokens, int64_t num_phys_blocks,
                        const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                        int32_t kt_block_tokens, int64_t num_kt_blocks,
                        int32_t batch, int32_t heads, int32_t head_dim)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0 || block_tokens <= 0 || max_blocks_per_seq <= 0 ||
        num_phys_blocks <= 0 || block_table == NULL || kt_block_table == NULL ||
        kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0)
        return -1;
    const paged_geometry g = {block_table, max_blocks_per_seq, block_tokens, heads, head_dim,
                              num_phys_blocks};
    const paged_geometry gt = {kt_block_table, kt_max_blocks_per_seq, kt_block_tokens, heads,
                               head_dim, num_kt_blocks};
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = seq_lens[b];
        if (L == 0) continue;
        if (L < 0 || (int64_t)L > (int64_t)max_blocks_per_seq * block_tokens ||
            (int64_t)L > (int64_t)kt_max_blocks_per_seq * kt_block_tokens)
            return -2;
        for (int32_t h = 0; h < heads; ++h) {
            const int64_t base = block_base(&g, b, h, L - 1);
            if (base < 0 || kt_offset(&gt, b, h, 0, L - 1) < 0) return -3;
            const int32_t slot = (L - 1) % block_tokens;
            const int64_t src = ((int64_t)b * heads + h) * head_dim;
            for (int32_t d = 0; d < head_dim; ++d) {
                k_pool[base + (int64_t)slot * head_dim + d] = k_new[src + d];
                v_pool[base + (int64_t)slot * head_dim + d] = v_new[src + d];
                kt_pool[kt_offset(&gt, b, h, d, L - 1)] = k_new[src + d];
                v_sum[src + d] = (float)((double)v_sum[src + d] + widen(v_new[src + d]));
            }
        }
    }
    return 0;
}

/*
 * Bulk append for the SparF state (prefill, Sec. IV-D): new_lens[b] tokens per sequence from
 * token-major k_new / v_new [batch][max_new][heads][head_dim] go to logical positions
 * seq_lens[b]-new_lens[b] .. seq_lens[b]-1 of K, V and the embedding-major copy, and each is
 * added to v_sum in token order with one fp32 rounding per addition.
 */
int oracle_sparf_append_bulk(uint16_t *k_pool, uint16_t *v_pool, uint16_t *kt_pool, float *v_sum,
                             const uint16_t *k_new, const uint16_t *v_new,
                             const int32_t *seq_lens, const int32_t *new_lens,
                             const int32_t *block_table, int32_t max_blocks_per_seq,
                             int32_t block_tokens, int64_t num_phys_blocks,
                             const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                             int32_t kt_block_tokens, int64_t num_kt_blocks,
                             int32_t batch, int32_t max_new, int32_t heads, int32_t head_dim)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0 || block_tokens <= 0 || max_blocks_per_seq <= 0 ||
        num_phys_blocks <= 0 || block_table == NULL || kt_block_table == NULL || max_new < 0 ||
        kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0)
        return -1;
    const paged_geometry g = {block_table, max_blocks_per_seq, block_tokens, heads, head_dim,
                              num_phys_blocks};
    const paged_geometry gt = {kt_block_table, kt_max_blocks_per_seq, kt_block_tokens, heads,
                               head_dim, num_kt_blocks};
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = seq_lens[b], n = new_lens[b];
        if (L < 0 || (int64_t)L > (int64_t)max_blocks_per_seq * block_tokens ||
            (int64_t)L > (int64_t)kt_max_blocks_per_seq * kt_block_tokens || n < 0 || n > max_new || n > L)
            return -2;
        for (int32_t t = 0; t < n; ++t) {
            const int32_t pos = L - n + t;
            for (int32_t h = 0; h < heads; ++h) {
                const int64_t base = block_base(&g, b, h, pos);
                if (base < 0 || kt_offset(&gt, b, h, 0, pos) < 0) return -3;
                const int64_t src = ((((int64_t)b * max_new + t) * heads) + h) * head_dim;
                const int64_t sum = ((int64_t)b * heads + h) * head_dim;
                for (int32_t d = 0; d < head_dim; ++d) {
                    k_pool[base + (int64_t)(pos % block_tokens) * head_dim + d] = k_new[src + d];
                    v_pool[base + (int64_t)(pos % block_tokens) * head_dim + d] = v_new[src + d];
                    kt_pool[kt_offset(&gt, b, h, d, pos)] = k_new[src + d];
                    v_sum[sum + d] = (float)((double)v_sum[sum + d] + widen(v_new[src + d]));
                }
            }
        }
    }
    return 0;
}

typedef struct {
    double key;
    int32_t index;
    int32_t mask;      /* m_i of step 5; 0 where unused */
} ranked;

static int by_key_desc_then_index(const void *pa, const void *pb)
{
    const ranked *a = (const ranked *)pa, *b = (const ranked *)pb;
    if (a->mask != b->mask) return a->mask > b->mask ? -1 : 1;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    return (a->index > b->index) - (a->index < b->index);
}

static int by_index(const void *pa, const void *pb)
{
    const int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/*
 *   out            fp64 [B][H][D]
 *   alpha          fp64 [B][H]                         (nullable)
 *   approx_weights fp64 [B][H][stride_s]               (nullable) s^ of step 4
 *   selected       int32 [B][H][stride_k]              (nullable) J ascending, -1 padded
 *   given          int32 [B][H][stride_k]              (nullable) if set, J is taken from
 *                  here (first min(k,S) entries) instead of step 6
 *   k_tokens       int32 [B], Algorithm 1's k per sequence
 */
int oracle_sparf_attention(double *out, double *alpha, double *approx_weights, int64_t stride_s,
                           int32_t *selected, const int32_t *given, int64_t stride_k,
                           const uint16_t *q, const uint16_t *k_pool, const uint16_t *v_pool,
                           const uint16_t *kt_pool, const float *v_sum,
                           const int32_t *seq_lens, const int32_t *k_tokens,
                           const int32_t *block_table, int32_t max_blocks_per_seq,
                           int32_t block_tokens, int64_t num_phys_blocks,
                           const int32_t *kt_block_table, int32_t kt_max_blocks_per_seq,
                           int32_t kt_block_tokens, int64_t num_kt_blocks,
                           int32_t batch, int32_t heads, int32_t head_dim,
                           int32_t r, int32_t l, float scale)
{
    if (batch < 0 || heads <= 0 || head_dim <= 0 || block_tokens <= 0 || max_blocks_per_seq <= 0 ||
        num_phys_blocks <= 0 || block_table == NULL || r <= 0 || r > head_dim || l < 0 ||
        kt_block_table == NULL || kt_block_tokens <= 0 || kt_max_blocks_per_seq <= 0 || num_kt_blocks <= 0)
        return -1;
    const paged_geometry g = {block_table, max_blocks_per_seq, block_tokens, heads, head_dim,
                              num_phys_blocks};
    const paged_geometry gt = {kt_block_table, kt_max_blocks_per_seq, kt_block_tokens, heads,
                               head_dim, num_kt_blocks};
    const int32_t D = head_dim, T = block_tokens;
    int failure = 0;
    for (int32_t b = 0; b < batch && !failure; ++b) {
        const int32_t S = seq_lens[b];
        if (S < 0 || (int64_t)S > (int64_t)max_blocks_per_seq * T ||
            (int64_t)S > (int64_t)kt_max_blocks_per_seq * kt_block_tokens)
            return -2;
        if (k_tokens[b] < 0) return -1;
        const int32_t k = k_tokens[b] < S ? k_tokens[b] : S;
        const int32_t window = l < k ? l : k;
        if ((selected || given) && k > stride_k) return -1;
        if (approx_weights && S > stride_s) return -1;
        double *a = (double *)malloc(sizeof(double) * (size_t)(S > 0 ? S : 1));
        ranked *order = (ranked *)malloc(sizeof(ranked) * (size_t)(S > 0 ? S : 1));
        int32_t *J = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
        double *s = (double *)malloc(sizeof(double) * (size_t)(k > 0 ? k : 1));
        for (int32_t h = 0; h < heads && !failure; ++h) {
            const int64_t pair = (int64_t)b * heads + h;
            double *o = out + pair * D;
            for (int32_t d = 0; d < D; ++d) o[d] = 0.0;
            if (alpha) alpha[pair] = 0.0;
            if (selected) for (int64_t t = 0; t < stride_k; ++t) selected[pair * stride_k + t] = -1;
            if (S == 0) continue;
            const uint16_t *qv = q + pair * D;

            /* step 1: the r largest |q_d| */
            ranked dims[1024];
            if (D > 1024) { failure = -1; break; }
            double q_l1 = 0.0;
            for (int32_t d = 0; d < D; ++d) {
                dims[d].key = fabs(widen(qv[d]));
                dims[d].index = d;
                dims[d].mask = 0;
                q_l1 += dims[d].key;
            }
            qsort(dims, (size_t)D, sizeof(ranked), by_key_desc_then_index);
            double qi_l1 = 0.0;
            for (int32_t t = 0; t < r; ++t) qi_l1 += dims[t].key;
            const double ratio = q_l1 > 0.0 ? qi_l1 / q_l1 : 1.0;
            const double approx_scale = (double)scale / sqrt(ratio);

            /* steps 2-4: approximate scores from the embedding-major copy of K */
            double top = -INFINITY;
            for (int32_t i = 0; i < S; ++i) {
                if (kt_offset(&gt, b, h, 0, i) < 0) { failure = -3; break; }
                double dot = 0.0;
                for (int32_t t = 0; t < r; ++t) {
                    const int32_t d = dims[t].index;
                    dot += widen(qv[d]) * widen(kt_pool[kt_offset(&gt, b, h, d, i)]);
                }
                a[i] = approx_scale * dot;
                if (a[i] > top) top = a[i];
            }
            if (failure) break;
            double z = 0.0;
            for (int32_t i = 0; i < S; ++i) { a[i] = exp(a[i] - top); z += a[i]; }
            for (int32_t i = 0; i < S; ++i) a[i] /= z;                      /* s^ */
            if (approx_weights) memcpy(approx_weights + pair * stride_s, a, sizeof(double) * (size_t)S);

            /* steps 5-6: J = the k largest of s^_i + m_i, where m_i = 1 on the last `window`
               positions and 0 elsewhere, ranked as the pairs (m_i, s^_i) (see the header) */
            if (given) {
                for (int32_t t = 0; t < k; ++t) J[t] = given[pair * stride_k + t];
            } else {
                for (int32_t i = 0; i < S; ++i) {
                    order[i].key = a[i];
                    order[i].mask = i >= S - window ? 1 : 0;
                    order[i].index = i;
                }
                qsort(order, (size_t)S, sizeof(ranked), by_key_desc_then_index);
                for (int32_t t = 0; t < k; ++t) J[t] = order[t].index;
                qsort(J, (size_t)k, sizeof(int32_t), by_index);
            }
            if (selected) for (int32_t t = 0; t < k; ++t) selected[pair * stride_k + t] = J[t];

            /* step 7 */
            double mass = 0.0;
            for (int32_t t = 0; t < k; ++t) {
                if (J[t] < 0 || J[t] >= S) { failure = -1; break; }
                mass += a[J[t]];
            }
            if (failure) break;
            if (alpha) alpha[pair] = mass;

            /* steps 8-10: exact attention over J */
            double smax = -INFINITY;
            for (int32_t t = 0; t < k; ++t) {
                const int64_t base = block_base(&g, b, h, J[t]);
                if (base < 0) { failure = -3; break; }
                double dot = 0.0;
                for (int32_t d = 0; d < D; ++d)
                    dot += widen(qv[d]) * widen(k_pool[base + (int64_t)(J[t] % T) * D + d]);
                s[t] = (double)scale * dot;
                if (s[t] > smax) smax = s[t];
            }
            if (failure) break;
            double zs = 0.0;
            for (int32_t t = 0; t < k; ++t) { s[t] = exp(s[t] - smax); zs += s[t]; }

            /* step 11 */
            for (int32_t t = 0; t < k; ++t) {
                const int64_t base = block_base(&g, b, h, J[t]);
                for (int32_t d = 0; d < D; ++d)
                    o[d] += s[t] * widen(v_pool[base + (int64_t)(J[t] % T) * D + d]);
            }
            for (int32_t d = 0; d < D; ++d) {
                const double attended = k > 0 ? o[d] / zs : 0.0;
                const double vbar = (double)v_sum[pair * D + d] / (double)S;
                o[d] = mass * attended + (1.0 - mass) * vbar;
            }
        }
        free(a); free(order); free(J); free(s);
    }
    return failure;
}
