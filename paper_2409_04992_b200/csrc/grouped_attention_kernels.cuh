// Split-KV decode attention for several query rows per KV head, for sm_100a.
//
// The paper's models give every query head its own KV head and decode one token per step
// (Sec. II-A, II-B); it notes that other configurations exist (Sec. IV-C).  Two of them put
// R > 1 query rows against the same cached K and V: grouped heads (`group` query heads share
// a KV head) and several new tokens per step (each attends causally).  Reading every K and V
// byte once then costs R times the arithmetic of the one-row kernel, which the FMA pipes
// cannot keep up with beyond R = 2, so here the two contractions run on the tensor cores:
//   S[16 x 16]  = Q[16 x D] K_tile^T      (rows beyond R are zero padding)
//   O[16 x D]  += P[16 x 16] V_tile
// as warp-level m16n8k16 fp16 MMAs with fp32 accumulators.  With at most 16 query rows the
// 64-row minimum of the asynchronous tcgen05 MMA would be three quarters padding and would
// route the softmax through tensor memory; the work is HBM-bound either way (the MMAs take
// well under a fifth of the issue slots), so the synchronous warp-level form is the right size.
//
// Structure as in the one-row kernel: a block owns one chunk of token positions of one
// (sequence, KV head); each warp streams its own 16-token tiles of K and V through a private
// ring of padded shared-memory rows filled by 16-byte cp.async copies, with no block barrier
// in the main loop; fragments come out of shared memory with ldmatrix (transposed for V);
// the online softmax keeps a per-row reference that follows the maximum lazily; softmax
// weights enter the second MMA as an fp16 hi + lo pair so that the result keeps fp32-level
// accuracy; the four warp states are merged at the end of the chunk.
#pragma once

#include "decode_attention_kernels.cuh"

namespace instinfer {

constexpr int kGroupRows = 16;         // query rows one MMA tile holds
constexpr int kGroupTile = 16;         // tokens per warp tile
constexpr int kGroupStages = 3;

struct GroupedParams {
    // a.heads = KV heads, a.pairs = batch * KV heads; a.q and a.out are
    // [batch, q_tokens, KV heads * group, D], a.lse [batch, q_tokens, KV heads * group];
    // a.part_o [pairs, n_splits, rows, D], a.part_lse [pairs, n_splits, rows].
    AttnParams a;
    int32_t group;         // query heads per KV head
    int32_t q_tokens;      // new tokens per sequence; token t sees positions < len - (q_tokens-1-t)
    int32_t rows;          // group * q_tokens <= kGroupRows; row r = t * group + g
};

template <int D>
struct GroupedGeometry {
    static constexpr int kRowBytes = D * 2;
    static constexpr int kRowStride = kRowBytes + 16;            // 8 rows x 16 B hit 32 distinct banks
    static constexpr int kTileBytes = kGroupTile * kRowStride;   // one tile of K (or of V)
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kRingBytes = kWarps * kGroupStages * kStageBytes;
    static constexpr bool kQInSmem = D > 128;                    // large heads: Q fragments re-read
    static constexpr int kQBytes = kQInSmem ? kGroupRows * kRowStride : 0;
    static constexpr int kSmemBytes = kRingBytes + kQBytes;
    static constexpr int kCtasPerSm = D <= 64 ? 4 : D <= 128 ? 2 : 1;
    static constexpr int kKSteps = D / 16;                       // MMA k-steps of Q K^T
    static constexpr int kSegsPerLane = D / 16;                  // 16-byte copies per lane per tile of K
};

__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], unsigned addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], unsigned addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// c += a (16x16, row-major fragments) * b (16x8, column fragments); fp16 inputs, fp32 accumulate
__device__ __forceinline__ void mma_16816(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, "
                 "{%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_half2(float x, float y)
{
    const __half2 h = __floats2half2_rn(x, y);
    return *reinterpret_cast<const unsigned *>(&h);
}

// Element offset of query (and output) row r of (sequence b, KV head hk).
__device__ __forceinline__ int64_t grouped_row_index(const GroupedParams &p, int b, int hk, int r)
{
    const int t = r / p.group, g = r - t * p.group;
    return ((int64_t)b * p.q_tokens + t) * ((int64_t)p.a.heads * p.group) + (int64_t)hk * p.group + g;
}

template <int D, bool kPaged>
__global__ void __launch_bounds__(kThreads, GroupedGeometry<D>::kCtasPerSm)
grouped_attn_split_kernel(const GroupedParams p)
{
    using G = GroupedGeometry<D>;
    extern __shared__ __align__(128) unsigned char smem[];
    const AttnParams &a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, quad = lane & 3;          // MMA fragment coordinates
    const int split = blockIdx.x / a.pairs;
    const int pair = blockIdx.x - split * a.pairs;
    const int b = pair / a.heads, hk = pair - b * a.heads;
    const bool final_writer = a.n_splits == 1;
    allow_next_kernel();
    wait_for_previous_kernels();

    const int len = checked_seq_len(a, b, threadIdx.x == 0 && hk == 0 && final_writer);
    int begin, chunk_size;
    chunk_range(a, split, begin, chunk_size);
    if (begin >= len) {
        if (final_writer) {                    // inactive slot: zero output, lse = -inf
            for (int i = threadIdx.x; i < p.rows * D; i += kThreads) {
                const int r = i / D, d = i - r * D;
                const int64_t row = grouped_row_index(p, b, hk, r);
                a.out[row * D + d] = __float2half_rn(0.f);
                if (a.lse && d == 0) a.lse[row] = -INFINITY;
            }
        }
        return;
    }
    const int end = min(begin + chunk_size, len);
    const int n_tiles = (end - begin + kGroupTile - 1) / kGroupTile;
    const int my_tiles = warp < n_tiles ? (n_tiles - warp + kWarps - 1) / kWarps : 0;

    // Rows gid and gid + 8 of the MMA tile belong to this lane: their query rows and how many
    // cached positions each may see (rows beyond p.rows are padding and see nothing).
    const bool has_lo = gid < p.rows, has_hi = gid + 8 < p.rows;
    const int vis_lo = has_lo ? len - (p.q_tokens - 1 - gid / p.group) : 0;
    const int vis_hi = has_hi ? len - (p.q_tokens - 1 - (gid + 8) / p.group) : 0;
    const unsigned smem_base = static_cast<unsigned>(__cvta_generic_to_shared(smem));

    // Query fragments (A operand of Q K^T), straight from global memory in fragment order.
    unsigned qa[G::kQInSmem ? 1 : G::kKSteps][4];
    const unsigned q_rd = smem_base + G::kRingBytes + ((lane & 7) + ((lane >> 3) & 1) * 8) * G::kRowStride +
                          (lane >> 4) * 16;
    if (G::kQInSmem) {
        // 16 padded rows in shared memory, zero beyond p.rows; fragments are re-read per tile
        unsigned char *q_sm = smem + G::kRingBytes;
        for (int i = threadIdx.x; i < kGroupRows * (D / 8); i += kThreads) {
            const int r = i / (D / 8), seg = i - r * (D / 8);
            uint4 v = make_uint4(0, 0, 0, 0);
            if (r < p.rows)
                v = reinterpret_cast<const uint4 *>(a.q + grouped_row_index(p, b, hk, r) * D)[seg];
            *reinterpret_cast<uint4 *>(q_sm + r * G::kRowStride + seg * 16) = v;
        }
        __syncthreads();
    } else {
        const __half *q_lo = a.q + (has_lo ? grouped_row_index(p, b, hk, gid) : 0) * D;
        const __half *q_hi = a.q + (has_hi ? grouped_row_index(p, b, hk, gid + 8) : 0) * D;
#pragma unroll
        for (int ks = 0; ks < G::kKSteps; ++ks) {
            const int c = ks * 16 + quad * 2;
            qa[ks][0] = has_lo ? *reinterpret_cast<const unsigned *>(q_lo + c) : 0u;
            qa[ks][1] = has_hi ? *reinterpret_cast<const unsigned *>(q_hi + c) : 0u;
            qa[ks][2] = has_lo ? *reinterpret_cast<const unsigned *>(q_lo + c + 8) : 0u;
            qa[ks][3] = has_hi ? *reinterpret_cast<const unsigned *>(q_hi + c + 8) : 0u;
        }
    }

    // ---- copy-issue side ----
    // A tile's 16 rows are contiguous in memory in both layouts (a paged block holds a
    // multiple of 16 tokens and chunks start on multiples of 64), so 16-byte segment s of the
    // tile sits at tile base + 16 s; in shared memory its row is padded.
    const unsigned ring = smem_base + warp * (kGroupStages * G::kStageBytes);
    constexpr int kTileRowSegs = D / 8;
    const unsigned char *k_bytes = reinterpret_cast<const unsigned char *>(a.k);
    const unsigned char *v_bytes = reinterpret_cast<const unsigned char *>(a.v);
    const int32_t *table_row = kPaged ? a.block_table + (int64_t)b * a.max_blocks_per_seq : nullptr;
    auto tile_token = [&](int j) { return begin + (warp + j * kWarps) * kGroupTile; };
    auto table_entry = [&](int j) -> int {
        return kPaged && j < my_tiles ? __ldg(table_row + tile_token(j) / a.block_tokens) : 0;
    };
    int next_phys = table_entry(0);            // looked up one tile ahead of its use

    int issue_j = 0;
    unsigned issue_stage = 0;
    auto issue = [&]() {
        if (issue_j < my_tiles) {
            const int tok0 = tile_token(issue_j);
            const int rows_here = min(kGroupTile, end - tok0);
            bool usable = true;
            int64_t off;
            if (kPaged) {
                const int phys = next_phys;
                next_phys = table_entry(issue_j + 1);
                usable = phys >= 0 && (int64_t)phys < a.num_phys_blocks;
                if (!usable && lane == 0 && a.status) atomicOr(a.status, kFlagBlockRange);
                const int slot = tok0 % a.block_tokens;
                off = usable ? (((int64_t)phys * a.heads + hk) * a.block_tokens + slot) * G::kRowBytes : 0;
            } else {
                off = ((int64_t)pair * a.s_max + tok0) * G::kRowBytes;
            }
            const unsigned dst = ring + issue_stage * G::kStageBytes;
#pragma unroll
            for (int i = 0; i < G::kSegsPerLane; ++i) {
                const int s = i * 32 + lane;
                const int row = s / kTileRowSegs, col = s - row * kTileRowSegs;
                const bool valid = usable && row < rows_here;
                const int64_t src = valid ? off + (int64_t)s * 16 : 0;
                const unsigned d = dst + row * G::kRowStride + col * 16;
                cp_async_16(d, k_bytes + src, valid ? 16 : 0);       // masked rows are zero-filled
                cp_async_16(d + G::kTileBytes, v_bytes + src, valid ? 16 : 0);
            }
        }
        cp_async_commit();                     // empty groups keep the count uniform
        ++issue_j;
        issue_stage = issue_stage + 1 == kGroupStages ? 0 : issue_stage + 1;
    };

    // ldmatrix lane addresses inside a stage.  K (operand B of Q K^T, "column" fragments):
    // matrices (tokens 0-7, dims +0..7), (tokens 0-7, dims +8..15), (tokens 8-15, dims +0..7),
    // (tokens 8-15, dims +8..15) per k-step.  V (operand B of P V, transposed on load):
    // matrices (tokens 0-7, dims +0..7), (tokens 8-15, dims +0..7), (tokens 0-7, dims +8..15),
    // (tokens 8-15, dims +8..15) per pair of 8-dim output blocks.
    const int mat = lane >> 3, mrow = lane & 7;
    const unsigned k_rd = (mrow + (mat >> 1) * 8) * G::kRowStride + (mat & 1) * 16;
    const unsigned v_rd = G::kTileBytes + (mrow + (mat & 1) * 8) * G::kRowStride + (mat >> 1) * 16;

    // Running state of rows gid (lo) and gid + 8 (hi): reference m (base-2 logits), this
    // lane's share of the sum l, and the output fragments, which carry kWeightScale.
    float m_lo = kMinusHuge, m_hi = kMinusHuge, l_lo = 0.f, l_hi = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

#pragma unroll
    for (int j = 0; j < kGroupStages - 1; ++j) issue();

    unsigned stage = 0;
    for (int j = 0; j < my_tiles; ++j) {
        cp_async_wait<kGroupStages - 2>();
        __syncwarp();                    // tile j visible to the warp; everyone is done with tile j-1
        issue();                         // refills the slot tile j-1 used
        const unsigned base = ring + stage * G::kStageBytes;
        stage = stage + 1 == kGroupStages ? 0 : stage + 1;
        const int tok0 = tile_token(j);

        // Logits of 16 rows x 16 tokens: s[n][0..1] row gid, s[n][2..3] row gid + 8, tokens
        // tok0 + 8 n + 2 quad + {0, 1}.
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int ks = 0; ks < G::kKSteps; ++ks) {
            unsigned kb[4];
            ldmatrix_x4(kb, base + k_rd + ks * 32);
            if (G::kQInSmem) {
                unsigned qf[4];
                ldmatrix_x4(qf, q_rd + ks * 32);
                mma_16816(s[0], qf, kb[0], kb[1]);
                mma_16816(s[1], qf, kb[2], kb[3]);
            } else {
                mma_16816(s[0], qa[ks], kb[0], kb[1]);
                mma_16816(s[1], qa[ks], kb[2], kb[3]);
            }
        }
        bool grows = false;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = tok0 + n * 8 + quad * 2 + e;
                s[n][e] = tok < vis_lo ? s[n][e] * a.scale_log2e : -INFINITY;
                s[n][2 + e] = tok < vis_hi ? s[n][2 + e] * a.scale_log2e : -INFINITY;
                grows |= s[n][e] > m_lo + kMaxLag || s[n][2 + e] > m_hi + kMaxLag;
            }
        }
        // Online softmax with per-row references that may lag the true maximum by up to
        // kMaxLag (base-2 units): weights reach at most 2^kMaxLag, inside the range of the
        // fp16 weight split.  References move, and accumulators are rescaled, only when some
        // logit exceeds its row's reference by more than that.
        if (__any_sync(0xffffffffu, grows)) {
            float top_lo = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
            float top_hi = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
            top_lo = fmaxf(top_lo, __shfl_xor_sync(0xffffffffu, top_lo, 1));
            top_lo = fmaxf(top_lo, __shfl_xor_sync(0xffffffffu, top_lo, 2));
            top_hi = fmaxf(top_hi, __shfl_xor_sync(0xffffffffu, top_hi, 1));
            top_hi = fmaxf(top_hi, __shfl_xor_sync(0xffffffffu, top_hi, 2));
            float alpha_lo = 1.f, alpha_hi = 1.f;
            if (top_lo > m_lo + kMaxLag) {
                alpha_lo = fast_exp2(m_lo - top_lo);
                m_lo = top_lo;
            }
            if (top_hi > m_hi + kMaxLag) {
                alpha_hi = fast_exp2(m_hi - top_hi);
                m_hi = top_hi;
            }
            l_lo *= alpha_lo;
            l_hi *= alpha_hi;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                o[i][0] *= alpha_lo;
                o[i][1] *= alpha_lo;
                o[i][2] *= alpha_hi;
                o[i][3] *= alpha_hi;
            }
        }
        // Weights, their sums, and the A fragments of P V as fp16 hi + lo of weight * 2^14.
        unsigned p_hi[4], p_lo[4];
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            float w[4], big[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = fast_exp2(s[n][e] - (e < 2 ? m_lo : m_hi)) * kWeightScale;
            l_lo += w[0] + w[1];
            l_hi += w[2] + w[3];
            p_hi[2 * n] = pack_half2(w[0], w[1]);
            p_hi[2 * n + 1] = pack_half2(w[2], w[3]);
            const float2 f_lo = __half22float2(*reinterpret_cast<const __half2 *>(&p_hi[2 * n]));
            const float2 f_hi = __half22float2(*reinterpret_cast<const __half2 *>(&p_hi[2 * n + 1]));
            big[0] = f_lo.x, big[1] = f_lo.y, big[2] = f_hi.x, big[3] = f_hi.y;
            p_lo[2 * n] = pack_half2(w[0] - big[0], w[1] - big[1]);
            p_lo[2 * n + 1] = pack_half2(w[2] - big[2], w[3] - big[3]);
        }
        // O += P V: two 8-dim output blocks per ldmatrix.
#pragma unroll
        for (int nb = 0; nb < D / 16; ++nb) {
            unsigned vb[4];
            ldmatrix_x4_trans(vb, base + v_rd + nb * 32);
            mma_16816(o[2 * nb], p_hi, vb[0], vb[1]);
            mma_16816(o[2 * nb + 1], p_hi, vb[2], vb[3]);
            mma_16816(o[2 * nb], p_lo, vb[0], vb[1]);
            mma_16816(o[2 * nb + 1], p_lo, vb[2], vb[3]);
        }
    }
    cp_async_wait<0>();

    // Row sums over the four lanes that share a row (both l and o carry kWeightScale).
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    __syncthreads();                     // every ring is idle: reuse shared memory for the merge

    float *sm_m = reinterpret_cast<float *>(smem);             // [kWarps][kGroupRows]
    float *sm_l = sm_m + kWarps * kGroupRows;
    float *sm_o = sm_l + kWarps * kGroupRows;                  // [kWarps][kGroupRows][D]
    if (quad == 0) {
        sm_m[warp * kGroupRows + gid] = m_lo;
        sm_m[warp * kGroupRows + gid + 8] = m_hi;
        sm_l[warp * kGroupRows + gid] = l_lo;
        sm_l[warp * kGroupRows + gid + 8] = l_hi;
    }
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
        float *dst = sm_o + ((warp * kGroupRows + gid) * D + i * 8 + quad * 2);
        *reinterpret_cast<float2 *>(dst) = make_float2(o[i][0], o[i][1]);
        *reinterpret_cast<float2 *>(dst + 8 * D) = make_float2(o[i][2], o[i][3]);
    }
    __syncthreads();

    for (int i = threadIdx.x; i < p.rows * D; i += kThreads) {
        const int r = i / D, d = i - r * D;
        float top = kMinusHuge;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) top = fmaxf(top, sm_m[w * kGroupRows + r]);
        float total = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float weight = fast_exp2(sm_m[w * kGroupRows + r] - top);
            total = fmaf(weight, sm_l[w * kGroupRows + r], total);
            acc = fmaf(weight, sm_o[(w * kGroupRows + r) * D + d], acc);
        }
        // A row that sees no position of this chunk (causal limit before the chunk) has total 0.
        const bool empty = !(total > 0.f);
        const float value = empty ? 0.f : acc / total;
        const float lse2 = empty ? kMinusHuge : top + log2f(total / kWeightScale);
        if (final_writer) {
            const int64_t row = grouped_row_index(p, b, hk, r);
            a.out[row * D + d] = __float2half_rn(value);
            if (a.lse && d == 0) a.lse[row] = empty ? -INFINITY : lse2 * kLn2;
        } else {
            const int64_t slot = ((int64_t)pair * a.n_splits + split) * p.rows + r;
            a.part_o[slot * D + d] = value;
            if (d == 0) a.part_lse[slot] = lse2;
        }
    }
}

// Log-sum-exp merge of the chunk partials of one query row; one block per (sequence, KV
// head, row), one thread per output dim.
template <int D>
__global__ void __launch_bounds__(D)
grouped_merge_kernel(const GroupedParams p)
{
    const AttnParams &a = p.a;
    const int pair = blockIdx.x / p.rows, r = blockIdx.x - pair * p.rows;
    const int b = pair / a.heads, hk = pair - b * a.heads;
    allow_next_kernel();
    wait_for_previous_kernels();
    const int len = checked_seq_len(a, b, threadIdx.x == 0 && hk == 0 && r == 0);
    const int live = live_chunks(a, len);
    const int64_t row = grouped_row_index(p, b, hk, r);
    const int64_t first = (int64_t)pair * a.n_splits * p.rows + r;      // slot of chunk 0
    float top = kMinusHuge;
    for (int s = 0; s < live; ++s) top = fmaxf(top, a.part_lse[first + (int64_t)s * p.rows]);
    if (!(top > kMinusHuge)) {                 // no chunk holds a position this row may see
        a.out[row * D + threadIdx.x] = __float2half_rn(0.f);
        if (a.lse && threadIdx.x == 0) a.lse[row] = -INFINITY;
        return;
    }
    float total = 0.f, acc = 0.f;
    for (int s = 0; s < live; ++s) {
        const int64_t slot = first + (int64_t)s * p.rows;
        const float w = fast_exp2(a.part_lse[slot] - top);
        total += w;
        acc = fmaf(w, a.part_o[slot * D + threadIdx.x], acc);
    }
    a.out[row * D + threadIdx.x] = __float2half_rn(acc / total);
    if (a.lse && threadIdx.x == 0) a.lse[row] = (top + log2f(total)) * kLn2;
}

}  // namespace instinfer
