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
// Softmax weights enter the second MMA as fp16 hi + lo of weight * 2^kGroupWeightLog2.  A
// reference may lag its row's maximum by kGroupLag (base 2), so weights reach 2^kGroupLag and
// the scaled ones 2^15 < 65504.  Small weights fall into fp16 subnormals, where hi and lo each
// carry an absolute error below 2^-25 (scaled), i.e. below 2^-26 of the row's largest weight.
constexpr float kGroupLag = 7.f;
constexpr float kGroupWeightLog2 = 8.f;
constexpr float kGroupWeightScale = 256.f;

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
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, "
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

// One 16-token tile against the 16 query rows: logits, online softmax, and O += P V.  `base`
// is the stage's shared-memory address; the running state (references, sums, output fragments)
// is updated in place.
template <int D>
__device__ __forceinline__ void grouped_tile(unsigned base, unsigned k_rd, unsigned v_rd, unsigned q_rd,
                                             const unsigned (&qa)[GroupedGeometry<D>::kQInSmem ? 1 : GroupedGeometry<D>::kKSteps][4],
                                             int tok0, int unmasked_end, int vis_lo, int vis_hi,
                                             float scale_log2e, int quad, float &m_lo, float &m_hi,
                                             float &l_lo, float &l_hi, float (&o)[D / 8][4])
{
    using G = GroupedGeometry<D>;
    // Logits of 16 rows x 16 tokens: s[n][0..1] row gid, s[n][2..3] row gid + 8, tokens
    // tok0 + 8 n + 2 quad + {0, 1}.  Even and odd k-steps accumulate separately so that
    // four independent MMA chains are in flight.
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float s_odd[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int ks = 0; ks < G::kKSteps; ++ks) {
        unsigned kb[4];
        ldmatrix_x4(kb, base + k_rd + ks * 32);
        float (&acc)[2][4] = (ks & 1) ? s_odd : s;
        if (G::kQInSmem) {
            unsigned qf[4];
            ldmatrix_x4(qf, q_rd + ks * 32);
            mma_16816(acc[0], qf, kb[0], kb[1]);
            mma_16816(acc[1], qf, kb[2], kb[3]);
        } else {
            mma_16816(acc[0], qa[ks], kb[0], kb[1]);
            mma_16816(acc[1], qa[ks], kb[2], kb[3]);
        }
    }
#pragma unroll
    for (int n = 0; n < 2; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[n][e] = (s[n][e] + s_odd[n][e]) * scale_log2e;
    }
    if (tok0 + kGroupTile > unmasked_end) {      // uniform: last tiles of the sequence only
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = tok0 + n * 8 + quad * 2 + e;
                if (tok >= vis_lo) s[n][e] = -INFINITY;
                if (tok >= vis_hi) s[n][2 + e] = -INFINITY;
            }
        }
    }
    // Online softmax with per-row references that may lag the true maximum by up to
    // kGroupLag (base-2 units): weights reach at most 2^kGroupLag, inside the range of the
    // fp16 weight split.  References move, and accumulators are rescaled, only when some
    // logit exceeds its row's reference by more than that: with 16 rows sharing the
    // rescaling, a tight lag would rescale on most tiles of a short chunk.
    const float top_lo_here = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
    const float top_hi_here = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
    if (__any_sync(0xffffffffu, top_lo_here > m_lo + kGroupLag || top_hi_here > m_hi + kGroupLag)) {
        float top_lo = top_lo_here, top_hi = top_hi_here;
        top_lo = fmaxf(top_lo, __shfl_xor_sync(0xffffffffu, top_lo, 1));
        top_lo = fmaxf(top_lo, __shfl_xor_sync(0xffffffffu, top_lo, 2));
        top_hi = fmaxf(top_hi, __shfl_xor_sync(0xffffffffu, top_hi, 1));
        top_hi = fmaxf(top_hi, __shfl_xor_sync(0xffffffffu, top_hi, 2));
        float alpha_lo = 1.f, alpha_hi = 1.f;
        if (top_lo > m_lo + kGroupLag) {
            alpha_lo = fast_exp2(m_lo - top_lo);
            m_lo = top_lo;
        }
        if (top_hi > m_hi + kGroupLag) {
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
    // Weights (scaled by kGroupWeightScale: the scale is folded into the exponent), their
    // sums, and the A fragments of P V as an fp16 hi + lo pair.
    const float e_lo = m_lo - kGroupWeightLog2, e_hi = m_hi - kGroupWeightLog2;
    unsigned p_hi[4], p_lo[4];
#pragma unroll
    for (int n = 0; n < 2; ++n) {
        float w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = fast_exp2(s[n][e] - (e < 2 ? e_lo : e_hi));
        l_lo += w[0] + w[1];
        l_hi += w[2] + w[3];
        p_hi[2 * n] = pack_half2(w[0], w[1]);
        p_hi[2 * n + 1] = pack_half2(w[2], w[3]);
        const float2 f_lo = __half22float2(*reinterpret_cast<const __half2 *>(&p_hi[2 * n]));
        const float2 f_hi = __half22float2(*reinterpret_cast<const __half2 *>(&p_hi[2 * n + 1]));
        p_lo[2 * n] = pack_half2(w[0] - f_lo.x, w[1] - f_lo.y);
        p_lo[2 * n + 1] = pack_half2(w[2] - f_hi.x, w[3] - f_hi.y);
    }
    // O += P V: two 8-dim output blocks per ldmatrix, four ldmatrix per group so that
    // eight independent accumulators separate the hi and the lo MMA of each block.
#pragma unroll
    for (int grp = 0; grp < D / 64; ++grp) {
        unsigned vb[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) ldmatrix_x4_trans(vb[i], base + v_rd + (grp * 4 + i) * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_16816(o[(grp * 4 + i) * 2], p_hi, vb[i][0], vb[i][1]);
            mma_16816(o[(grp * 4 + i) * 2 + 1], p_hi, vb[i][2], vb[i][3]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_16816(o[(grp * 4 + i) * 2], p_lo, vb[i][0], vb[i][1]);
            mma_16816(o[(grp * 4 + i) * 2 + 1], p_lo, vb[i][2], vb[i][3]);
        }
    }
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
    const int order = blockIdx.x / a.pairs;
    const int pair = blockIdx.x - order * a.pairs;
    const int split = scheduled_chunk(a, order);
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
    // tile sits at tile base + 16 s; in shared memory its row is padded.  Lane `lane` copies
    // segments lane + 32 i: global offset 16 lane + 512 i, shared offset lane_dst + i kDstStep.
    const unsigned ring = smem_base + warp * (kGroupStages * G::kStageBytes);
    constexpr int kTileRowSegs = D / 8;                          // 16-byte segments per row
    constexpr int kRowsPerPass = 32 / kTileRowSegs > 0 ? 32 / kTileRowSegs : 1;   // rows one warp copy covers
    constexpr int kPassesPerRow = kTileRowSegs / 32 > 0 ? kTileRowSegs / 32 : 1;  // D = 512 and up only
    static_assert(kPassesPerRow == 1, "rows longer than 512 bytes are not laid out here");
    constexpr unsigned kDstStep = kRowsPerPass * G::kRowStride;
    const int lane_row = lane / kTileRowSegs;
    const unsigned lane_dst = lane_row * G::kRowStride + (lane - lane_row * kTileRowSegs) * 16;
    const unsigned char *k_lane = reinterpret_cast<const unsigned char *>(a.k) + lane * 16;
    const unsigned char *v_lane = reinterpret_cast<const unsigned char *>(a.v) + lane * 16;
    constexpr int kStepTokens = kWarps * kGroupTile;             // a warp's next tile is this far ahead
    const int first_token = begin + warp * kGroupTile;
    // Walks this warp's tiles incrementally (no division per tile): contiguous byte offset,
    // or paged (block index, slot inside the block) and the table entry one tile ahead.
    int64_t src_off = 0, block_stride = 0, head_off = 0;
    int blk = 0, rem = 0, step_blk = 0, step_rem = 0, next_phys = 0;
    const int32_t *table_row = nullptr;
    if (kPaged) {
        const int tokens = a.block_tokens;
        table_row = a.block_table + (int64_t)b * a.max_blocks_per_seq;
        blk = first_token / tokens;
        rem = first_token - blk * tokens;
        step_blk = kStepTokens / tokens;
        step_rem = kStepTokens - step_blk * tokens;
        block_stride = (int64_t)a.heads * tokens * G::kRowBytes;
        head_off = (int64_t)hk * tokens * G::kRowBytes;
        next_phys = my_tiles > 0 && bounds_ok(blk < a.max_blocks_per_seq, a.status) ? __ldg(table_row + blk) : 0;
    } else {
        src_off = ((int64_t)pair * a.s_max + first_token) * G::kRowBytes;
    }

    int issue_j = 0;
    unsigned issue_stage = 0;
    auto issue = [&]() {
        if (issue_j < my_tiles) {
            const int rows_here = end - (first_token + issue_j * kStepTokens);     // >= 1
            bool usable = true;
            int64_t off;
            if (kPaged) {
                const int phys = next_phys;
                usable = phys >= 0 && (int64_t)phys < a.num_phys_blocks;
                if (!usable && lane == 0 && a.status) atomicOr(a.status, kFlagBlockRange);
                off = usable ? (int64_t)phys * block_stride + head_off + rem * G::kRowBytes : 0;
                blk += step_blk;
                rem += step_rem;
                if (rem >= a.block_tokens) {
                    rem -= a.block_tokens;
                    ++blk;
                }
                if (issue_j + 1 < my_tiles)
                    next_phys = bounds_ok(blk < a.max_blocks_per_seq, a.status) ? __ldg(table_row + blk) : -1;
            } else {
                off = src_off;
                src_off += (int64_t)kStepTokens * G::kRowBytes;
            }
            usable = usable && bounds_ok(off >= 0 && off + (int64_t)min(rows_here, kGroupTile) * G::kRowBytes <= a.kv_bytes, a.status);
            if (!usable) off = 0;
            const unsigned char *ks = k_lane + off, *vs = v_lane + off;
            const unsigned dst = ring + issue_stage * G::kStageBytes + lane_dst;
            if (usable && rows_here >= kGroupTile) {               // full tile: no predicates
#pragma unroll
                for (int i = 0; i < G::kSegsPerLane; ++i) {
                    cp_async_16(dst + i * kDstStep, ks + i * 512, 16);
                    cp_async_16(dst + i * kDstStep + G::kTileBytes, vs + i * 512, 16);
                }
            } else {                                               // ragged tail: masked rows are zero-filled
#pragma unroll
                for (int i = 0; i < G::kSegsPerLane; ++i) {
                    const bool valid = usable && lane_row + i * kRowsPerPass < rows_here;
                    const int src = valid ? i * 512 : 0;
                    cp_async_16(dst + i * kDstStep, ks + src, valid ? 16 : 0);
                    cp_async_16(dst + i * kDstStep + G::kTileBytes, vs + src, valid ? 16 : 0);
                }
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
    // lane's share of the sum l, and the output fragments; l and o carry kGroupWeightScale.
    float m_lo = kMinusHuge, m_hi = kMinusHuge, l_lo = 0.f, l_hi = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    // Tiles that end at or before this position need no causal or length mask for any row.
    const int unmasked_end = len - (p.q_tokens - 1);

#pragma unroll
    for (int j = 0; j < kGroupStages - 1; ++j) issue();

    unsigned stage = 0;
    for (int j = 0; j < my_tiles; ++j) {
        cp_async_wait<kGroupStages - 2>();
        __syncwarp();                    // tile j visible to the warp; everyone is done with tile j-1
        issue();                         // refills the slot tile j-1 used
        const unsigned base = ring + stage * G::kStageBytes;
        stage = stage + 1 == kGroupStages ? 0 : stage + 1;
        const int tok0 = first_token + j * kStepTokens;

        grouped_tile<D>(base, k_rd, v_rd, q_rd, qa, tok0, unmasked_end, vis_lo, vis_hi, a.scale_log2e, quad,
                        m_lo, m_hi, l_lo, l_hi, o);
    }
    cp_async_wait<0>();

    // Row sums over the four lanes that share a row (both l and o carry kGroupWeightScale).
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
        const float lse2 = empty ? kMinusHuge : top + log2f(total) - kGroupWeightLog2;
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
    const int parts = live_chunks(a, len);
    const int64_t row = grouped_row_index(p, b, hk, r);
    const int64_t first = (int64_t)pair * a.n_splits * p.rows + r;      // slot of chunk 0
    float top = kMinusHuge;
    for (int s = 0; s < parts; ++s) top = fmaxf(top, a.part_lse[first + (int64_t)s * p.rows]);
    if (!(top > kMinusHuge)) {                 // no part holds a position this row may see
        a.out[row * D + threadIdx.x] = __float2half_rn(0.f);
        if (a.lse && threadIdx.x == 0) a.lse[row] = -INFINITY;
        return;
    }
    float total = 0.f, acc = 0.f;
    for (int s = 0; s < parts; ++s) {
        const int64_t slot = first + (int64_t)s * p.rows;
        const float w = fast_exp2(a.part_lse[slot] - top);
        total += w;
        acc = fmaf(w, a.part_o[slot * D + threadIdx.x], acc);
    }
    a.out[row * D + threadIdx.x] = __float2half_rn(acc / total);
    if (a.lse && threadIdx.x == 0) a.lse[row] = (top + log2f(total)) * kLn2;
}

}  // namespace instinfer
