// Split-KV decode attention for several query rows per KV head on the fifth-generation tensor
// cores (tcgen05 MMAs with accumulators in tensor memory), head size 128, for sm_100a.
//
// Same operation and same split plan as grouped_attn_split_kernel (grouped heads and several
// new tokens per step put R <= 16 query rows against one KV head's cache: the paper's "other
// configurations", Sec. IV-C, on the Logit / Attend operators of Sec. III-B).  Here the two
// contractions are written with the TOKENS as the long side of the MMA, so that nothing is
// padding:
//   S^T[128 tokens x 16 rows]  = K_tile[128 x D] Q^T[D x 16]        (M = 128, N = 16, K = D)
//   O^T[D x 32]               += V_tile^T[D x 128] P^T[128 x 32]    (M = D = 128, N = 32, K = 128)
// where the 32 columns of P^T are the fp16 high and low parts of the 16 rows' softmax weights
// (so that the result keeps fp32-level accuracy), added up in the epilogue.
//
// A block owns one chunk of token positions of one (sequence, KV head) and is specialised by
// warp:
//   * warp 4 (producer) moves 128-token tiles of K and of V with tensor-map copies
//     (cp.async.bulk.tensor, 128-byte swizzle, this GPU's memory, no multicast) into a ring of
//     32 KiB slots; a paged tile is 128 / T copies of one (block, head) run each, the block
//     ids read one tile ahead; a block with a bad id is not fetched but zero-filled;
//   * one lane of warp 5 issues the MMAs: K tile (K-major, as it lies in the cache) against the
//     query rows held in shared memory -> logits in tensor memory (two buffers, so the next
//     tile's logits are computed while this tile's are being exponentiated); V tile (the same
//     bytes read MN-major: no transpose anywhere) against the weights in shared memory ->
//     the output accumulator in tensor memory;
//   * warps 0-3 (softmax): thread t owns token t of the tile, i.e. lane t of tensor memory: it
//     reads its 16 logits, masks, exponentiates against per-row references that all threads
//     hold alike and that follow the maximum lazily (a reference moves only when a logit
//     exceeds it by more than kGroupLag; then the accumulator in tensor memory is rescaled,
//     which is rare), and writes its 32 fp16 weights where the second MMA expects them;
//   * the epilogue reads the accumulator (thread = output dim), adds the high and low halves,
//     divides by the row sums and writes the chunk's partial (or the result itself when the
//     sequence is one chunk).
// Every wait is on an mbarrier and bounded by the clock; a wait that runs out sets
// kFlagCopyTimeout, the block stops waiting, releases its tensor memory and ends.
#pragma once

#include <cuda.h>

#include "grouped_attention_kernels.cuh"

namespace instinfer {

constexpr int kUmmaTile = 128;                         // tokens per tile
constexpr int kUmmaPanelBytes = kUmmaTile * 128;       // 64 dims of 128 tokens (rows of 128 bytes)
constexpr int kUmmaItemBytes = 2 * kUmmaPanelBytes;    // a K tile, or a V tile: 32 KiB
constexpr int kUmmaSlots = 3;
constexpr int kUmmaQBytes = kGroupRows * 256;          // 16 query rows, core-matrix order
constexpr int kUmmaPBytes = 32 * kUmmaTile * 2;        // 32 weight columns of 128 tokens
constexpr int kUmmaMiscBytes = 1024;                   // barriers, tensor-memory address, reductions
constexpr int kUmmaCarveBytes = kUmmaSlots * kUmmaItemBytes + kUmmaQBytes + kUmmaPBytes + kUmmaMiscBytes;
constexpr int kUmmaSmemBytes = kUmmaCarveBytes + 1024; // room to align the ring to 1024 bytes
constexpr int kUmmaThreads = 192;                      // 4 softmax warps, producer warp, MMA warp
constexpr int kUmmaCtasPerSm = 2;
constexpr int kUmmaTmemCols = 64;                      // 2 x 16 logits, 32 output accumulator

// offsets inside the misc region
constexpr int kUmmaBarFull = 0;        // [kUmmaSlots] tile landed
constexpr int kUmmaBarEmpty = 24;      // [kUmmaSlots] the MMAs that read the slot are complete
constexpr int kUmmaBarSFull = 48;      // [2] logits of a tile are in tensor memory
constexpr int kUmmaBarSFree = 64;      // [2] the softmax warps have read them
constexpr int kUmmaBarPFull = 80;      // weights of a tile are in shared memory
constexpr int kUmmaBarPvDone = 88;     // the second MMA of a tile is complete
constexpr int kUmmaTmemPtr = 96;
constexpr int kUmmaAbort = 100;        // set by a softmax thread whose wait ran out
constexpr int kUmmaRed = 128;          // [4][16] floats: per-warp row maxima, later row sums

// ---- tcgen05 / TMA wrappers ----------------------------------------------------------------
__device__ __forceinline__ void mbarrier_arrive(unsigned bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_proxy()    // generic-proxy writes -> visible to the MMA / TMA units
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned bar)   // arrives on bar when all MMAs issued so far are complete
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_f16(unsigned d_tmem, uint64_t a_desc, uint64_t b_desc, unsigned idesc,
                                           unsigned accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_load16(float (&v)[16], unsigned taddr)     // 16 columns of this thread's lane
{
    unsigned r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_store16(unsigned taddr, const float (&v)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 :: "r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                    "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
                    "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
                    "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                    "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
                    "r"(__float_as_uint(v[15])) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// One box of a 2-D tensor map (x: element column, y: row) into shared memory; its bytes are
// reported to the mbarrier.  x is a multiple of 64 fp16 elements here (128 bytes).
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap *map, int x, int y, unsigned bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Shared-memory matrix descriptor: start address, leading and stride byte offsets (all in
// 16-byte units), descriptor version 1, swizzle mode (0 none, 2 = 128 bytes).
__device__ __forceinline__ uint64_t umma_desc(unsigned addr, unsigned leading_bytes, unsigned stride_bytes,
                                              unsigned swizzle)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (uint64_t)(leading_bytes >> 4) << 16 |
           (uint64_t)(stride_bytes >> 4) << 32 | (uint64_t)1 << 46 | (uint64_t)swizzle << 61;
}
// Instruction descriptor, kind::f16: fp16 A and B, fp32 accumulator, M x N, operand majors
// (0: K-major, 1: MN-major).
__host__ __device__ constexpr unsigned umma_idesc(int m, int n, int a_mn_major, int b_mn_major)
{
    return 1u << 4 | (unsigned)a_mn_major << 15 | (unsigned)b_mn_major << 16 | (unsigned)(n >> 3) << 17 |
           (unsigned)(m >> 4) << 24;
}
// Barrier over the 128 softmax threads that also ORs a predicate.
__device__ __forceinline__ bool softmax_any(bool mine)
{
    unsigned out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.or.pred p, 1, 128, q;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(out) : "r"((unsigned)mine) : "memory");
    return out != 0;
}
__device__ __forceinline__ void softmax_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }

template <bool kPaged>
__global__ void __launch_bounds__(kUmmaThreads, kUmmaCtasPerSm)
grouped_attn_umma_kernel(const GroupedParams p, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v)
{
    constexpr int D = 128;
    extern __shared__ unsigned char smem_raw[];
    const AttnParams &a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
    if (begin >= len) {                        // the whole block leaves before anything is set up
        if (final_writer) {                    // inactive slot: zero output, lse = -inf
            for (int i = threadIdx.x; i < p.rows * D; i += kUmmaThreads) {
                const int r = i / D, d = i - r * D;
                const int64_t row = grouped_row_index(p, b, hk, r);
                a.out[row * D + d] = __float2half_rn(0.f);
                if (a.lse && d == 0) a.lse[row] = -INFINITY;
            }
        }
        return;
    }
    const int end = min(begin + chunk_size, len);
    const int n_tiles = (end - begin + kUmmaTile - 1) / kUmmaTile;

    // Shared memory: ring (1024-byte aligned: the 128-byte swizzle is a function of the address),
    // query rows, weights, misc.
    const unsigned raw = static_cast<unsigned>(__cvta_generic_to_shared(smem_raw));
    const unsigned ring = (raw + 1023u) & ~1023u;
    unsigned char *smem = smem_raw + (ring - raw);
    const unsigned q_smem = ring + kUmmaSlots * kUmmaItemBytes;
    const unsigned p_smem = q_smem + kUmmaQBytes;
    const unsigned misc = p_smem + kUmmaPBytes;
    unsigned char *misc_ptr = smem + kUmmaSlots * kUmmaItemBytes + kUmmaQBytes + kUmmaPBytes;
    volatile unsigned *abort_word = reinterpret_cast<volatile unsigned *>(misc_ptr + kUmmaAbort);
    float *red = reinterpret_cast<float *>(misc_ptr + kUmmaRed);

    // ---- set-up ----
    if (warp == 5) {                           // tensor memory: one warp allocates and later frees
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(misc + kUmmaTmemPtr), "n"(kUmmaTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else if (warp == 4) {
        if (lane == 0) {
#pragma unroll
            for (int s = 0; s < kUmmaSlots; ++s) {
                mbarrier_init(misc + kUmmaBarFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarEmpty + s * 8, 1);
            }
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                mbarrier_init(misc + kUmmaBarSFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarSFree + s * 8, 4);
            }
            mbarrier_init(misc + kUmmaBarPFull, 4);
            mbarrier_init(misc + kUmmaBarPvDone, 1);
            mbarrier_init_fence();
            *abort_word = 0u;
            asm volatile("prefetch.tensormap [%0];" :: "l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
            asm volatile("prefetch.tensormap [%0];" :: "l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
        }
    } else {
        // Query rows as operand B of the first MMA (N = 16 rows, K = D, K-major, no swizzle):
        // 8 x 16-byte core matrices, 128 bytes each; along K at 128 bytes, the second group of
        // 8 rows at 2048 bytes.  Rows beyond p.rows are zero.
        for (int i = threadIdx.x; i < kGroupRows * 16; i += 128) {
            const int r = i >> 4, seg = i & 15;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < p.rows) v = reinterpret_cast<const uint4 *>(a.q + grouped_row_index(p, b, hk, r) * D)[seg];
            *reinterpret_cast<uint4 *>(smem + kUmmaSlots * kUmmaItemBytes + (r >> 3) * 2048 + seg * 128 + (r & 7) * 16) = v;
        }
        fence_async_proxy();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = *reinterpret_cast<volatile unsigned *>(misc_ptr + kUmmaTmemPtr);

    if (warp == 4) {
        // ================================ producer ================================
        const int T = kPaged ? a.block_tokens : kUmmaTile;
        const int32_t *table_row = kPaged ? a.block_table + (int64_t)b * a.max_blocks_per_seq : nullptr;
        const int64_t total_rows = a.kv_bytes / (2 * D);
        auto fetch_ids = [&](int j) -> int {           // lane i: physical block of the tile's i-th block
            if (!kPaged) return 0;
            const int tile_start = begin + j * kUmmaTile;
            const int nb = (min(end - tile_start, kUmmaTile) + T - 1) / T;
            const int idx = tile_start / T + lane;
            if (j >= n_tiles || lane >= nb || !bounds_ok(idx < a.max_blocks_per_seq, a.status)) return -1;
            return __ldg(table_row + idx);
        };
        int ids_next = fetch_ids(0);
        int issued = 0;
        bool fine = true;
        for (int j = 0; j < n_tiles && fine; ++j) {
            const int tile_start = begin + j * kUmmaTile;
            const int nb = kPaged ? (min(end - tile_start, kUmmaTile) + T - 1) / T : 1;
            const int phys = ids_next;
            ids_next = fetch_ids(j + 1);
            bool good = lane < nb;
            int row0;
            if (kPaged) {
                const bool in_range = phys >= 0 && (int64_t)phys < a.num_phys_blocks;
                if (good && !in_range && a.status) atomicOr(a.status, kFlagBlockRange);
                row0 = in_range ? (phys * a.heads + hk) * T : 0;      // < 2^31 rows: checked by the host
                good = good && in_range && bounds_ok((int64_t)row0 + T <= total_rows, a.status);
            } else {
                row0 = pair * a.s_max + tile_start;            // rows past the tensor's end read as zeros
            }
            for (int which = 0; which < 2 && fine; ++which) {
                const int item = 2 * j + which;
                const int slot = item % kUmmaSlots;
                if (item >= kUmmaSlots)
                    fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarEmpty + slot * 8,
                                                                         (item / kUmmaSlots - 1) & 1));
                if (!fine) break;
                const unsigned dst = ring + slot * kUmmaItemBytes + (kPaged ? lane * T * 128 : 0);
                const unsigned bar = misc + kUmmaBarFull + slot * 8;
                if (kPaged && lane < nb && !good) {            // a block that cannot be read counts as zeros
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    unsigned char *z = smem + slot * kUmmaItemBytes + lane * T * 128;
                    for (int i = 0; i < T * 8; ++i) {
                        *reinterpret_cast<uint4 *>(z + i * 16) = zero;
                        *reinterpret_cast<uint4 *>(z + kUmmaPanelBytes + i * 16) = zero;
                    }
                    fence_async_proxy();
                }
                const unsigned fetched = __popc(__ballot_sync(0xffffffffu, good));
                __syncwarp();
                if (lane == 0) mbarrier_expect_bytes(bar, fetched * (unsigned)T * 256u);
                __syncwarp();
                if (good) {
                    const CUtensorMap *map = which == 0 ? &map_k : &map_v;
                    tma_load_2d(dst, map, 0, row0, bar);
                    tma_load_2d(dst + kUmmaPanelBytes, map, 64, row0, bar);
                }
                ++issued;
            }
        }
        if (!fine) {
            if (lane == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
            // copies in flight must land (or be given up, bounded) before shared memory is handed on
            for (int item = max(issued - kUmmaSlots, 0); item < issued; ++item)
                (void)mbarrier_wait_bounded(misc + kUmmaBarFull + (item % kUmmaSlots) * 8, (item / kUmmaSlots) & 1);
        }
    } else if (warp == 5) {
        // ================================ MMA issue ================================
        if (lane == 0) {
            constexpr unsigned idesc_logits = umma_idesc(128, 16, 0, 0);   // K tile K-major, Q K-major
            constexpr unsigned idesc_output = umma_idesc(128, 32, 1, 1);   // V tile MN-major, weights MN-major
            auto logits = [&](int j) -> bool {
                const int item = 2 * j, slot = item % kUmmaSlots;
                if (!mbarrier_wait_bounded(misc + kUmmaBarFull + slot * 8, (item / kUmmaSlots) & 1)) return false;
                if (j >= 2 && !mbarrier_wait_bounded(misc + kUmmaBarSFree + (j & 1) * 8, ((j >> 1) - 1) & 1)) return false;
                tc_fence_after();
                const unsigned k_tile = ring + slot * kUmmaItemBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    // K tile: rows of 128 bytes per 64-dim panel, 8-row groups 1024 bytes apart,
                    // 128-byte swizzle; a k-step of 16 dims is 32 bytes further along the row
                    const uint64_t ad = umma_desc(k_tile + (ks >> 2) * kUmmaPanelBytes + (ks & 3) * 32, 16, 1024, 2);
                    const uint64_t bd = umma_desc(q_smem + ks * 256, 128, 2048, 0);
                    tc_mma_f16(tmem + (j & 1) * 16, ad, bd, idesc_logits, ks > 0);
                }
                tc_commit(misc + kUmmaBarSFull + (j & 1) * 8);
                tc_commit(misc + kUmmaBarEmpty + slot * 8);
                return true;
            };
            auto output = [&](int j) -> bool {
                const int item = 2 * j + 1, slot = item % kUmmaSlots;
                if (!mbarrier_wait_bounded(misc + kUmmaBarFull + slot * 8, (item / kUmmaSlots) & 1)) return false;
                if (!mbarrier_wait_bounded(misc + kUmmaBarPFull, j & 1)) return false;
                tc_fence_after();
                const unsigned v_tile = ring + slot * kUmmaItemBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    // V tile read MN-major (M = dims): the two 64-dim panels are kUmmaPanelBytes
                    // apart (leading offset), 8-token groups 1024 bytes apart; a k-step is 16 tokens.
                    // Weights: 8-column blocks of [128 tokens][16 bytes], 2048 bytes apart; 8-token
                    // groups 128 bytes apart.
                    const uint64_t ad = umma_desc(v_tile + ks * 2048, kUmmaPanelBytes, 1024, 2);
                    const uint64_t bd = umma_desc(p_smem + ks * 256, 128, 2048, 0);
                    tc_mma_f16(tmem + 32, ad, bd, idesc_output, j > 0 || ks > 0);
                }
                tc_commit(misc + kUmmaBarEmpty + slot * 8);
                tc_commit(misc + kUmmaBarPvDone);
                return true;
            };
            bool fine = logits(0);
            for (int j = 0; j < n_tiles && fine; ++j) {
                if (j + 1 < n_tiles) fine = logits(j + 1);
                if (fine) fine = output(j);
            }
            if (!fine && a.status) atomicOr(a.status, kFlagCopyTimeout);
        }
        __syncwarp();
    } else {
        // ================================ softmax and epilogue ================================
        const int t = threadIdx.x;                                 // token of the tile = lane of tensor memory
        const unsigned lane_base = tmem + ((unsigned)(warp * 32) << 16);
        float m[16], l[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            m[r] = kMinusHuge;
            l[r] = 0.f;
        }
        const int unmasked_end = min(end, len - (p.q_tokens - 1));  // tiles ending here or before need no mask
        bool aborted = false;
        for (int j = 0; j < n_tiles; ++j) {
            const int sb = j & 1;
            // (warp-uniform: the tensor-memory loads below are warp-wide instructions)
            bool fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarSFull + sb * 8, (j >> 1) & 1));
            float s[16];
            if (fine) {
                tc_fence_after();
                tc_load16(s, lane_base + sb * 16);
                tc_fence_before();
            } else {
#pragma unroll
                for (int r = 0; r < 16; ++r) s[r] = 0.f;
            }
            __syncwarp();
            if (lane == 0) mbarrier_arrive(misc + kUmmaBarSFree + sb * 8);
            const int tile_start = begin + j * kUmmaTile;
            const int tok = tile_start + t;
#pragma unroll
            for (int r = 0; r < 16; ++r) s[r] *= a.scale_log2e;
            if (tile_start + kUmmaTile > unmasked_end) {           // uniform: last tiles of the sequence / chunk
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    const int vis = r < p.rows ? len - (p.q_tokens - 1 - r / p.group) : 0;
                    if (tok >= min(vis, end)) s[r] = -INFINITY;
                }
                if (tok >= end) {
                    // The value row of a position outside the chunk gets weight zero, but its bytes
                    // may be anything (the tail of a block, a slot not fetched): 0 x NaN must not
                    // reach the accumulator, so the row is cleared once the tile has landed.
                    const int item = 2 * j + 1, slot = item % kUmmaSlots;
                    fine = mbarrier_wait_bounded(misc + kUmmaBarFull + slot * 8, (item / kUmmaSlots) & 1) && fine;
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    unsigned char *vrow = smem + slot * kUmmaItemBytes + t * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        *reinterpret_cast<uint4 *>(vrow + i * 16) = zero;
                        *reinterpret_cast<uint4 *>(vrow + kUmmaPanelBytes + i * 16) = zero;
                    }
                }
            }
            bool moved = false;
#pragma unroll
            for (int r = 0; r < 16; ++r) moved = moved || s[r] > m[r] + kGroupLag;
            if (!fine) *abort_word = 1u;
            bool waited = false;
            if (softmax_any(moved || !fine)) {
                if (*abort_word != 0u) {                            // the same for all 128 threads
                    aborted = true;
                    break;
                }
                // Some row's reference moves: row maxima over the tile, new references, and the
                // accumulator (and the sums) rescaled to them.
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    float top = s[r];
                    top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 1));
                    top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 2));
                    top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 4));
                    top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 8));
                    top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 16));
                    if (lane == 0) red[warp * 16 + r] = top;
                }
                softmax_sync();
                float alpha[16];
                bool any_change = false;
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    const float top = fmaxf(fmaxf(red[r], red[16 + r]), fmaxf(red[32 + r], red[48 + r]));
                    alpha[r] = 1.f;
                    if (top > m[r] + kGroupLag) {
                        alpha[r] = fast_exp2(m[r] - top);
                        m[r] = top;
                        any_change = true;
                    }
                    l[r] *= alpha[r];
                }
                if (j > 0 && any_change) {
                    // the accumulator holds tiles 0 .. j-1 once the previous tile's MMA is complete
                    fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarPvDone, (j - 1) & 1));
                    waited = true;
                    if (fine) {
                        tc_fence_after();
                        float o[16];
#pragma unroll
                        for (int half = 0; half < 2; ++half) {      // columns 0-15: high parts, 16-31: low parts
                            tc_load16(o, lane_base + 32 + half * 16);
#pragma unroll
                            for (int r = 0; r < 16; ++r) o[r] *= alpha[r];
                            tc_store16(lane_base + 32 + half * 16, o);
                        }
                    } else {
                        *abort_word = 1u;                           // seen by all at the next tile's vote
                    }
                }
            }
            // Weights against the references (scaled by kGroupWeightScale inside the exponent),
            // their sums, and the fp16 high and low parts: thread t holds row t of operand B
            // (MN-major: 8 columns = 16 bytes per token and column block).
            unsigned hi[8], lo[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float w0 = fast_exp2(s[2 * i] - (m[2 * i] - kGroupWeightLog2));
                const float w1 = fast_exp2(s[2 * i + 1] - (m[2 * i + 1] - kGroupWeightLog2));
                l[2 * i] += w0;
                l[2 * i + 1] += w1;
                hi[i] = pack_half2(w0, w1);
                const float2 back = __half22float2(*reinterpret_cast<const __half2 *>(&hi[i]));
                lo[i] = pack_half2(w0 - back.x, w1 - back.y);
            }
            if (j > 0 && !waited && fine) {                         // the previous MMA has read the weights
                fine = mbarrier_wait_bounded(misc + kUmmaBarPvDone, (j - 1) & 1);
                if (!fine) *abort_word = 1u;
            }
            unsigned char *prow = smem + kUmmaSlots * kUmmaItemBytes + kUmmaQBytes + t * 16;
            *reinterpret_cast<uint4 *>(prow) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4 *>(prow + 2048) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            *reinterpret_cast<uint4 *>(prow + 4096) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            *reinterpret_cast<uint4 *>(prow + 6144) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
            fence_async_proxy();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbarrier_arrive(misc + kUmmaBarPFull);
        }
        if (!aborted) aborted = softmax_any(*abort_word != 0u) || false;
        if (aborted) {
            if (t == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
        } else if (!mbarrier_wait_bounded(misc + kUmmaBarPvDone, (n_tiles - 1) & 1)) {
            if (a.status) atomicOr(a.status, kFlagCopyTimeout);
            aborted = true;
        }
        // Row sums over the block (every thread joins the barrier, also after a give-up).
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            float sum = l[r];
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            sum += __shfl_xor_sync(0xffffffffu, sum, 4);
            sum += __shfl_xor_sync(0xffffffffu, sum, 8);
            sum += __shfl_xor_sync(0xffffffffu, sum, 16);
            if (lane == 0) red[warp * 16 + r] = sum;
        }
        softmax_sync();
        if (!softmax_any(aborted)) {
            // Epilogue: thread t owns output dim t; columns r and 16 + r are the high and low
            // parts of row r.  Sums and accumulator both carry kGroupWeightScale.
            tc_fence_after();
            float o_hi[16], o_lo[16];
            tc_load16(o_hi, lane_base + 32);
            tc_load16(o_lo, lane_base + 48);
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                if (r < p.rows) {
                    const float total = (red[r] + red[16 + r]) + (red[32 + r] + red[48 + r]);
                    // A row that sees no position of this chunk (causal limit before the chunk) has total 0.
                    const bool empty = !(total > 0.f);
                    const float value = empty ? 0.f : (o_hi[r] + o_lo[r]) / total;
                    const float lse2 = empty ? kMinusHuge : m[r] + log2f(total) - kGroupWeightLog2;
                    if (final_writer) {
                        const int64_t row = grouped_row_index(p, b, hk, r);
                        a.out[row * D + t] = __float2half_rn(value);
                        if (a.lse && t == 0) a.lse[row] = empty ? -INFINITY : lse2 * kLn2;
                    } else {
                        const int64_t slot = ((int64_t)pair * a.n_splits + split) * p.rows + r;
                        a.part_o[slot * D + t] = value;
                        if (t == 0) a.part_lse[slot] = lse2;
                    }
                }
            }
        }
    }

    // ---- teardown: everyone is done with tensor memory before it is released ----
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "n"(kUmmaTmemCols) : "memory");
    }
}

}  // namespace instinfer
