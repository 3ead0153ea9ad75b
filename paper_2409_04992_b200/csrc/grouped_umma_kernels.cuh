// Split-KV decode attention for several query rows per KV head on the fifth-generation tensor
// cores (tcgen05 MMAs with accumulators in tensor memory), head sizes 128 and 256, for sm_100a.
//
// Same operation and same split plan as grouped_attn_split_kernel (grouped heads and several
// new tokens per step put R <= 16 query rows against one KV head's cache: the paper's "other
// configurations", Sec. IV-C, on the Logit / Attend operators of Sec. III-B).  Here the two
// contractions are written with the TOKENS as the long side of the MMA, so that nothing is
// padding:
//   S^T[128 tokens x 16 rows]  = K_tile[128 x D] Q^T[D x 16]        (M = 128, N = 16, K = D)
//   O^T[D x 32]               += V_tile^T[D x 128] P^T[128 x 32]    (M = 128 dims at a time, N = 32, K = 128)
// where the 32 columns of P^T are the fp16 high and low parts of the 16 rows' softmax weights
// (so that the result keeps fp32-level accuracy), added up in the epilogue.  With head size 256
// the first product takes its K in two halves and the second is two MMAs into two accumulators.
//
// The kernel is persistent: one block per SM draws chunks (token ranges of one (sequence, KV
// head), the same list one block per chunk would run) from a ticket counter, and its copy
// pipeline runs on across chunk boundaries.  A block has eight warps, each with one job, that
// hand tiles to one another through mbarriers:
//   * warp 4 (K producer) moves 128-token tiles of K with tensor-map copies (cp.async.bulk.tensor,
//     128-byte swizzle, this GPU's memory, every block fetching its own tiles) into a ring of
//     three 32 KiB slots (128 dims of a tile each: head size 256 takes two per tile); a
//     paged tile is 128 / T copies of one (block, head) run each (one copy of 128 rows where a
//     block holds a multiple of 128 tokens), the block ids read one tile
//     ahead; a block with a bad id is not fetched but zero-filled.  It also draws the tickets
//     (two chunks ahead, so the atomic's round trip is hidden), announces each chunk to the
//     other warps through a small queue in shared memory and fetches the chunk's query rows;
//   * warp 5 (V producer) does the same for the V tiles into a ring of its own;
//   * warp 6 issues the logit MMAs: K tile (K-major, as it lies in the cache) against the query
//     rows -> logits in tensor memory (two buffers, so it runs up to two tiles ahead of the
//     softmax); warp 7 issues the output MMAs: V tile (the same bytes read MN-major: no
//     transpose anywhere) against the weights in shared memory -> the accumulator in tensor
//     memory (one per chunk parity).  One thread issuing both took 2250 cycles per tile, more
//     than the tile's copy time: two issuers halve that.  Both warps run converged and
//     predicate only the issue, so descriptors stay warp-uniform values;
//   * warps 0-3 (softmax): thread t owns token t of the tile, i.e. lane t of tensor memory: it
//     reads its 16 logits, masks, exponentiates against per-row references that all threads
//     hold alike and that follow the maximum lazily (a reference moves only when a logit
//     exceeds it by more than kGroupLag; then the accumulator in tensor memory is rescaled,
//     which is rare), and writes its 32 fp16 weights where the output MMA expects them;
//   * a chunk's epilogue (thread = output dim: accumulator columns r and 16 + r added, divided
//     by the row sum, written as the chunk's partial, or as the result when the sequence is
//     one chunk) runs after the first tile of the next chunk has been handed on, so that
//     nothing waits for it.
// Waits of the warps that run ahead (producers, logit issuer) let the hardware park the warp;
// the waits on the chain softmax -> output MMA -> softmax poll, because there the time to
// notice a completed phase adds to every tile.
// Every wait is on an mbarrier and bounded by the clock; a wait that runs out sets
// kFlagCopyTimeout, the block stops waiting, releases its tensor memory and ends.
#pragma once

#include <cuda.h>

#include "grouped_attention_kernels.cuh"

namespace instinfer {

constexpr int kUmmaTile = 128;                         // tokens per tile
constexpr int kUmmaPanelBytes = kUmmaTile * 128;       // 64 dims of 128 tokens (rows of 128 bytes)
constexpr int kUmmaQBuffers = 2;                       // the next chunk's query rows arrive early
constexpr int kUmmaPBytes = 32 * kUmmaTile * 2;        // 32 weight columns of 128 tokens
constexpr int kUmmaMiscBytes = 2048;                   // barriers, work queue, tensor-memory address, reductions
constexpr int kUmmaThreads = 256;                      // 4 softmax warps, K and V producers, logit and output MMA issuers
constexpr int kUmmaWarpK = 4, kUmmaWarpV = 5, kUmmaWarpLogits = 6, kUmmaWarpOutput = 7;
constexpr int kUmmaQueue = 4;                          // chunks the producer may be ahead of the consumers
constexpr int kUmmaSlots = 3;                          // ring depth of each cache, in items (96 KiB)
constexpr int kUmmaItemPanels = 2;                     // panels per ring item: 128 dims of 128 tokens, 32 KiB
constexpr int kUmmaItemBytes = kUmmaItemPanels * kUmmaPanelBytes;

// Sizes that follow from the head size D (128 or 256).  A token row is D / 64 panels of 64 dims;
// the rings hold items of two panels, so a tile of head size 256 is two items per cache and the
// bytes in flight are the same for both head sizes.  (Head size 64 is not taken: a tile would
// be half the bytes for the same softmax work per token, and the softmax chain, one thread per
// token, then bounds the kernel: 4.4 TB/s measured, against 6.8 for the warp-level kernel.)
template <int D>
struct UmmaGeometry {
    static_assert(D == 128 || D == 256, "head sizes of the tcgen05 form");
    static constexpr int kPanels = D / 64;
    static constexpr int kItems = kPanels / kUmmaItemPanels;             // ring items per tile and cache
    static constexpr int kAccs = D / 128;                                // output accumulators of 128 dims
    static constexpr int kQBytes = kGroupRows * D * 2;                   // 16 query rows, panel by panel
    static constexpr int kTmemCols = D == 256 ? 256 : 128;               // 2 x 16 logits, 2 x kAccs x 32 output columns
    static constexpr int kCarveBytes = 2 * kUmmaSlots * kUmmaItemBytes + kUmmaQBuffers * kQBytes + kUmmaPBytes + kUmmaMiscBytes;
    static constexpr int kSmemBytes = kCarveBytes + 1024;                // room to align the rings to 1024 bytes
    static_assert(kSmemBytes <= 227 * 1024, "one block per SM must fit");
};

// offsets inside the misc region
constexpr int kUmmaBarKFull = 0;       // [slots] K item landed
constexpr int kUmmaBarKEmpty = 48;     // [slots] the logit MMAs that read the slot are complete
constexpr int kUmmaBarVFull = 96;      // [slots] V item landed
constexpr int kUmmaBarVEmpty = 144;    // [slots] the output MMAs that read the slot are complete
constexpr int kUmmaBarSFull = 192;     // [2] logits of a tile are in tensor memory
constexpr int kUmmaBarSFree = 208;     // [2] the softmax warps have read them
constexpr int kUmmaBarPFull = 224;     // weights of a tile are in shared memory
constexpr int kUmmaBarPvDone = 232;    // the output MMAs of a tile are complete
constexpr int kUmmaBarQFull = 240;     // [2] query rows of a chunk landed
constexpr int kUmmaBarQEmpty = 256;    // [2] the chunk's last logit MMA is complete
constexpr int kUmmaBarWorkFull = 272;  // [kUmmaQueue] a chunk is announced
constexpr int kUmmaBarWorkEmpty = 304; // [kUmmaQueue] all seven consumers have read the announcement
constexpr int kUmmaBarAccFree = 336;   // [2] the epilogue has read the accumulator of a chunk of this parity
constexpr int kUmmaTmemPtr = 352;
constexpr int kUmmaAbort = 356;        // set by a softmax thread whose wait ran out
constexpr int kUmmaWork = 384;         // [kUmmaQueue] int2 {chunk number or -1, sequence length}
constexpr int kUmmaRed = 448;          // [4][16] floats: per-warp row maxima of a tile
constexpr int kUmmaSavedM = 704;       // [2][16] floats: a finished chunk's references, by chunk parity
constexpr int kUmmaSavedL = 832;       // [2][4][16] floats: its per-warp row sums
static_assert(kUmmaBarKEmpty - kUmmaBarKFull >= 8 * kUmmaSlots && kUmmaWork + 8 * kUmmaQueue <= kUmmaRed, "barriers overlap");
static_assert(kUmmaSavedL + 512 <= kUmmaMiscBytes, "misc region too small");

// ---- tcgen05 / TMA wrappers ----------------------------------------------------------------
// The roles of this kernel hand tiles to one another in a chain (copy -> MMA -> softmax -> MMA),
// one or two warps per role, so the time a waiter takes to notice a completed phase adds to
// every tile: these waits poll (no suspend-time hint), still bounded by the clock.
__device__ __forceinline__ bool mbarrier_test(unsigned bar, unsigned parity)
{
    unsigned done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbarrier_poll_bounded(unsigned bar, unsigned parity)
{
    for (int i = 0; i < 64; ++i)
        if (mbarrier_test(bar, parity)) return true;
    const long long start = clock64();
    for (;;) {
        if (mbarrier_test(bar, parity)) return true;
        if (clock64() - start > kWaitCycles) return false;
    }
}
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
// The first N (4, 8 or 16) columns of this thread's lane.
template <int N>
__device__ __forceinline__ void tc_load(float (&v)[N], unsigned taddr)
{
    static_assert(N == 4 || N == 8 || N == 16, "column counts of the loads used here");
    unsigned r[N];
    if constexpr (N == 16) {
        float all[16];
        tc_load16(all, taddr);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = all[i];
        return;
    } else if constexpr (N == 8) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr) : "memory");
    } else {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
    }
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = __uint_as_float(r[i]);
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
// One lane of a converged warp (the MMA warps run converged so that descriptors and addresses
// stay warp-uniform values; only the issue itself is predicated).
__device__ __forceinline__ bool elect_one()
{
    unsigned chosen;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(chosen));
    return chosen != 0;
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

// Reduces 16 per-lane values over the warp (maximum or sum) in 16 shuffles: each step halves the
// number of values a lane carries and exchanges the other half with the lane `offset` away.
// Lane L ends up with the result for row warp_reduce16_row(L) (lanes L and L ^ 1 hold the same).
template <bool kMax>
__device__ __forceinline__ float warp_reduce16(const float (&v)[16], int lane)
{
    auto both = [](float x, float y) { return kMax ? fmaxf(x, y) : x + y; };
    float a8[8], a4[4], a2[2];
    const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0, up4 = (lane & 4) != 0, up2 = (lane & 2) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        a8[i] = both(up16 ? v[i + 8] : v[i], __shfl_xor_sync(0xffffffffu, up16 ? v[i] : v[i + 8], 16));
#pragma unroll
    for (int i = 0; i < 4; ++i)
        a4[i] = both(up8 ? a8[i + 4] : a8[i], __shfl_xor_sync(0xffffffffu, up8 ? a8[i] : a8[i + 4], 8));
#pragma unroll
    for (int i = 0; i < 2; ++i)
        a2[i] = both(up4 ? a4[i + 2] : a4[i], __shfl_xor_sync(0xffffffffu, up4 ? a4[i] : a4[i + 2], 4));
    const float a1 = both(up2 ? a2[1] : a2[0], __shfl_xor_sync(0xffffffffu, up2 ? a2[0] : a2[1], 2));
    return both(a1, __shfl_xor_sync(0xffffffffu, a1, 1));
}
__device__ __forceinline__ int warp_reduce16_row(int lane) { return ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1); }

__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap *map, int x, int y, int z, int w,
                                            unsigned bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%2, %3, %4, %5}], [%6];"
                 :: "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}

// A chunk of the grid's work list: number w counts (order, pair) with the order (long chunks
// first) slowest, exactly the order in which one block per chunk would be scheduled.
struct UmmaChunk {
    int pair, split, b, hk, begin, end, n_tiles;
};
__device__ __forceinline__ UmmaChunk umma_chunk(const AttnParams &a, int w, int len)
{
    UmmaChunk c;
    const int order = w / a.pairs;
    c.pair = w - order * a.pairs;
    c.split = scheduled_chunk(a, order);
    c.b = c.pair / a.heads;
    c.hk = c.pair - c.b * a.heads;
    int size;
    chunk_range(a, c.split, c.begin, size);
    c.end = min(c.begin + size, len);
    c.n_tiles = c.end > c.begin ? (c.end - c.begin + kUmmaTile - 1) / kUmmaTile : 0;
    return c;
}

// Persistent: one block per SM; blocks draw chunks from a ticket counter (`ticket`, zeroed by
// the host before the launch) until the list is exhausted, and the producers stream tiles
// across chunk boundaries, so the copy pipeline never drains between chunks.
// R: the query rows per KV head the softmax warps work on (4, 8 or 16; p.rows <= R): the MMAs
// always take 16 rows, of which those from p.rows on are zeros, but logits, exponentials and
// weights of rows that do not exist are not computed.
template <int D, bool kPaged, int R>
__global__ void __launch_bounds__(kUmmaThreads, 1)
grouped_attn_umma_kernel(const GroupedParams p, unsigned *ticket, const __grid_constant__ CUtensorMap map_q,
                         const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v)
{
    using Geo = UmmaGeometry<D>;
    constexpr int kSlots = kUmmaSlots, kItems = Geo::kItems, kItemPanels = kUmmaItemPanels, kItemBytes = kUmmaItemBytes;
    constexpr int kQBytes = Geo::kQBytes, kAccs = Geo::kAccs;
    constexpr int kQPanelBytes = kGroupRows * 128;              // 16 query rows of 64 dims
    extern __shared__ unsigned char smem_raw[];
    const AttnParams &a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool final_writer = a.n_splits == 1;
    const int total = a.pairs * a.n_splits;
    allow_next_kernel();
    wait_for_previous_kernels();

    // Shared memory: K ring, V ring (1024-byte aligned: the 128-byte swizzle is a function of the
    // address), query rows, weights, misc.
    const unsigned raw = static_cast<unsigned>(__cvta_generic_to_shared(smem_raw));
    const unsigned ring = (raw + 1023u) & ~1023u;
    unsigned char *smem = smem_raw + (ring - raw);
    constexpr int kKOffset = 0;
    constexpr int kVOffset = kSlots * kItemBytes;
    constexpr int kQOffset = kVOffset + kSlots * kItemBytes;
    constexpr int kPOffset = kQOffset + kUmmaQBuffers * kQBytes;
    constexpr int kMiscOffset = kPOffset + kUmmaPBytes;
    const unsigned q_smem = ring + kQOffset;
    const unsigned p_smem = ring + kPOffset;
    const unsigned misc = ring + kMiscOffset;
    unsigned char *misc_ptr = smem + kMiscOffset;
    volatile unsigned *abort_word = reinterpret_cast<volatile unsigned *>(misc_ptr + kUmmaAbort);
    volatile int2 *work = reinterpret_cast<volatile int2 *>(misc_ptr + kUmmaWork);
    float *red = reinterpret_cast<float *>(misc_ptr + kUmmaRed);

    // ---- set-up ----
    if (warp == kUmmaWarpLogits) {             // tensor memory: one warp allocates and later frees
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(misc + kUmmaTmemPtr), "n"(Geo::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else if (warp == kUmmaWarpK) {
        if (lane == 0) {
#pragma unroll
            for (int s = 0; s < kSlots; ++s) {
                mbarrier_init(misc + kUmmaBarKFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarKEmpty + s * 8, 1);
                mbarrier_init(misc + kUmmaBarVFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarVEmpty + s * 8, 1);
            }
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                mbarrier_init(misc + kUmmaBarSFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarSFree + s * 8, 4);
                mbarrier_init(misc + kUmmaBarQFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarQEmpty + s * 8, 1);
                mbarrier_init(misc + kUmmaBarAccFree + s * 8, 4);
            }
#pragma unroll
            for (int s = 0; s < kUmmaQueue; ++s) {
                mbarrier_init(misc + kUmmaBarWorkFull + s * 8, 1);
                mbarrier_init(misc + kUmmaBarWorkEmpty + s * 8, 7);       // V producer, 2 MMA lanes, 4 softmax warps
            }
            mbarrier_init(misc + kUmmaBarPFull, 4);
            mbarrier_init(misc + kUmmaBarPvDone, 1);
            mbarrier_init_fence();
            *abort_word = 0u;
            asm volatile("prefetch.tensormap [%0];" :: "l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
            asm volatile("prefetch.tensormap [%0];" :: "l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
            asm volatile("prefetch.tensormap [%0];" :: "l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
        }
    } else if (warp < 4) {
        // The query buffers start as zeros: a chunk's copy overwrites rows < p.rows only, so the
        // padding rows of the 16-row operand stay zero for the whole launch.
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        for (int i = threadIdx.x; i < kUmmaQBuffers * kQBytes / 16; i += 128)
            *reinterpret_cast<uint4 *>(smem + kQOffset + i * 16) = zero;
        // so does the weight buffer: the columns of rows >= R are never written
        for (int i = threadIdx.x; i < kUmmaPBytes / 16; i += 128)
            *reinterpret_cast<uint4 *>(smem + kPOffset + i * 16) = zero;
        fence_async_proxy();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = *reinterpret_cast<volatile unsigned *>(misc_ptr + kUmmaTmemPtr);

    // What both producers do for one chunk: the chunk's tiles of one cache (K or V) into that
    // cache's ring, item `count` of this block going to slot count % kSlots; returns false if a
    // wait ran out.
    // A copy moves `T` rows: a whole block of 16, 32 or 64 tokens, or 128 rows of a larger block
    // (a multiple of 128 tokens: tiles start on multiples of 128 then and never straddle a block),
    // or of a contiguous cache.
    const int T = kPaged ? min(a.block_tokens, kUmmaTile) : kUmmaTile;
    auto stream_chunk = [&](const UmmaChunk &c, const CUtensorMap *map, int ring_offset, int bar_full,
                            int bar_empty, int &count) -> bool {
        const int64_t total_rows = a.kv_bytes / (2 * D);
        const int32_t *table_row = kPaged ? a.block_table + (int64_t)c.b * a.max_blocks_per_seq : nullptr;
        auto fetch_ids = [&](int j) -> int {            // lane i: physical block of the tile's i-th block
            if (!kPaged) return 0;
            const int tile_start = c.begin + j * kUmmaTile;
            const int nb = (min(c.end - tile_start, kUmmaTile) + T - 1) / T;
            const int idx = (tile_start + lane * T) / a.block_tokens;
            if (j >= c.n_tiles || lane >= nb || !bounds_ok(idx < a.max_blocks_per_seq, a.status)) return -1;
            return __ldg(table_row + idx);
        };
        int ids_next = fetch_ids(0);
        for (int j = 0; j < c.n_tiles; ++j) {
            const int tile_start = c.begin + j * kUmmaTile;
            const int nb = kPaged ? (min(c.end - tile_start, kUmmaTile) + T - 1) / T : 1;
            const int phys = ids_next;
            ids_next = fetch_ids(j + 1);
            bool good = lane < nb;
            int row0;
            if (kPaged) {
                const bool in_range = phys >= 0 && (int64_t)phys < a.num_phys_blocks;
                if (good && !in_range && a.status) atomicOr(a.status, kFlagBlockRange);
                // (< 2^31 rows: checked by the host)
                row0 = in_range ? (phys * a.heads + c.hk) * a.block_tokens + (tile_start + lane * T) % a.block_tokens : 0;
                good = good && in_range && bounds_ok((int64_t)row0 + T <= total_rows, a.status);
            } else {
                row0 = c.pair * a.s_max + tile_start;          // rows past the tensor's end read as zeros
            }
            const unsigned fetched = __popc(__ballot_sync(0xffffffffu, good));
#pragma unroll
            for (int item = 0; item < kItems; ++item, ++count) {
                const int slot = count % kSlots;
                if (count >= kSlots &&
                    !__all_sync(0xffffffffu, mbarrier_wait_bounded(misc + bar_empty + slot * 8, (count / kSlots - 1) & 1)))
                    return false;
                const int slot_offset = ring_offset + slot * kItemBytes + (kPaged ? lane * T * 128 : 0);
                const unsigned bar = misc + bar_full + slot * 8;
                if (kPaged && lane < nb && !good) {            // a block that cannot be read counts as zeros
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    for (int i = 0; i < T * 8; ++i) {
#pragma unroll
                        for (int panel = 0; panel < kItemPanels; ++panel)
                            *reinterpret_cast<uint4 *>(smem + slot_offset + panel * kUmmaPanelBytes + i * 16) = zero;
                    }
                    fence_async_proxy();
                }
                if (lane == 0) mbarrier_expect_bytes(bar, fetched * (unsigned)(T * 128 * kItemPanels));
                __syncwarp();
                if (good) {
#pragma unroll
                    for (int panel = 0; panel < kItemPanels; ++panel)
                        tma_load_2d(ring + slot_offset + panel * kUmmaPanelBytes, map, (item * kItemPanels + panel) * 64, row0, bar);
                }
            }
        }
        return true;
    };
    // copies in flight must land (or be given up, bounded) before shared memory is handed on
    auto drain = [&](int bar_full, int count) {
        for (int i = max(count - kSlots, 0); i < count; ++i)
            (void)mbarrier_poll_bounded(misc + bar_full + (i % kSlots) * 8, (i / kSlots) & 1);
    };

    if (warp == kUmmaWarpK) {
        // ================== K producer: also draws the tickets and announces the chunks ==================
        // Tickets are drawn two chunks ahead and lengths read one chunk ahead: the atomic and the
        // load are issued at the start of a chunk and their results first used at its end, so
        // their round trips through a busy memory system overlap with the chunk's copies.
        auto issue_draw = [&]() -> unsigned {           // lane 0's return value is the ticket
            unsigned w = 0;
            if (lane == 0) w = atomicAdd(ticket, 1u);
            return w;
        };
        auto ticket_of = [&](unsigned raw_ticket) -> int {     // chunk number (total: none left)
            raw_ticket = __shfl_sync(0xffffffffu, raw_ticket, 0);
            return raw_ticket < (unsigned)total ? (int)raw_ticket : total;
        };
        auto issue_length = [&](int w) -> int {         // raw length of the chunk's sequence
            int len = 0;
            if (w < total) {
                const int b = (w % a.pairs) / a.heads;
                asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(len) : "l"(a.seq_lens + b) : "memory");
            }
            return len;
        };
        auto checked_length = [&](int w, int len) -> int {    // out-of-range lengths make the slot inactive
            if (w >= total) return 0;
            if (len < 0 || len > a.max_seq_len) {
                const int order = w / a.pairs, pair = w - order * a.pairs;
                if (lane == 0 && order == 0 && pair % a.heads == 0 && a.status) atomicOr(a.status, kFlagSeqLenRange);
                return 0;
            }
            return len;
        };
        int w_now = ticket_of(issue_draw());
        int w_next = ticket_of(issue_draw());
        int len_now = checked_length(w_now, issue_length(w_now));
        int count = 0;                                  // K items issued so far (ring position)
        int k = 0;                                      // chunks announced so far
        bool fine = true;
        bool first = true;
        unsigned raw_after = 0;
        int raw_len_next = 0;
        while (fine) {
            if (!first) {                               // what was requested a chunk ago has arrived by now
                w_now = w_next;
                len_now = checked_length(w_now, raw_len_next);
                w_next = ticket_of(raw_after);
            }
            first = false;
            const int w = w_now, len = len_now;
            if (w >= total) break;
            raw_after = issue_draw();
            raw_len_next = issue_length(w_next);
            const UmmaChunk c = umma_chunk(a, w, len);
            if (c.n_tiles == 0) {
                if (final_writer) {                     // inactive sequence: zero output, lse = -inf
                    for (int i = lane; i < p.rows * D; i += 32) {
                        const int r = i / D, d = i - r * D;
                        const int64_t row = grouped_row_index(p, c.b, c.hk, r);
                        a.out[row * D + d] = __float2half_rn(0.f);
                        if (a.lse && d == 0) a.lse[row] = -INFINITY;
                    }
                }
                continue;
            }
            // announce the chunk to the other warps
            const int wq = k % kUmmaQueue;
            if (k >= kUmmaQueue)
                fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarWorkEmpty + wq * 8,
                                                                     (k / kUmmaQueue - 1) & 1));
            if (!fine) break;
            if (lane == 0) {
                work[wq].x = w;
                work[wq].y = len;
                mbarrier_arrive(misc + kUmmaBarWorkFull + wq * 8);
            }
            // its query rows: rows t * group + g of (sequence, KV head), 64 dims per panel
            const int qb = k & 1;
            if (k >= 2)
                fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarQEmpty + qb * 8, (k / 2 - 1) & 1));
            if (!fine) break;
            if (lane == 0) {
                const unsigned bar = misc + kUmmaBarQFull + qb * 8;
                mbarrier_expect_bytes(bar, (unsigned)(p.rows * D * 2));
#pragma unroll
                for (int panel = 0; panel < Geo::kPanels; ++panel)
                    tma_load_4d(q_smem + qb * kQBytes + panel * kQPanelBytes, &map_q, panel * 64, c.hk * p.group, 0, c.b, bar);
            }
            ++k;
            fine = stream_chunk(c, &map_k, kKOffset, kUmmaBarKFull, kUmmaBarKEmpty, count);
        }
        if (fine) {                                     // no chunk is left: tell the others
            const int wq = k % kUmmaQueue;
            if (k >= kUmmaQueue)
                fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarWorkEmpty + wq * 8,
                                                                     (k / kUmmaQueue - 1) & 1));
            if (fine && lane == 0) {
                work[wq].x = -1;
                work[wq].y = 0;
                mbarrier_arrive(misc + kUmmaBarWorkFull + wq * 8);
            }
        }
        if (!fine) {
            if (lane == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
            drain(kUmmaBarKFull, count);
        }
    } else if (warp == kUmmaWarpV) {
        // ================================ V producer ================================
        int count = 0;
        bool fine = true;
        for (int k = 0; fine; ++k) {
            const int wq = k % kUmmaQueue;
            fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarWorkFull + wq * 8, (k / kUmmaQueue) & 1));
            if (!fine) break;
            const int w = work[wq].x, len = work[wq].y;
            __syncwarp();
            if (lane == 0) mbarrier_arrive(misc + kUmmaBarWorkEmpty + wq * 8);
            if (w < 0) break;
            fine = stream_chunk(umma_chunk(a, w, len), &map_v, kVOffset, kUmmaBarVFull, kUmmaBarVEmpty, count);
        }
        if (!fine) {
            if (lane == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
            drain(kUmmaBarVFull, count);
        }
    } else if (warp == kUmmaWarpLogits) {
        // ================================ logit MMAs ================================
        // One lane issues S^T = K_tile Q^T for every tile of every chunk of this block, as far
        // ahead of the softmax warps as the two logit buffers allow.
        {
            constexpr unsigned idesc = umma_idesc(128, 16, 0, 0);          // K tile K-major, Q K-major
            bool fine = true;
            int g = 0;                                                      // tiles of all chunks so far
            for (int k = 0; fine; ++k) {
                const int wq = k % kUmmaQueue;
                fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarWorkFull + wq * 8, (k / kUmmaQueue) & 1));
                if (!fine) break;
                const int w = __shfl_sync(0xffffffffu, work[wq].x, 0), len = __shfl_sync(0xffffffffu, work[wq].y, 0);
                __syncwarp();
                if (elect_one()) mbarrier_arrive(misc + kUmmaBarWorkEmpty + wq * 8);
                if (w < 0) break;
                const int n_tiles = umma_chunk(a, w, len).n_tiles;
                fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarQFull + (k & 1) * 8, (k / 2) & 1));
                // K tile and query rows alike: rows of 128 bytes per 64-dim panel, 8-row groups 1024
                // bytes apart, 128-byte swizzle; a k-step of 16 dims is 32 bytes along the row
                const uint64_t q_desc = umma_desc(q_smem + (k & 1) * kQBytes, 16, 1024, 2);
                for (int j = 0; j < n_tiles && fine; ++j, ++g) {
                    if (g >= 2)
                        fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarSFree + (g & 1) * 8, ((g >> 1) - 1) & 1));
#pragma unroll
                    for (int item = 0; item < kItems; ++item) {
                        if (!fine) break;
                        const int n = g * kItems + item, slot = n % kSlots;
                        fine = __all_sync(0xffffffffu, mbarrier_wait_bounded(misc + kUmmaBarKFull + slot * 8, (n / kSlots) & 1));
                        if (!fine) break;
                        tc_fence_after();
                        const uint64_t k_desc = umma_desc(ring + kKOffset + slot * kItemBytes, 16, 1024, 2);
                        if (elect_one()) {
#pragma unroll
                            for (int ks = 0; ks < 4 * kItemPanels; ++ks)
                                tc_mma_f16(tmem + (g & 1) * 16, k_desc + (uint64_t)(((ks >> 2) * kUmmaPanelBytes + (ks & 3) * 32) >> 4),
                                           q_desc + (uint64_t)(((item * kItemPanels + (ks >> 2)) * kQPanelBytes + (ks & 3) * 32) >> 4),
                                           idesc, item > 0 || ks > 0);
                            tc_commit(misc + kUmmaBarKEmpty + slot * 8);
                            if (item + 1 == kItems) {
                                tc_commit(misc + kUmmaBarSFull + (g & 1) * 8);
                                // after the chunk's last logit MMA its query rows may be replaced
                                if (j + 1 == n_tiles) tc_commit(misc + kUmmaBarQEmpty + (k & 1) * 8);
                            }
                        }
                        __syncwarp();
                    }
                    if (!fine) break;
                }
            }
            if (!fine && lane == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
        }
        __syncwarp();
    } else if (warp == kUmmaWarpOutput) {
        // ================================ output MMAs ================================
        // One lane issues O^T += V_tile^T P^T for every tile, into the accumulator of the chunk's parity.
        {
            constexpr unsigned idesc = umma_idesc(128, 32, 1, 1);          // V tile MN-major, weights MN-major
            // Weights: 8-column blocks of [128 tokens][16 bytes], 2048 bytes apart; 8-token groups
            // 128 bytes apart; a k-step is 16 tokens = 256 bytes.
            const uint64_t p_desc = umma_desc(p_smem, 128, 2048, 0);
            bool fine = true;
            int g = 0;
            for (int k = 0; fine; ++k) {
                const int wq = k % kUmmaQueue;
                fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarWorkFull + wq * 8, (k / kUmmaQueue) & 1));
                if (!fine) break;
                const int w = __shfl_sync(0xffffffffu, work[wq].x, 0), len = __shfl_sync(0xffffffffu, work[wq].y, 0);
                __syncwarp();
                if (elect_one()) mbarrier_arrive(misc + kUmmaBarWorkEmpty + wq * 8);
                if (w < 0) break;
                const int n_tiles = umma_chunk(a, w, len).n_tiles;
                // the accumulator of this parity was last used two chunks ago: its epilogue must have read it
                if (k >= 2)
                    fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarAccFree + (k & 1) * 8, (k / 2 - 1) & 1));
                const unsigned acc = tmem + 32 + (k & 1) * (kAccs * 32);
                for (int j = 0; j < n_tiles && fine; ++j, ++g) {
                    fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarPFull, g & 1));
#pragma unroll
                    for (int item = 0; item < kItems; ++item) {
                        if (!fine) break;
                        const int n = g * kItems + item, slot = n % kSlots;
                        fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarVFull + slot * 8, (n / kSlots) & 1));
                        if (!fine) break;
                        tc_fence_after();
                        // V item read MN-major (M = 128 dims): its two 64-dim panels are kUmmaPanelBytes
                        // apart (leading offset), 8-token groups 1024 bytes apart; a k-step is 16 tokens
                        // = 2048 bytes
                        const uint64_t v_desc = umma_desc(ring + kVOffset + slot * kItemBytes, kUmmaPanelBytes, 1024, 2);
                        if (elect_one()) {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)
                                tc_mma_f16(acc + item * 32, v_desc + (uint64_t)((ks * 2048) >> 4), p_desc + (uint64_t)((ks * 256) >> 4),
                                           idesc, j > 0 || ks > 0);
                            tc_commit(misc + kUmmaBarVEmpty + slot * 8);
                            if (item + 1 == kItems) tc_commit(misc + kUmmaBarPvDone);
                        }
                        __syncwarp();
                    }
                    if (!fine) break;
                }
            }
            if (!fine && lane == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
        }
        __syncwarp();
    } else {
        // ================================ softmax and epilogue ================================
        const int t = threadIdx.x;                                 // token of the tile = lane of tensor memory
        const unsigned lane_base = tmem + ((unsigned)(warp * 32) << 16);
        float *saved_m = reinterpret_cast<float *>(misc_ptr + kUmmaSavedM);     // [2][16]
        float *saved_l = reinterpret_cast<float *>(misc_ptr + kUmmaSavedL);     // [2][4][16]
        // The epilogue of a chunk (accumulator -> partial result) runs after the first tile of the
        // next chunk has been handed to the MMA, so that the tensor pipe and the copies go on
        // meanwhile; the accumulators alternate between two regions of tensor memory.
        auto epilogue = [&](const UmmaChunk &c, int parity) {
            // Thread t owns output dims t, 128 + t, ... (one per accumulator); columns r and 16 + r
            // are the high and low parts of row r.
            // Sums and accumulator both carry kGroupWeightScale.
            tc_fence_after();
            const float *sl = saved_l + parity * 64, *sm = saved_m + parity * 16;
#pragma unroll
            for (int acc_i = 0; acc_i < kAccs; ++acc_i) {
                float o_hi[16], o_lo[16];
                tc_load16(o_hi, lane_base + 32 + (parity * kAccs + acc_i) * 32);
                tc_load16(o_lo, lane_base + 48 + (parity * kAccs + acc_i) * 32);
                const int d = acc_i * 128 + t;
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    if (r < p.rows) {
                        const float total_w = (sl[r] + sl[16 + r]) + (sl[32 + r] + sl[48 + r]);
                        // A row that sees no position of this chunk (causal limit before the chunk) has total 0.
                        const bool empty = !(total_w > 0.f);
                        const float value = empty ? 0.f : (o_hi[r] + o_lo[r]) / total_w;
                        const float lse2 = empty ? kMinusHuge : sm[r] + log2f(total_w) - kGroupWeightLog2;
                        if (final_writer) {
                            const int64_t row = grouped_row_index(p, c.b, c.hk, r);
                            a.out[row * D + d] = __float2half_rn(value);
                            if (a.lse && d == 0) a.lse[row] = empty ? -INFINITY : lse2 * kLn2;
                        } else {
                            const int64_t slot = ((int64_t)c.pair * a.n_splits + c.split) * p.rows + r;
                            a.part_o[slot * D + d] = value;
                            if (d == 0) a.part_lse[slot] = lse2;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbarrier_arrive(misc + kUmmaBarAccFree + parity * 8);
        };
        bool aborted = false, pending = false;
        UmmaChunk before = {};                                      // the chunk whose epilogue is pending
        int g = 0;                                                  // tiles of all chunks so far
        int k = 0;
        for (; !aborted; ++k) {
            const int wq = k % kUmmaQueue;
            bool fine = mbarrier_poll_bounded(misc + kUmmaBarWorkFull + wq * 8, (k / kUmmaQueue) & 1);
            if (softmax_any(!fine)) {                               // one decision for the four warps
                aborted = true;
                break;
            }
            const int w = work[wq].x, len = work[wq].y;
            __syncwarp();
            if (lane == 0) mbarrier_arrive(misc + kUmmaBarWorkEmpty + wq * 8);
            if (w < 0) break;
            const UmmaChunk c = umma_chunk(a, w, len);
            const int n_tiles = c.n_tiles;
            const unsigned acc = lane_base + 32 + (k & 1) * (kAccs * 32);     // this chunk's accumulator(s)
            float m[R], l[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                m[r] = kMinusHuge;
                l[r] = 0.f;
            }
            const int unmasked_end = min(c.end, len - (p.q_tokens - 1));   // tiles ending here or before need no mask
            for (int j = 0; j < n_tiles; ++j, ++g) {
                const int sb = g & 1;
                // (warp-uniform: the tensor-memory loads below are warp-wide instructions)
                if (fine) fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarSFull + sb * 8, (g >> 1) & 1));
                float s[R];
                if (fine) {
                    tc_fence_after();
                    tc_load<R>(s, lane_base + sb * 16);
                    tc_fence_before();
                } else {
#pragma unroll
                    for (int r = 0; r < R; ++r) s[r] = 0.f;
                }
                __syncwarp();
                if (lane == 0) mbarrier_arrive(misc + kUmmaBarSFree + sb * 8);
                const int tile_start = c.begin + j * kUmmaTile;
                const int tok = tile_start + t;
#pragma unroll
                for (int r = 0; r < R; ++r) s[r] *= a.scale_log2e;
                if (tile_start + kUmmaTile > unmasked_end) {       // uniform: last tiles of the sequence / chunk
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const int vis = r < p.rows ? len - (p.q_tokens - 1 - r / p.group) : 0;
                        if (tok >= min(vis, c.end)) s[r] = -INFINITY;
                    }
                    if (tok >= c.end && fine) {
                        // The value row of a position outside the chunk gets weight zero, but its bytes
                        // may be anything (the tail of a block, a slot not fetched): 0 x NaN must not
                        // reach the accumulator, so the row is cleared once the tile has landed.
                        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                        for (int item = 0; item < kItems; ++item) {
                            const int n = g * kItems + item, slot = n % kSlots;
                            if (fine) fine = mbarrier_poll_bounded(misc + kUmmaBarVFull + slot * 8, (n / kSlots) & 1);
                            unsigned char *vrow = smem + kVOffset + slot * kItemBytes + t * 128;
#pragma unroll
                            for (int panel = 0; panel < kItemPanels; ++panel) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) *reinterpret_cast<uint4 *>(vrow + panel * kUmmaPanelBytes + i * 16) = zero;
                            }
                        }
                    }
                }
                bool moved = false;
#pragma unroll
                for (int r = 0; r < R; ++r) moved = moved || s[r] > m[r] + kGroupLag;
                if (!fine) *abort_word = 1u;
                bool waited = false;
                if (softmax_any(moved || !fine)) {
                    if (*abort_word != 0u) {                        // the same for all 128 threads
                        aborted = true;
                        break;
                    }
                    // Some row's reference moves: row maxima over the tile, new references, and the
                    // accumulator (and the sums) rescaled to them.
                    float tops[16];
#pragma unroll
                    for (int r = 0; r < 16; ++r) tops[r] = r < R ? s[r % R] : kMinusHuge;
                    const float top_mine = warp_reduce16<true>(tops, lane);
                    if ((lane & 1) == 0) red[warp * 16 + warp_reduce16_row(lane)] = top_mine;
                    softmax_sync();
                    float alpha[16];
                    bool any_change = false;
#pragma unroll
                    for (int r = 0; r < 16; ++r) alpha[r] = 1.f;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const float top = fmaxf(fmaxf(red[r], red[16 + r]), fmaxf(red[32 + r], red[48 + r]));
                        if (top > m[r] + kGroupLag) {
                            alpha[r] = fast_exp2(m[r] - top);
                            m[r] = top;
                            any_change = true;
                        }
                        l[r] *= alpha[r];
                    }
                    if (j > 0 && any_change) {
                        // the accumulator holds tiles 0 .. j-1 once the previous tile's MMA is complete
                        fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarPvDone, (g - 1) & 1));
                        waited = true;
                        if (fine) {
                            tc_fence_after();
                            float o[16];
#pragma unroll
                            for (int half = 0; half < 2 * kAccs; ++half) {  // per accumulator, columns 0-15: high parts, 16-31: low parts
                                tc_load16(o, acc + half * 16);
#pragma unroll
                                for (int r = 0; r < 16; ++r) o[r] *= alpha[r];
                                tc_store16(acc + half * 16, o);
                            }
                        } else {
                            *abort_word = 1u;                       // seen by all at the next vote
                        }
                    }
                }
                // Weights against the references (scaled by kGroupWeightScale inside the exponent),
                // their sums, and the fp16 high and low parts: thread t holds row t of operand B
                // (MN-major: 8 columns = 16 bytes per token and column block).
                unsigned hi[8], lo[8];
#pragma unroll
                for (int i = R / 2; i < 8; ++i) hi[i] = lo[i] = 0u;
#pragma unroll
                for (int i = 0; i < R / 2; ++i) {
                    const float w0 = fast_exp2(s[2 * i] - (m[2 * i] - kGroupWeightLog2));
                    const float w1 = fast_exp2(s[2 * i + 1] - (m[2 * i + 1] - kGroupWeightLog2));
                    l[2 * i] += w0;
                    l[2 * i + 1] += w1;
                    hi[i] = pack_half2(w0, w1);
                    const float2 back = __half22float2(*reinterpret_cast<const __half2 *>(&hi[i]));
                    lo[i] = pack_half2(w0 - back.x, w1 - back.y);
                }
                if (g > 0 && !waited && fine) {                     // the previous MMA has read the weights
                    fine = mbarrier_poll_bounded(misc + kUmmaBarPvDone, (g - 1) & 1);
                    if (!fine) *abort_word = 1u;
                }
                unsigned char *prow = smem + kPOffset + t * 16;
                *reinterpret_cast<uint4 *>(prow) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4 *>(prow + 4096) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                if (R > 8) {                                        // rows 8-15: the second column block of each part
                    *reinterpret_cast<uint4 *>(prow + 2048) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
                    *reinterpret_cast<uint4 *>(prow + 6144) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
                }
                fence_async_proxy();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbarrier_arrive(misc + kUmmaBarPFull);
                if (j == 0 && pending) {
                    // The previous chunk's last MMA is complete (this thread waited for it before
                    // writing this tile's weights) and its sums were stored before this tile's vote.
                    if (__all_sync(0xffffffffu, fine)) epilogue(before, (k - 1) & 1);
                    pending = false;
                }
            }
            if (aborted) break;
            // the chunk's references and row sums, for its epilogue
            float sums[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) sums[r] = r < R ? l[r % R] : 0.f;
            const float sum_mine = warp_reduce16<false>(sums, lane);
            if ((lane & 1) == 0) saved_l[(k & 1) * 64 + warp * 16 + warp_reduce16_row(lane)] = sum_mine;
            if (t < R) {
                float mine = m[0];
#pragma unroll
                for (int r = 1; r < R; ++r) mine = t == r ? m[r] : mine;
                saved_m[(k & 1) * 16 + t] = mine;
            }
            before = c;
            pending = true;
            if (!fine) *abort_word = 1u;
        }
        if (!aborted && pending) {
            // the last chunk: its last MMA has not been waited for yet
            const bool fine = __all_sync(0xffffffffu, mbarrier_poll_bounded(misc + kUmmaBarPvDone, (g - 1) & 1));
            if (!softmax_any(!fine || *abort_word != 0u)) epilogue(before, (k - 1) & 1);
            else aborted = true;
        }
        if (aborted && t == 0 && a.status) atomicOr(a.status, kFlagCopyTimeout);
    }

    // ---- teardown: everyone is done with tensor memory before it is released ----
    tc_fence_before();
    __syncthreads();
    if (warp == kUmmaWarpLogits) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "n"(Geo::kTmemCols) : "memory");
    }
}

}  // namespace instinfer
