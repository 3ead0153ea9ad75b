// Last kernel of the head-sharded path: the log-sum-exp merge of one (sequence, head) with
// the all-gather of the outputs fused in.  Every rank keeps a full [batch, total_heads, 128]
// output buffer; the block that finishes a local head stores its 256-byte row into all of
// them (its own and the peers', mapped into this GPU's address space) with 16-byte stores.
// No block waits for another GPU.
#pragma once

#include "decode_attention_kernels.cuh"

namespace instinfer {

constexpr int kMaxRanks = 16;
constexpr int kRowSegments = kHeadDim * 2 / 16;      // 16-byte pieces of one fp16 output row

struct GatherTargets {
    __half *out[kMaxRanks];      // rank r's [batch, total_heads, kHeadDim] buffer
    const __half *staged;        // [pairs, kHeadDim] finished rows when the plan has one chunk
    int32_t n_ranks;
    int32_t head_offset;         // global index of this shard's head 0
    int32_t total_heads;
};

// One block per local (sequence, head), one thread per output dim.  With a single chunk the
// split kernel has already produced the final row (in t.staged) and only the fan-out is left.
__global__ void __launch_bounds__(kHeadDim)
lse_merge_allgather_kernel(const AttnParams p, const GatherTargets t)
{
    __shared__ __align__(16) __half row[kHeadDim];
    const int pair = blockIdx.x;
    const int b = pair / p.heads, h = pair - b * p.heads;
    allow_next_kernel();
    wait_for_previous_kernels();
    if (p.n_splits == 1) {
        row[threadIdx.x] = t.staged[(int64_t)pair * kHeadDim + threadIdx.x];
    } else {
        const int len = checked_seq_len(p, b, threadIdx.x == 0 && h == 0);
        const int live = live_chunks(p, len);
        if (live == 0) {
            row[threadIdx.x] = __float2half_rn(0.f);
            if (p.lse && threadIdx.x == 0) p.lse[pair] = -INFINITY;
        } else {
            const float *lse2 = p.part_lse + (int64_t)pair * p.n_splits;
            const float *po = p.part_o + (int64_t)pair * p.n_splits * kHeadDim + threadIdx.x;
            float top = kMinusHuge;
            for (int s = 0; s < live; ++s) top = fmaxf(top, lse2[s]);
            float total = 0.f, o = 0.f;
            for (int s = 0; s < live; ++s) {
                const float w = fast_exp2(lse2[s] - top);
                total += w;
                o = fmaf(w, po[(int64_t)s * kHeadDim], o);
            }
            row[threadIdx.x] = __float2half_rn(o / total);
            if (p.lse && threadIdx.x == 0) p.lse[pair] = (top + log2f(total)) * kLn2;
        }
    }
    __syncthreads();
    const int64_t dst_row = ((int64_t)b * t.total_heads + t.head_offset + h) * kHeadDim;
    for (int i = threadIdx.x; i < t.n_ranks * kRowSegments; i += kHeadDim) {
        const int rank = i / kRowSegments, seg = i - rank * kRowSegments;
        reinterpret_cast<uint4 *>(t.out[rank] + dst_row)[seg] = reinterpret_cast<const uint4 *>(row)[seg];
    }
}

}  // namespace instinfer
