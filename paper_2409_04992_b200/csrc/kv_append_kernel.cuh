// KV append for sm_100a: the new token's k,v rows join the cache (Sec. II-B; the decode
// phase's incremental writes of Sec. IV-C).  A pure bit copy: one thread moves one 16-byte
// segment of K and one of V; head_dim / 8 threads cover a (sequence, head) row pair.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "decode_attention_kernels.cuh"

namespace instinfer {

struct AppendParams {
    uint4 *k_cache;
    uint4 *v_cache;
    const uint4 *k_new;           // [batch, heads, head_dim] fp16 = segs_per_row uint4 per row
    const uint4 *v_new;
    const int32_t *seq_lens;
    const int32_t *block_table;   // nullptr: contiguous
    int32_t *status;              // nullable
    int64_t num_phys_blocks;
    int32_t batch;
    int32_t heads;
    int32_t s_max;
    int32_t block_tokens;
    int32_t max_blocks_per_seq;
    int32_t segs_per_row;         // 16-byte segments of one row: head_dim / 8 (16 at head_dim 128)
    int64_t cache_rows;           // rows of the K cache (= of the V cache) that the call's shapes imply
};

constexpr int kAppendThreads = 128;

__global__ void __launch_bounds__(kAppendThreads)
kv_append_kernel(const AppendParams p)
{
    const int64_t idx = (int64_t)blockIdx.x * kAppendThreads + threadIdx.x;
    const int64_t pair = idx / p.segs_per_row;
    if (pair >= (int64_t)p.batch * p.heads) return;
    const int seg = (int)(idx % p.segs_per_row);
    const int b = (int)(pair / p.heads), h = (int)(pair % p.heads);
    const bool reporter = seg == 0 && h == 0 && p.status != nullptr;
    asm volatile("griddepcontrol.launch_dependents;");      // the next kernel may start being scheduled
    asm volatile("griddepcontrol.wait;" ::: "memory");      // earlier kernels' writes are visible from here

    const int len = p.seq_lens[b];
    if (len == 0) return;                                   // inactive slot
    const int64_t capacity = p.block_table ? (int64_t)p.max_blocks_per_seq * p.block_tokens
                                           : (int64_t)p.s_max;
    if (len < 0 || len > capacity) {
        if (reporter) atomicOr(p.status, 1);                // seq_len out of range
        return;
    }
    const int pos = len - 1;
    int64_t row;
    if (p.block_table) {
        const int phys = p.block_table[(int64_t)b * p.max_blocks_per_seq + pos / p.block_tokens];
        if (phys < 0 || (int64_t)phys >= p.num_phys_blocks) {
            if (reporter) atomicOr(p.status, 2);            // block id out of range
            return;
        }
        row = ((int64_t)phys * p.heads + h) * p.block_tokens + pos % p.block_tokens;
    } else {
        row = pair * p.s_max + pos;
    }
    if (!bounds_ok(row >= 0 && row < p.cache_rows, p.status)) return;
    p.k_cache[row * p.segs_per_row + seg] = p.k_new[idx];
    p.v_cache[row * p.segs_per_row + seg] = p.v_new[idx];
}

// Bulk append (prefill, Sec. IV-D): new_lens[b] tokens per sequence from token-major
// k_new / v_new [batch, max_new, heads, head_dim] into positions seq_lens[b]-new_lens[b] ... of
// the cache.  A thread moves one 16-byte segment of kBulkTokens consecutive tokens of one head,
// K and V: its 2 * kBulkTokens loads are issued before the first store, so that a pure copy
// keeps enough bytes in flight; reads of a warp are contiguous 512-byte runs, each written row
// is a contiguous run of head_dim * 2 bytes.
struct BulkAppendParams {
    AppendParams base;            // k_new / v_new point at [batch, max_new, heads, head_dim]
    const int32_t *new_lens;
    int32_t max_new;
};

constexpr int kBulkTokens = 4;

__global__ void __launch_bounds__(kAppendThreads)
kv_append_bulk_kernel(const BulkAppendParams q)
{
    const AppendParams &p = q.base;
    const int64_t idx = (int64_t)blockIdx.x * kAppendThreads + threadIdx.x;
    const int row_segs = p.heads * p.segs_per_row;               // 16-byte segments of one token
    const int groups = (q.max_new + kBulkTokens - 1) / kBulkTokens;
    const int64_t item = idx / row_segs;                         // (b, group of tokens)
    if (item >= (int64_t)p.batch * groups) return;
    const int in_row = (int)(idx - item * row_segs);             // (h, seg)
    const int h = in_row / p.segs_per_row, seg = in_row - h * p.segs_per_row;
    const int b = (int)(item / groups), t0 = (int)(item - (int64_t)b * groups) * kBulkTokens;
    const bool reporter = in_row == 0 && t0 == 0 && p.status != nullptr;

    const int len = p.seq_lens[b], fresh = q.new_lens[b];
    const int64_t capacity = p.block_table ? (int64_t)p.max_blocks_per_seq * p.block_tokens
                                           : (int64_t)p.s_max;
    if (len < 0 || len > capacity || fresh < 0 || fresh > q.max_new || fresh > len) {
        if (reporter) atomicOr(p.status, 1);                // lengths out of range: sequence skipped
        return;
    }
    const int64_t src = ((int64_t)b * q.max_new + t0) * row_segs + in_row;
    uint4 k[kBulkTokens], v[kBulkTokens];
#pragma unroll
    for (int u = 0; u < kBulkTokens; ++u) {
        if (t0 + u < fresh) {
            k[u] = p.k_new[src + (int64_t)u * row_segs];
            v[u] = p.v_new[src + (int64_t)u * row_segs];
        }
    }
#pragma unroll
    for (int u = 0; u < kBulkTokens; ++u) {
        if (t0 + u >= fresh) break;
        const int pos = len - fresh + t0 + u;
        int64_t dst;
        if (p.block_table) {
            const int phys = p.block_table[(int64_t)b * p.max_blocks_per_seq + pos / p.block_tokens];
            if (phys < 0 || (int64_t)phys >= p.num_phys_blocks) {
                if (in_row == 0 && p.status) atomicOr(p.status, 2);
                continue;                                    // rows of a bad block are skipped
            }
            dst = ((int64_t)phys * p.heads + h) * p.block_tokens + pos % p.block_tokens;
        } else {
            dst = ((int64_t)b * p.heads + h) * p.s_max + pos;
        }
        if (!bounds_ok(dst >= 0 && dst < p.cache_rows, p.status)) continue;
        p.k_cache[dst * p.segs_per_row + seg] = k[u];
        p.v_cache[dst * p.segs_per_row + seg] = v[u];
    }
}

}  // namespace instinfer
