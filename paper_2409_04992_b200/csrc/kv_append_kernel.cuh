// KV append for sm_100a: the new token's k,v rows join the cache (Sec. II-B; the decode
// phase's incremental writes of Sec. IV-C).  A pure bit copy: one thread moves one 16-byte
// segment of K and one of V; head_dim / 8 threads cover a (sequence, head) row pair.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

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
    p.k_cache[row * p.segs_per_row + seg] = p.k_new[idx];
    p.v_cache[row * p.segs_per_row + seg] = p.v_new[idx];
}

// Bulk append (prefill, Sec. IV-D): new_lens[b] tokens per sequence from token-major
// k_new / v_new [batch, max_new, heads, 128] into positions seq_lens[b]-new_lens[b] ... of the
// cache.  One thread per 16-byte segment; reads are fully contiguous, each written row is a
// contiguous 256 bytes.
struct BulkAppendParams {
    AppendParams base;            // k_new / v_new point at [batch, max_new, heads, 128]
    const int32_t *new_lens;
    int32_t max_new;
};

__global__ void __launch_bounds__(kAppendThreads)
kv_append_bulk_kernel(const BulkAppendParams q)
{
    const AppendParams &p = q.base;
    const int64_t idx = (int64_t)blockIdx.x * kAppendThreads + threadIdx.x;
    const int64_t row = idx / p.segs_per_row;                    // (b, t, h)
    if (row >= (int64_t)p.batch * q.max_new * p.heads) return;
    const int seg = (int)(idx % p.segs_per_row);
    const int h = (int)(row % p.heads);
    const int64_t bt = row / p.heads;
    const int t = (int)(bt % q.max_new), b = (int)(bt / q.max_new);
    const bool reporter = seg == 0 && h == 0 && t == 0 && p.status != nullptr;

    const int len = p.seq_lens[b], fresh = q.new_lens[b];
    const int64_t capacity = p.block_table ? (int64_t)p.max_blocks_per_seq * p.block_tokens
                                           : (int64_t)p.s_max;
    if (len < 0 || len > capacity || fresh < 0 || fresh > q.max_new || fresh > len) {
        if (reporter) atomicOr(p.status, 1);                // lengths out of range: sequence skipped
        return;
    }
    if (t >= fresh) return;
    const int pos = len - fresh + t;
    int64_t dst;
    if (p.block_table) {
        const int phys = p.block_table[(int64_t)b * p.max_blocks_per_seq + pos / p.block_tokens];
        if (phys < 0 || (int64_t)phys >= p.num_phys_blocks) {
            if (seg == 0 && h == 0 && p.status) atomicOr(p.status, 2);
            return;
        }
        dst = ((int64_t)phys * p.heads + h) * p.block_tokens + pos % p.block_tokens;
    } else {
        dst = ((int64_t)b * p.heads + h) * p.s_max + pos;
    }
    p.k_cache[dst * p.segs_per_row + seg] = p.k_new[idx];
    p.v_cache[dst * p.segs_per_row + seg] = p.v_new[idx];
}

}  // namespace instinfer
