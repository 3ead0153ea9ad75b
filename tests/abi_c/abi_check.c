/*
 * abi_check.c -- a plain C99 caller of libinstinfer.so that uses nothing but the public
 * header.  It exists to catch drift between include/instinfer.h and the Python binding's
 * hand-written argument types: it takes every entry point down an argument-rejection path
 * (nothing is ever enqueued, so it runs without a GPU; the test runs it with no device
 * visible) and prints the planner / workspace figures for the test to compare with what the
 * binding returns for the same sizes.  Every pointer below is a made-up aligned address that
 * a correct library never dereferences on these paths.
 */
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "instinfer.h"

static int failures = 0;

static void expect(const char *what, int got, int want)
{
    if (got != want) {
        printf("FAIL %s: got %d (%s), want %d\n", what, got, instinfer_status_string(got), want);
        ++failures;
    }
}

int main(void)
{
    void *const fake = (void *)(uintptr_t)0x10000;
    void *const odd = (void *)(uintptr_t)0x10008;          /* not 16-byte aligned */
    const int32_t *const lens = (const int32_t *)fake;
    const int32_t *const table = (const int32_t *)fake;
    const size_t big = (size_t)1 << 30;
    void *outs[1];
    outs[0] = fake;

    /* append: a distinct value in every integer slot, so a swapped pair shows */
    expect("append null cache", instinfer_kv_append(NULL, fake, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 128, 64, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("append head_dim", instinfer_kv_append(fake, fake, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 96, 64, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("append block_tokens", instinfer_kv_append(fake, fake, fake, fake, lens, table, 4, 20, 9, 2, 4, 128, 0, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("append num_phys_blocks", instinfer_kv_append(fake, fake, fake, fake, lens, table, 4, 16, 0, 2, 4, 128, 0, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("append empty", instinfer_kv_append(NULL, NULL, NULL, NULL, NULL, NULL, 0, 0, 0, 0, 4, 128, 64, NULL, NULL),
           INSTINFER_OK);
    expect("bulk append max_new", instinfer_kv_append_bulk(fake, fake, fake, fake, lens, lens, NULL, 0, 0, 0, 2, -1, 4, 128, 64, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("bulk append new_lens", instinfer_kv_append_bulk(fake, fake, fake, fake, lens, NULL, NULL, 0, 0, 0, 2, 3, 4, 128, 64, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("bulk append nothing new", instinfer_kv_append_bulk(fake, fake, fake, fake, lens, lens, NULL, 0, 0, 0, 2, 0, 4, 128, 64, NULL, NULL),
           INSTINFER_OK);

    /* contiguous attention */
    expect("attention misaligned q", instinfer_decode_attention(fake, NULL, odd, fake, fake, lens, 2, 4, 128, 256, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("attention max_seq_len > s_max", instinfer_decode_attention(fake, NULL, fake, fake, fake, lens, 2, 4, 128, 256, 257, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("attention head_dim", instinfer_decode_attention(fake, NULL, fake, fake, fake, lens, 2, 4, 64, 256, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("attention scale", instinfer_decode_attention(fake, NULL, fake, fake, fake, lens, 2, 4, 128, 256, 256, (float)NAN, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("attention workspace size", instinfer_decode_attention(fake, NULL, fake, fake, fake, lens, 2, 4, 128, 256, 256, 0.1f, fake, 16, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);
    expect("attention empty", instinfer_decode_attention(NULL, NULL, NULL, NULL, NULL, NULL, 0, 4, 128, 256, 256, 0.1f, NULL, 0, NULL, NULL),
           INSTINFER_OK);

    /* paged attention: max_seq_len against max_blocks_per_seq * block_tokens */
    expect("paged table", instinfer_decode_attention_paged(fake, NULL, fake, fake, fake, NULL, lens, 2, 4, 128, 16, 16, 40, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("paged capacity", instinfer_decode_attention_paged(fake, NULL, fake, fake, fake, table, lens, 2, 4, 128, 16, 16, 40, 257, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("paged block_tokens", instinfer_decode_attention_paged(fake, NULL, fake, fake, fake, table, lens, 2, 4, 128, 12, 32, 40, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("paged num_phys_blocks", instinfer_decode_attention_paged(fake, NULL, fake, fake, fake, table, lens, 2, 4, 128, 16, 16, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("paged workspace", instinfer_decode_attention_paged(fake, NULL, fake, fake, fake, table, lens, 2, 4, 128, 16, 16, 40, 256, 0.1f, fake, 0, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);

    /* built-in scratch: a plan whose partials exceed the 16 MiB array is refused on the host */
    expect("static chunk override", instinfer_set_chunk_tokens(64), INSTINFER_OK);
    expect("static too large", instinfer_decode_attention_static(fake, NULL, fake, fake, fake, NULL, lens, 64, 40, 128, 131072, 0, 0, 0, 131072, 0.1f, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);
    expect("static chunk override off", instinfer_set_chunk_tokens(0), INSTINFER_OK);
    expect("static head_dim", instinfer_decode_attention_static(fake, NULL, fake, fake, fake, NULL, lens, 0, 4, 64, 256, 0, 0, 0, 256, 0.1f, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);

    /* head-sharded */
    expect("allgather n_ranks", instinfer_decode_attention_allgather(outs, 0, NULL, fake, fake, fake, NULL, lens, 2, 4, 0, 8, 128, 256, 0, 0, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("allgather head range", instinfer_decode_attention_allgather(outs, 1, NULL, fake, fake, fake, NULL, lens, 2, 4, 5, 8, 128, 256, 0, 0, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("allgather workspace", instinfer_decode_attention_allgather(outs, 1, NULL, fake, fake, fake, NULL, lens, 2, 4, 4, 8, 128, 256, 0, 0, 0, 256, 0.1f, fake,
                                                                       instinfer_workspace_bytes(2, 4, 128, 256), NULL, NULL),
           INSTINFER_ERR_WORKSPACE);

    /* grouped heads / several tokens */
    expect("grouped head ratio", instinfer_decode_attention_grouped(fake, NULL, fake, fake, fake, NULL, lens, 2, 1, 7, 2, 128, 256, 0, 0, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("grouped rows", instinfer_decode_attention_grouped(fake, NULL, fake, fake, fake, NULL, lens, 2, 9, 8, 2, 128, 256, 0, 0, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("grouped head_dim", instinfer_decode_attention_grouped(fake, NULL, fake, fake, fake, NULL, lens, 2, 1, 8, 2, 96, 256, 0, 0, 0, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("grouped paged capacity", instinfer_decode_attention_grouped(fake, NULL, fake, fake, fake, table, lens, 2, 1, 8, 2, 128, 0, 16, 4, 9, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("grouped workspace", instinfer_decode_attention_grouped(fake, NULL, fake, fake, fake, NULL, lens, 2, 1, 8, 2, 128, 256, 0, 0, 0, 256, 0.1f, fake, 64, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);

    /* host-buffer step */
    expect("host step null host buffer", instinfer_decode_step_host(NULL, fake, fake, fake, NULL, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 128, 256, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("host step head_dim", instinfer_decode_step_host(fake, fake, fake, fake, NULL, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 64, 256, 256, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("host step workspace", instinfer_decode_step_host(fake, fake, fake, fake, NULL, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 128, 256, 256, 0.1f, fake, 16, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);
    expect("overlapped host step without its upload event", instinfer_decode_step_host_overlapped(fake, fake, fake, fake, NULL, fake, fake, lens, NULL, 0, 0, 0, 2, 4, 128, 256, 256, 0.1f, fake, big, NULL, NULL, fake, NULL, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);

    /* sparse path */
    expect("sparse append kt table", instinfer_sparf_append(fake, fake, fake, (float *)fake, fake, fake, lens, table, 16, 16, 40, NULL, 2, 128, 9, 2, 4, 128, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("sparse append head_dim", instinfer_sparf_append(fake, fake, fake, (float *)fake, fake, fake, lens, table, 16, 16, 40, table, 2, 128, 9, 2, 4, 64, NULL, NULL),
           INSTINFER_ERR_UNSUPPORTED);
    expect("sparse bulk append max_new", instinfer_sparf_append_bulk(fake, fake, fake, (float *)fake, fake, fake, lens, lens, table, 16, 16, 40, table, 2, 128, 9, 2, -1, 4, 128, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("sparse attention r", instinfer_sparf_decode_attention(fake, NULL, NULL, fake, fake, fake, fake, (const float *)fake, table, lens, lens, 2, 4, 128, 16, 16, 40,
                                                                  table, 2, 128, 9, 256, 32, 129, 4, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("sparse attention max_k", instinfer_sparf_decode_attention(fake, NULL, NULL, fake, fake, fake, fake, (const float *)fake, table, lens, lens, 2, 4, 128, 16, 16, 40,
                                                                      table, 2, 128, 9, 256, 257, 16, 4, 0.1f, fake, big, NULL, NULL),
           INSTINFER_ERR_INVALID_ARG);
    expect("sparse attention workspace", instinfer_sparf_decode_attention(fake, NULL, NULL, fake, fake, fake, fake, (const float *)fake, table, lens, lens, 2, 4, 128, 16, 16, 40,
                                                                          table, 2, 128, 9, 256, 32, 16, 4, 0.1f, fake, 64, NULL, NULL),
           INSTINFER_ERR_WORKSPACE);

    /* knobs */
    expect("chunk override granule", instinfer_set_chunk_tokens(100), INSTINFER_ERR_INVALID_ARG);
    expect("sparse path range", instinfer_set_sparse_path(3), INSTINFER_ERR_INVALID_ARG);
    expect("grouped path range", instinfer_set_grouped_path(3), INSTINFER_ERR_INVALID_ARG);
    expect("grouped path automatic", instinfer_set_grouped_path(0), INSTINFER_OK);
    expect("grouped path of a refused head size", instinfer_grouped_path_for(96, 16), 0);
    expect("timing events one null", instinfer_set_timing_events(fake, NULL), INSTINFER_ERR_INVALID_ARG);
    expect("timing events off", instinfer_set_timing_events(NULL, NULL), INSTINFER_OK);
    if (strcmp(instinfer_status_string(INSTINFER_OK), "ok") != 0) {
        printf("FAIL status string\n");
        ++failures;
    }

    /* figures the test compares with the binding's */
    printf("workspace %zu\n", instinfer_workspace_bytes(16, 40, 128, 8192));
    printf("workspace_bad_dim %zu\n", instinfer_workspace_bytes(16, 40, 64, 8192));
    printf("allgather_workspace %zu\n", instinfer_allgather_workspace_bytes(16, 5, 128, 8192));
    printf("grouped_workspace %zu\n", instinfer_grouped_workspace_bytes(4, 2, 32, 8, 128, 16384));
    printf("sparf_workspace %zu\n", instinfer_sparf_workspace_bytes(8, 40, 128, 131072, 16384));
    printf("plan_chunk %d\n", (int)instinfer_plan_chunk_tokens(16, 40, 8192));
    printf("plan_splits %d\n", (int)instinfer_plan_num_splits(16, 40, 8192));
    printf("static_bytes %zu\n", (size_t)INSTINFER_STATIC_WORKSPACE_BYTES);
    printf("max_ranks %d\n", INSTINFER_MAX_RANKS);
    printf("failures %d\n", failures);
    return failures ? 1 : 0;
}
