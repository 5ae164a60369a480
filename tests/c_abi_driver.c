/*
 * Test infrastructure: one whole iteration through libcascade's C ABI from plain C99 (CUDA runtime API
 * only, no Python, no PyTorch).  Reads a little-endian input file written by tests/test_gpu_c_abi.py,
 * runs budget -> schedule -> tier plan -> evict -> restore on the default stream and writes every output
 * to a second file.  Exit code 0 on success, otherwise the line number of the failing call.
 * Optional third argument: "step" issues the whole iteration as ONE cascade_step call (with the fused move),
 * "staged" moves the blocks through the copy engines (cascade_kv_move_staged) after the three plan calls.
 *
 * Input file:  int64 header[16] = { n, maxb, n_hbm, n_host, n_chunks, chunk_bytes, hbm_free_count,
 *              host_free_count, now_ns, D_act, K_act, sizeof(cascade_params), 0... }, then the parameter
 *              block, then the arrays in the order read below.
 */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "cascade.h"

#define CHECK(cond) do { if (!(cond)) { fprintf(stderr, "c_abi_driver: failed at line %d\n", __LINE__); return __LINE__; } } while (0)

static void *read_exact(FILE *f, size_t bytes) {
    void *p = malloc(bytes ? bytes : 1);
    if (p && bytes && fread(p, 1, bytes, f) != bytes) { free(p); return NULL; }
    return p;
}

static void *to_device(const void *host, size_t bytes) {
    void *d = NULL;
    if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) return NULL;
    if (bytes && host && cudaMemcpy(d, host, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return NULL;
    if (bytes && !host && cudaMemset(d, 0, bytes) != cudaSuccess) return NULL;   /* output buffer */
    return d;
}

static int write_back(FILE *f, const void *dev, size_t bytes) {
    void *h = malloc(bytes ? bytes : 1);
    if (!h) return 0;
    if (bytes && cudaMemcpy(h, dev, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return 0;
    const int ok = fwrite(h, 1, bytes, f) == bytes;
    free(h);
    return ok;
}

int main(int argc, char **argv) {
    CHECK(argc == 3 || argc == 4);
    const int use_step = argc == 4 && strcmp(argv[3], "step") == 0;
    const int use_staged = argc == 4 && strcmp(argv[3], "staged") == 0;
    FILE *in = fopen(argv[1], "rb");
    CHECK(in);
    int64_t hd[16];
    CHECK(fread(hd, sizeof(int64_t), 16, in) == 16);
    const int n = (int)hd[0], maxb = (int)hd[1];
    const int64_t n_hbm = hd[2], n_host = hd[3];
    const int n_chunks = (int)hd[4];
    const int64_t chunk_bytes = hd[5];
    const int32_t hbm_free_count = (int32_t)hd[6], host_free_count = (int32_t)hd[7];
    const int64_t now_ns = hd[8];
    const int32_t D_act = (int32_t)hd[9];
    const int64_t K_act = hd[10];
    CHECK(hd[11] == (int64_t)sizeof(cascade_params));
    cascade_params params;
    CHECK(fread(&params, sizeof params, 1, in) == 1);
    const int64_t bb = (int64_t)n_chunks * chunk_bytes;
    const size_t N = (size_t)n, tbl_bytes = N * (size_t)maxb * 4;

    /* request arrays, tables, free lists, pool bytes */
    void *h_arr = read_exact(in, N * 8), *h_prompt = read_exact(in, N * 4), *h_out = read_exact(in, N * 4);
    void *h_n0 = read_exact(in, N * 4), *h_n1 = read_exact(in, N * 4), *h_n2 = read_exact(in, N * 4);
    void *h_id = read_exact(in, N * 4), *h_cls = read_exact(in, N), *h_flags = read_exact(in, N);
    void *h_hbm_tbl = read_exact(in, tbl_bytes), *h_host_tbl = read_exact(in, tbl_bytes);
    void *h_hbm_free = read_exact(in, (size_t)n_hbm * 4), *h_host_free = read_exact(in, (size_t)n_host * 4);
    void *h_hbm_pool = read_exact(in, (size_t)(n_hbm * bb)), *h_host_pool = read_exact(in, (size_t)(n_host * bb));
    CHECK(h_arr && h_prompt && h_out && h_n0 && h_n1 && h_n2 && h_id && h_cls && h_flags && h_hbm_tbl && h_host_tbl &&
          h_hbm_free && h_host_free && h_hbm_pool && h_host_pool);
    fclose(in);

    CHECK(cudaSetDevice(0) == cudaSuccess);
    cascade_reqs r;
    r.arrival_ns = (const int64_t *)to_device(h_arr, N * 8);
    r.prompt = (const int32_t *)to_device(h_prompt, N * 4);
    r.pred_out = (const int32_t *)to_device(h_out, N * 4);
    r.n0 = (const int32_t *)to_device(h_n0, N * 4);
    r.n1 = (const int32_t *)to_device(h_n1, N * 4);
    r.n2 = (const int32_t *)to_device(h_n2, N * 4);
    r.id = (const uint32_t *)to_device(h_id, N * 4);
    r.cls = (const uint8_t *)to_device(h_cls, N);
    r.flags = (const uint8_t *)to_device(h_flags, N);
    CHECK(r.arrival_ns && r.prompt && r.pred_out && r.n0 && r.n1 && r.n2 && r.id && r.cls && r.flags);

    cascade_pools pools;
    pools.hbm_tbl = (int32_t *)to_device(h_hbm_tbl, tbl_bytes);
    pools.host_tbl = (int32_t *)to_device(h_host_tbl, tbl_bytes);
    pools.maxb = maxb;
    pools.hbm_free = (int32_t *)to_device(h_hbm_free, (size_t)n_hbm * 4);
    pools.hbm_free_count = (int32_t *)to_device(&hbm_free_count, 4);
    pools.hbm_free_cap = (int32_t)n_hbm;
    pools.host_free = (int32_t *)to_device(h_host_free, (size_t)n_host * 4);
    pools.host_free_count = (int32_t *)to_device(&host_free_count, 4);
    pools.host_free_cap = (int32_t)n_host;
    CHECK(pools.hbm_tbl && pools.host_tbl && pools.hbm_free && pools.hbm_free_count && pools.host_free &&
          pools.host_free_count);

    void *hbm_pool = to_device(h_hbm_pool, (size_t)(n_hbm * bb));
    void *host_pool = NULL;                     /* pinned, mapped host memory: the kernels read and write it in place */
    CHECK(hbm_pool && cudaHostAlloc(&host_pool, (size_t)(n_host * bb), cudaHostAllocMapped) == cudaSuccess);
    memcpy(host_pool, h_host_pool, (size_t)(n_host * bb));

    int64_t *budget = (int64_t *)to_device(NULL, N * 8);
    uint64_t *key = (uint64_t *)to_device(NULL, N * 8);
    uint32_t *order = (uint32_t *)to_device(NULL, N * 4);
    int32_t *grant = (int32_t *)to_device(NULL, N * 4);
    cascade_sched_counts *sc = (cascade_sched_counts *)to_device(NULL, sizeof *sc);
    cascade_plan plan;
    plan.x1 = (int32_t *)to_device(NULL, N * 4);
    plan.x2 = (int32_t *)to_device(NULL, N * 4);
    plan.tokens_run = (int32_t *)to_device(NULL, N * 4);
    plan.action = (uint8_t *)to_device(NULL, N);
    plan.restore_cap = (int32_t)n_hbm;
    plan.evict_cap = (int32_t)n_host;
    plan.restore_src = (int32_t *)to_device(NULL, (size_t)n_hbm * 4);
    plan.restore_dst = (int32_t *)to_device(NULL, (size_t)n_hbm * 4);
    plan.evict_src = (int32_t *)to_device(NULL, (size_t)n_host * 4);
    plan.evict_dst = (int32_t *)to_device(NULL, (size_t)n_host * 4);
    plan.counts = (cascade_plan_counts *)to_device(NULL, sizeof(cascade_plan_counts));
    CHECK(budget && key && order && grant && sc && plan.x1 && plan.x2 && plan.tokens_run && plan.action &&
          plan.restore_src && plan.restore_dst && plan.evict_src && plan.evict_dst && plan.counts);
    CHECK(cudaMemset(plan.restore_src, 0xff, (size_t)n_hbm * 4) == cudaSuccess);
    CHECK(cudaMemset(plan.restore_dst, 0xff, (size_t)n_hbm * 4) == cudaSuccess);
    CHECK(cudaMemset(plan.evict_src, 0xff, (size_t)n_host * 4) == cudaSuccess);
    CHECK(cudaMemset(plan.evict_dst, 0xff, (size_t)n_host * 4) == cudaSuccess);

    cascade_kv_layout lay;
    lay.n_blocks = n_hbm;
    lay.n_chunks = n_chunks;
    lay.reserved = 0;
    lay.chunk_bytes = chunk_bytes;
    lay.chunk_stride = n_hbm * chunk_bytes;
    lay.block_stride = chunk_bytes;

    cascade_ctx *ctx = NULL;
    CHECK(cascade_create(&ctx, &params, n, 0) == CASCADE_OK);
    if (use_step) {
        const int64_t words = cascade_kv_move_scratch_len(plan.evict_cap, plan.restore_cap);
        CHECK(words > 0);
        cascade_step_args a;
        memset(&a, 0, sizeof a);
        a.reqs = &r;
        a.n = n;
        a.D_act = D_act;
        a.K_act = K_act;
        a.now_ns = now_ns;
        a.budget = budget;
        a.key = key;
        a.order = order;
        a.grant = grant;
        a.sched_counts = sc;
        a.pools = &pools;
        a.plan = &plan;
        a.layout = &lay;
        a.hbm_pool = hbm_pool;
        a.host_pool = host_pool;
        a.host_blocks = n_host;
        a.move_scratch = (int32_t *)to_device(NULL, (size_t)words * 4);
        CHECK(a.move_scratch);
        CHECK(cascade_step(ctx, &a, NULL) == CASCADE_OK);
    } else {
        CHECK(cascade_budget(ctx, &r, n, now_ns, D_act, K_act, budget, key, NULL) == CASCADE_OK);
        CHECK(cascade_schedule(ctx, &r, key, n, D_act, order, grant, sc, NULL) == CASCADE_OK);
        CHECK(cascade_tier_plan(ctx, &r, budget, order, grant, n, D_act, K_act, &pools, &plan, NULL) == CASCADE_OK);
        if (use_staged) {
            const int64_t words = cascade_kv_mailbox_len(plan.evict_cap, plan.restore_cap);
            const int64_t staging_blocks = 24;                 /* smaller than the lists: the batches wrap */
            int32_t *mailbox = NULL;
            void *staging = to_device(NULL, (size_t)(staging_blocks * bb));
            CHECK(words > 0 && staging && cudaHostAlloc((void **)&mailbox, (size_t)words * 4, cudaHostAllocMapped) == cudaSuccess);
            CHECK(cascade_kv_move_staged(ctx, &lay, hbm_pool, host_pool, n_host, plan.evict_src, plan.evict_dst,
                                         &plan.counts->n_evict, plan.evict_cap, plan.restore_src, plan.restore_dst,
                                         &plan.counts->n_restore, plan.restore_cap, staging, staging_blocks, mailbox,
                                         NULL) == CASCADE_OK);
        } else {
            CHECK(cascade_kv_evict(ctx, &lay, hbm_pool, host_pool, n_host, 0, plan.evict_src, plan.evict_dst,
                                   &plan.counts->n_evict, plan.evict_cap, NULL) == CASCADE_OK);
            CHECK(cascade_kv_restore(ctx, &lay, hbm_pool, host_pool, n_host, 0, plan.restore_src, plan.restore_dst,
                                     &plan.counts->n_restore, plan.restore_cap, NULL) == CASCADE_OK);
        }
    }
    cascade_status_t st;
    CHECK(cascade_status(ctx, &st, 1, NULL) == CASCADE_OK);

    FILE *out = fopen(argv[2], "wb");
    CHECK(out);
    int64_t oh[4] = { (int64_t)st.bits, (int64_t)st.cuda_error, (int64_t)cascade_version(), 0 };
    CHECK(fwrite(oh, sizeof(int64_t), 4, out) == 4);
    CHECK(write_back(out, budget, N * 8) && write_back(out, key, N * 8) && write_back(out, order, N * 4) &&
          write_back(out, grant, N * 4) && write_back(out, sc, sizeof *sc) && write_back(out, plan.x1, N * 4) &&
          write_back(out, plan.x2, N * 4) && write_back(out, plan.tokens_run, N * 4) && write_back(out, plan.action, N) &&
          write_back(out, plan.counts, sizeof(cascade_plan_counts)) &&
          write_back(out, plan.restore_src, (size_t)n_hbm * 4) && write_back(out, plan.restore_dst, (size_t)n_hbm * 4) &&
          write_back(out, plan.evict_src, (size_t)n_host * 4) && write_back(out, plan.evict_dst, (size_t)n_host * 4) &&
          write_back(out, pools.hbm_tbl, tbl_bytes) && write_back(out, pools.host_tbl, tbl_bytes) &&
          write_back(out, pools.hbm_free_count, 4) && write_back(out, pools.host_free_count, 4) &&
          write_back(out, hbm_pool, (size_t)(n_hbm * bb)));
    CHECK(fwrite(host_pool, 1, (size_t)(n_host * bb), out) == (size_t)(n_host * bb));
    fclose(out);
    cascade_destroy(ctx);
    return 0;
}
