// Context management, parameter validation and status read-back of libcascade.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

static bool in_range(int64_t v, int64_t lo, int64_t hi) { return v >= lo && v <= hi; }

int cascade_validate_params(const cascade_params *p) {
    if (!p) return CASCADE_EINVAL;
    const int64_t one = 1;
    bool ok = in_range(p->bt, 1, 4096) && in_range(p->chunk_shift, 0, 20) && in_range(p->max_batch, 1, 65536) &&
              in_range(p->max_ctx_avg, 0, one << 20) && in_range(p->gamma_q16, 0, one << 17) &&
              in_range(p->n_classes, 1, CASCADE_MAX_CLASSES) && in_range(p->token_budget, 0, one << 30) && p->tier2_reserve >= 0 &&
              in_range(p->c_tok_q20, 0, one << 40) && in_range(p->c_attn_q20, 0, one << 20) &&
              in_range(p->c_iter_q20, 0, one << 50) && in_range(p->c_dseq_q20, 0, one << 40) &&
              in_range(p->c_dkv_q20, 0, one << 28);
    if (ok) ok = (int64_t)(p->max_batch - 1) * p->max_ctx_avg <= (one << 32);
    if (ok) ok = in_range(p->policy, CASCADE_POLICY_BUDGET, CASCADE_POLICY_SJF) && in_range(p->plan_first, 0, 1);
    for (int k = 1; ok && k <= 2; ++k)
        ok = in_range(p->delta_ns[k], 0, one << 30) && in_range(p->blk_ns[k], 1, one << 27);
    for (int c = 0; ok && c < p->n_classes; ++c)
        ok = in_range(p->ttft_ns[c], 0, one << 40) && in_range(p->tpot_ns[c], 0, one << 40);
    return ok ? CASCADE_OK : CASCADE_ERANGE;
}

extern "C" int cascade_version(void) { return 100; }

extern "C" int cascade_create(cascade_ctx **out, const cascade_params *p, int max_requests, int device) {
    if (!out || !p) return CASCADE_EINVAL;
    *out = nullptr;
    if (max_requests < 1 || max_requests > CASCADE_MAX_REQUESTS) return CASCADE_EINVAL;
    int rc = cascade_validate_params(p);
    if (rc != CASCADE_OK) return rc;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return CASCADE_ECUDA;
    int prev_device = 0;
    if (cudaGetDevice(&prev_device) != cudaSuccess) return CASCADE_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) return CASCADE_ECUDA;
    // the calling thread's current device is put back before returning, whatever the outcome
    struct Restore {
        int d;
        ~Restore() { cudaSetDevice(d); }
    } restore{prev_device};
    cascade_ctx *ctx = (cascade_ctx *)calloc(1, sizeof(cascade_ctx));
    if (!ctx) return CASCADE_ENOMEM;
    ctx->params = *p;
    ctx->device = device;
    ctx->max_requests = max_requests;
    cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device);
    ctx->max_cluster = cascade_probe_max_cluster();
    const char *e = getenv("CASCADE_MAX_CLUSTER");   // lower it to exercise the fallback geometry
    if (e && atoi(e) > 0 && atoi(e) < ctx->max_cluster) ctx->max_cluster = atoi(e);
    if ((long long)max_requests > (long long)ctx->max_cluster * 4096) {  // the cluster kernels could not hold the queue
        free(ctx);
        return CASCADE_EINVAL;
    }
    e = getenv("CASCADE_SORT_CLUSTER");
    ctx->sort_cluster = e ? atoi(e) : 0;
    e = getenv("CASCADE_SORT_ITEMS");
    ctx->sort_items = e ? atoi(e) : 0;
    e = getenv("CASCADE_SORT_THREADS");
    ctx->sort_threads = e ? atoi(e) : 0;
    e = getenv("CASCADE_SORT_STAGE");
    ctx->sort_stage = e ? atoi(e) : -1;  // -1: staged scatter only when a thread holds four or more keys
    e = getenv("CASCADE_SORT_ASYNC");
    ctx->sort_async = e ? atoi(e) : 1;
    e = getenv("CASCADE_COPY_CTAS_HOST");
    ctx->copy_ctas_host = e && atoi(e) > 0 ? atoi(e) : 4;
    e = getenv("CASCADE_COPY_CTAS_DEV");
    ctx->copy_ctas_dev = e && atoi(e) > 0 ? atoi(e) : 8;
    e = getenv("CASCADE_COPY_BULK_HOST");
    ctx->copy_bulk_host = e ? atoi(e) : 1;
    e = getenv("CASCADE_COPY_BULK_DEV");
    ctx->copy_bulk_dev = e ? atoi(e) : 2;
    e = getenv("CASCADE_MOVE_CTAS");
    ctx->move_ctas = e ? atoi(e) : 0;
    e = getenv("CASCADE_COPY_GRID_HOST");
    ctx->copy_grid_host = e ? atoi(e) : 0;
    e = getenv("CASCADE_MOVE_CTAS_RESTORE");
    ctx->move_ctas_restore = e ? atoi(e) : 0;
    e = getenv("CASCADE_MOVE_VECTOR");
    ctx->move_vector = e ? (atoi(e) & 3) : 1;   // measured: bulk reads of the restore grid starve beside the evict grid's bulk writes
    e = getenv("CASCADE_CE_LANES");
    ctx->ce_lanes = e && atoi(e) == 2 ? 2 : 1;   // measured: a second stream per direction gains nothing
    e = getenv("CASCADE_COPY_AHEAD_SUB");
    ctx->copy_ahead_sub = e && atoi(e) == 1 ? 1 : 2;   // measured: refilling the slot of the store just issued stalls the ring
    e = getenv("CASCADE_COPY_DYNAMIC");
    ctx->copy_dynamic = e ? (atoi(e) != 0) : 1;
    e = getenv("CASCADE_COPY_PIECE");
    ctx->copy_piece = e ? atoi(e) : 0;
    if (ctx->copy_piece != 8192 && ctx->copy_piece != 16384 && ctx->copy_piece != 32768) ctx->copy_piece = 0;
    e = getenv("CASCADE_COPY_RING_KB");
    ctx->copy_ring_kb = e ? atoi(e) : 0;
    if (ctx->copy_ring_kb < 64 || ctx->copy_ring_kb > 128) ctx->copy_ring_kb = 0;
    e = getenv("CASCADE_MERGE_SORT");
    ctx->merge_sort = e ? atoi(e) : 1;
    e = getenv("CASCADE_SORT_TOP_FIRST");
    ctx->sort_top_first = e ? (atoi(e) != 0) : 1;
    e = getenv("CASCADE_RANK_SORT_MAX");
    ctx->rank_sort_max = e ? atoi(e) : 2048;
    e = getenv("CASCADE_TEST_MOVE_STALL");
    ctx->test_move_stall = e ? atoi(e) : 0;
    if (ctx->test_move_stall < 0 || ctx->test_move_stall > 3) ctx->test_move_stall = 0;
    e = getenv("CASCADE_PDL");
    ctx->pdl = e ? (atoi(e) != 0) : 1;
    size_t n = (size_t)max_requests;
    bool ok = cudaMalloc(&ctx->status_dev, sizeof(uint32_t)) == cudaSuccess &&
              cudaMallocHost(&ctx->status_host, sizeof(uint32_t)) == cudaSuccess &&
              cudaMalloc(&ctx->pack_by_slot, n * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMalloc(&ctx->want_by_slot, n * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&ctx->work_admit, n * sizeof(int4)) == cudaSuccess &&
              cudaMalloc(&ctx->work_victim, n * sizeof(int4)) == cudaSuccess &&
              cudaMalloc(&ctx->plan_scalars, PS_COUNT * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&ctx->copy_tickets, 128 * sizeof(unsigned)) == cudaSuccess;
    for (int i = 0; ok && i < 4; ++i)
        ok = cudaStreamCreateWithFlags(&ctx->ce_stream[i], cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 7; ++i)
        ok = cudaEventCreateWithFlags(&ctx->ce_event[i], cudaEventDisableTiming) == cudaSuccess;
    e = getenv("CASCADE_PLAN_PREPARE_MIN");
    ctx->plan_prepare_min = e ? atoi(e) : 8191;   // measured: a gain from 8192 requests up (16384: 12.2 -> 9.9 us, 65536: 21.5 -> 16.1 us)
    e = getenv("CASCADE_MULTI_SORT");
    ctx->multi_sort = e ? atoi(e) : 1;
    if (ok && max_requests > 16384 && ctx->max_cluster >= 16)
        ok = cudaMalloc(&ctx->sort_runs, n * 16) == cudaSuccess && cudaMalloc(&ctx->sort_sorted, n * 16) == cudaSuccess;
    if (ok) ok = cudaMemset(ctx->status_dev, 0, sizeof(uint32_t)) == cudaSuccess &&
                 cudaMemset(ctx->plan_scalars, 0, PS_COUNT * sizeof(int32_t)) == cudaSuccess &&
                 cudaMemset(ctx->copy_tickets, 0, 128 * sizeof(unsigned)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        cascade_destroy(ctx);
        return CASCADE_ENOMEM;
    }
    *out = ctx;
    return CASCADE_OK;
}

extern "C" void cascade_destroy(cascade_ctx *ctx) {
    if (!ctx) return;
    int prev_device = -1;
    cudaGetDevice(&prev_device);
    cudaSetDevice(ctx->device);
    cudaFree(ctx->status_dev);
    cudaFreeHost(ctx->status_host);
    cudaFree(ctx->pack_by_slot);
    cudaFree(ctx->want_by_slot);
    cudaFree(ctx->work_admit);
    cudaFree(ctx->work_victim);
    cudaFree(ctx->plan_scalars);
    cudaFree(ctx->copy_tickets);
    cudaFree(ctx->sort_runs);
    cudaFree(ctx->sort_sorted);
    for (int i = 0; i < 4; ++i)
        if (ctx->ce_stream[i]) cudaStreamDestroy(ctx->ce_stream[i]);
    for (int i = 0; i < 7; ++i)
        if (ctx->ce_event[i]) cudaEventDestroy(ctx->ce_event[i]);
    free(ctx->ce_bitmap);
    if (prev_device >= 0) cudaSetDevice(prev_device);
    free(ctx);
}

extern "C" int cascade_set_params(cascade_ctx *ctx, const cascade_params *p) {
    if (!ctx) return CASCADE_EINVAL;
    int rc = cascade_validate_params(p);
    if (rc != CASCADE_OK) return rc;
    ctx->params = *p;
    return CASCADE_OK;
}

extern "C" int cascade_step(cascade_ctx *ctx, const cascade_step_args *a, void *stream) {
    CascadeRange nvtx_range("cascade_step");
    if (!ctx || !a || !a->reqs || !a->pools || !a->plan) return CASCADE_EINVAL;
    int rc = CASCADE_OK;
    if (a->upd_m > 0) {
        rc = cascade_reqs_update(ctx, a->reqs, a->upd_cap, a->upd_src, a->upd_slots, a->upd_m, stream);
        if (rc != CASCADE_OK) return rc;
    }
    rc = cascade_budget(ctx, a->reqs, a->n, a->now_ns, a->D_act, a->K_act, a->budget, a->key, stream);
    if (rc != CASCADE_OK) return rc;
    rc = cascade_schedule(ctx, a->reqs, a->key, a->n, a->D_act, a->order, a->grant, a->sched_counts, stream);
    if (rc != CASCADE_OK) return rc;
    rc = cascade_tier_plan(ctx, a->reqs, a->budget, a->order, a->grant, a->n, a->D_act, a->K_act, a->pools, a->plan,
                           stream);
    if (rc != CASCADE_OK) return rc;
    if (a->layout) {
        const cascade_plan *pl = a->plan;
        if (!pl->counts) return CASCADE_EINVAL;
        rc = cascade_kv_move(ctx, a->layout, a->hbm_pool, a->host_pool, a->host_blocks, pl->evict_src, pl->evict_dst,
                             &pl->counts->n_evict, pl->evict_cap, pl->restore_src, pl->restore_dst,
                             &pl->counts->n_restore, pl->restore_cap, a->move_scratch, stream);
    }
    return rc;
}

extern "C" int cascade_status(cascade_ctx *ctx, cascade_status_t *host_out, int clear, void *stream) {
    if (!ctx || !host_out) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    CASCADE_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(uint32_t),
                                          cudaMemcpyDeviceToHost, s));
    if (clear) CASCADE_CUDA_TRY(ctx, cudaMemsetAsync(ctx->status_dev, 0, sizeof(uint32_t), s));
    CASCADE_CUDA_TRY(ctx, cudaStreamSynchronize(s));
    host_out->bits = *ctx->status_host;
    host_out->cuda_error = ctx->cuda_error;
    if (clear) ctx->cuda_error = 0;
    return CASCADE_OK;
}
