// cascade_prefetch_plan: budget-bounded prefetch for requests that stay queued (the prefix
// prefetcher acting ahead of admission).  After the tier plan, link time the admitted set did not
// use and HBM blocks above a reserve are given, in schedule order, to queued requests that hold
// host blocks: each gets at most its Eq. 7 bound (and only if restoring beats recomputing), then
// what the link budget and the free HBM still allow.
//
// Kernel 1 (thread-block cluster, same geometry as the tier plan): gather through `order`, Eq. 7
// per queued request, prefix sums of transfer time / blocks / requests over the order, one exchange
// of CTA totals through distributed shared memory.  Walking the order with a running allowance is
// a clamped scan: every request before the first one that is cut gets its full bound, the cut one
// gets what is left, nothing behind it gets anything.
// Kernel 2 (one warp per served request): pop HBM ids, extend the restore list, fill the HBM table.
#include <cooperative_groups.h>

#include "cluster_scan.cuh"
#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kMaxCluster = 16;

struct PrefetchArgs {
    const int32_t *prompt, *n0, *n1, *n2;
    const int64_t *budget;
    const uint32_t *order;
    const int32_t *grant;
    const uint8_t *action;
    cascade_pools pools;
    cascade_plan plan;
    int32_t *pf_out;
    cascade_prefetch_counts *counts;
    int4 *work;
    int32_t *scalars;
    uint32_t *status;
    int64_t A_act;
    int64_t link_budget_ns;
    int hbm_reserve;
    int n;
    int with_tables;
};

struct __align__(16) PfExch1 {
    long long time, used;
    int blocks, count;
    long long pad;
};
struct __align__(16) PfExch2 {
    int n_pf, n_req, pad0, pad1;
};

template <int T, int K>
__global__ void __launch_bounds__(T, 1)
prefetch_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ PrefetchArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int per = T * K;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();
    __shared__ int ws3[33][3];
    __shared__ long long ws8[33][8];
    __shared__ PfExch1 ex1[kMaxCluster];
    __shared__ PfExch2 ex2[kMaxCluster];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n;
    const int bt = p.bt;
    uint32_t st = 0;
    // "I have started": waited for in front of the first store into another CTA's shared memory (which must exist by
    // then); the barrier's latency hides behind the per-request work
    cluster.barrier_arrive();

    long long hbm_cnt = *a.pools.hbm_free_count;
    if (a.with_tables && (hbm_cnt < 0 || hbm_cnt > a.pools.hbm_free_cap)) {
        st |= CASCADE_ST_EBOUNDS;
        hbm_cnt = hbm_cnt < 0 ? 0 : a.pools.hbm_free_cap;
    }
    const int n_restore0 = a.plan.counts->n_restore;

    // ---- per request: is it queued, and what does Eq. 7 allow ------------------------------------
    uint32_t slot[K];
    int mv[K], cv[K], zero[K];
    long long tv[K];
    bool real[K];
    long long used = 0;
    const long long pos0 = (long long)crank * per + (warp * K) * 32 + lane;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long q = pos0 + k * 32;
        slot[k] = q < n ? a.order[q] : 0u;
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long q = pos0 + k * 32;
        mv[k] = 0;
        cv[k] = 0;
        zero[k] = 0;
        tv[k] = 0;
        real[k] = q < n;
        if (!real[k]) continue;
        const uint32_t r = slot[k];
        const long long P = a.prompt[r], n0 = a.n0[r], n1 = a.n1[r], n2 = a.n2[r];
        bool valid = dev_request_valid(bt, P, n0, n1, n2);
        if (valid && a.with_tables) valid = (P + bt - 1) / bt <= a.pools.maxb;
        if (!valid) continue;
        const int g = a.grant[r];
        if (g > 0) {
            used += dev_restore_time(p, 1, a.plan.x1[r]);   // link time of the admitted set's own restores
            continue;
        }
        const unsigned act = a.action[r];
        if (n1 <= 0 || act == CASCADE_ACT_EVICT || act == CASCADE_ACT_DROP) continue;
        const long long b = a.budget[r];
        const long long rem = b > 0 ? b : 0;
        long long head = rem - p.delta_ns[1];
        if (head < 0) head = 0;
        long long m = head / p.blk_ns[1];
        if (m > n1) m = n1;
        if (m > 0) {
            const long long F1 = (dev_restore_time(p, 1, m) << 20) + dev_comp_q(a.A_act, p.c_attn_q20, P, (n0 + m) * bt);
            const long long F0 = dev_comp_q(a.A_act, p.c_attn_q20, P, n0 * bt);
            if (F1 > F0) m = 0;
        }
        if (m > 0) {
            mv[k] = (int)m;
            cv[k] = 1;
            tv[k] = dev_restore_time(p, 1, m);
        }
    }

    // ---- prefix sums over the order, one exchange -------------------------------------------------
    int want[K];
#pragma unroll
    for (int k = 0; k < K; ++k) want[k] = mv[k];
    int tot[3];
    cta_scan3<T, K>(mv, cv, zero, tot, ws3);               // mv, cv now inclusive
    const long long t_total = cta_scan_ll<T, K>(tv, &ws8[0][0]);
    long long red[1] = {used};
    cta_sum<T, 1>(red, ws8);
    cluster.barrier_wait();
    if (tid < csize) {
        PfExch1 x;
        x.time = t_total;
        x.used = red[0];
        x.blocks = tot[0];
        x.count = tot[1];
        x.pad = 0;
        cluster.map_shared_rank(ex1, tid)[crank] = x;
    }
    cluster.sync();
    long long off_t = 0, used_all = 0;
    int off_b = 0, off_c = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < csize) {
            const PfExch1 x = ex1[c];
            used_all += x.used;
            if (c < crank) { off_t += x.time; off_b += x.blocks; off_c += x.count; }
        }
    }
    const long long link0 = a.link_budget_ns - used_all;
    const long long avail0 = hbm_cnt - a.hbm_reserve;
    long long s_pf = 0, s_req = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (!real[k]) continue;
        int b = 0;
        if (want[k] > 0) {
            const long long m = want[k];
            const long long e_t = off_t + tv[k] - dev_restore_time(p, 1, m);   // exclusive
            const long long e_b = (long long)off_b + mv[k] - m;
            const long long left = link0 - e_t;
            long long by_link = left > p.delta_ns[1] ? (left - p.delta_ns[1]) / p.blk_ns[1] : 0;
            long long by_hbm = avail0 - e_b;
            if (by_hbm < 0) by_hbm = 0;
            long long bb = m < by_link ? m : by_link;
            if (by_hbm < bb) bb = by_hbm;
            b = (int)bb;
            if (b > 0) {
                // every served request before this one got its full bound, so the exclusive sums are exact
                a.work[off_c + cv[k] - 1] = make_int4((int)slot[k], (int)e_b, n_restore0 + (int)e_b, b);
                s_pf += b;
                ++s_req;
            }
        }
        a.pf_out[slot[k]] = b;
    }
    long long red2[2] = {s_pf, s_req};
    cta_sum<T, 2>(red2, ws8);
    if (tid == 0) {
        PfExch2 x;
        x.n_pf = (int)red2[0];
        x.n_req = (int)red2[1];
        x.pad0 = x.pad1 = 0;
        cluster.map_shared_rank(ex2, 0)[crank] = x;
    }
    st = __reduce_or_sync(kFull, st);
    if (lane == 0 && st) atomicOr(a.status, st);
    cluster.sync();
    if (crank == 0 && tid == 0) {
        int n_pf = 0, n_req = 0;
        for (unsigned c = 0; c < csize; ++c) {
            n_pf += ex2[c].n_pf;
            n_req += ex2[c].n_req;
        }
        a.counts->n_prefetch = n_pf;
        a.counts->n_requests = n_req;
        a.counts->hbm_free_after = (int)(hbm_cnt - n_pf);
        a.counts->n_restore_total = n_restore0 + n_pf;
        a.counts->link_ns_left = link0;
        a.scalars[PS_N_ADMIT] = n_req;
        a.scalars[PS_HBM_CNT0] = (int)hbm_cnt;
        if (a.with_tables) {
            *a.pools.hbm_free_count = (int)(hbm_cnt - n_pf);
            a.plan.counts->n_restore = n_restore0 + n_pf;
        }
    }
}

__global__ void __launch_bounds__(256) apply_prefetch_kernel(const __grid_constant__ PrefetchArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const int n_items = a.scalars[PS_N_ADMIT];
    const long long top = a.scalars[PS_HBM_CNT0];
    uint32_t st = 0;
    for (int i = warp; i < n_items; i += n_warps) {
        const int4 it = a.work[i];
        const int slot = it.x;
        const int n0 = a.n0[slot];
        int32_t *hrow = a.pools.hbm_tbl + (size_t)slot * a.pools.maxb;
        const int32_t *orow = a.pools.host_tbl + (size_t)slot * a.pools.maxb;
        for (int jj = lane; jj < it.w; jj += 32) {
            const int j = n0 + jj;
            if (j >= a.pools.maxb) break;
            const long long pp = top - 1 - ((long long)it.y + jj);
            int32_t g = -1;
            if (pp >= 0 && pp < a.pools.hbm_free_cap) g = a.pools.hbm_free[pp]; else st |= CASCADE_ST_EBOUNDS;
            const long long e = (long long)it.z + jj;
            if (e < a.plan.restore_cap) {
                a.plan.restore_src[e] = orow[j];
                a.plan.restore_dst[e] = g;
            } else {
                st |= CASCADE_ST_ELISTCAP;
            }
            hrow[j] = g;
        }
    }
    if (st) atomicOr(a.status, st);
}

template <int T, int K>
cudaError_t launch_pf(const cascade_params &p, const PrefetchArgs &a, int cluster_size, bool pdl, cudaStream_t stream) {
    static CascadeDeviceOnce configured;
    int device = 0;
    cudaGetDevice(&device);
    if (!configured.is_set(device)) {
        cudaError_t e = cudaFuncSetAttribute(prefetch_kernel<T, K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured.set(device);
    }
    return cascade_launch(pdl, cluster_size, dim3(cluster_size), dim3(T), 0, stream, prefetch_kernel<T, K>, p, a);
}

template <int T>
cudaError_t launch_pf_k(int K, const cascade_params &p, const PrefetchArgs &a, int C, bool pdl, cudaStream_t s) {
    switch (K) {
        case 1: return launch_pf<T, 1>(p, a, C, pdl, s);
        case 2: return launch_pf<T, 2>(p, a, C, pdl, s);
        case 4: return launch_pf<T, 4>(p, a, C, pdl, s);
        default: return launch_pf<T, 8>(p, a, C, pdl, s);
    }
}

}  // namespace

extern "C" int cascade_prefetch_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget,
                                     const uint32_t *order, const int32_t *grant, const uint8_t *action, int n,
                                     int32_t D_act, int64_t K_act, int64_t link_budget_ns, int32_t hbm_reserve,
                                     const cascade_pools *pools, const cascade_plan *plan, int32_t *pf_out,
                                     cascade_prefetch_counts *counts_dev, void *stream) {
    CascadeRange nvtx_range("cascade_prefetch_plan");
    if (!ctx || !r || !pools || !plan || !counts_dev || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (!plan->counts || !pools->hbm_free_count) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    if (link_budget_ns < 0 || link_budget_ns > (int64_t(1) << 50) || hbm_reserve < 0) return CASCADE_ERANGE;
    const bool with_tables = pools->hbm_tbl != nullptr;
    if (n > 0 && (!budget || !order || !grant || !action || !pf_out || !plan->x1 || !r->prompt || !r->n0 || !r->n1 ||
                  !r->n2))
        return CASCADE_EINVAL;
    if (with_tables) {
        if (!pools->host_tbl || !pools->hbm_free || pools->maxb < 1 || pools->hbm_free_cap < 0 ||
            plan->restore_cap < 0 || (plan->restore_cap > 0 && (!plan->restore_src || !plan->restore_dst)))
            return CASCADE_EINVAL;
    }
    cudaStream_t s = (cudaStream_t)stream;
    PrefetchArgs a;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.budget = budget;
    a.order = order;
    a.grant = grant;
    a.action = action;
    a.pools = *pools;
    a.plan = *plan;
    a.pf_out = pf_out;
    a.counts = counts_dev;
    a.work = ctx->work_admit;
    a.scalars = ctx->plan_scalars;
    a.status = ctx->status_dev;
    a.A_act = make_load_consts(ctx->params, D_act, K_act).A_act;
    a.link_budget_ns = link_budget_ns;
    a.hbm_reserve = hbm_reserve;
    a.n = n;
    a.with_tables = with_tables ? 1 : 0;
    int T, C, K;
    if (!cascade_pick_geometry(ctx, n > 0 ? n : 1, &T, &C, &K)) return CASCADE_EINVAL;
    cudaError_t e = T == 256 ? launch_pf_k<256>(K, ctx->params, a, C, ctx->pdl, s) : launch_pf_k<512>(K, ctx->params, a, C, ctx->pdl, s);
    CASCADE_CUDA_TRY(ctx, e);
    if (with_tables && n > 0) {
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(ctx->num_sms * 2), dim3(256), 0, s, apply_prefetch_kernel, a));
    }
    return CASCADE_OK;
}
