// cascade_tier_plan: restore bound (Eq. 7), restore-vs-recompute choice, HBM capacity check,
// preemption victims with their disposition (Algorithm 1), and deterministic block-id allocation.
//
// Kernel 1 (one thread-block cluster, the queue spread over its CTAs in schedule order, K
// elements per thread held in registers):
//   phase 1  in slot order (coalesced loads): Eq. 7 and the candidate plans (the only int64 divisions
//            of the path, at most two per admitted request), default per-request outputs, and one
//            packed decision word per request; after a cluster barrier the schedule-order phases
//            gather just that word through `order`;
//   phase 2  forward prefix sums over the admitted set (cumulative HBM need, restore-list offsets)
//            and the sum of preemptable blocks; one exchange of per-CTA totals through distributed
//            shared memory; the admitted set is cut where the cumulative need exceeds the capacity;
//   phase 3  prefix sums over the preemptable holders; one more exchange; walking the order
//            backwards is the same as subtracting the forward inclusive sum from the total, so the
//            sequential "pop one request / preempt the largest budget" loops of Algorithm 1 become
//            two scans because admitted requests and victims are prefixes of the two walks;
//   phase 4  per-request outputs are scattered by slot; CTA 0 writes the counts.
// Four hardware cluster barriers are the only inter-CTA waits (no spin loops).
// Kernels 2 and 3 (many CTAs, one warp per request): rewrite block tables, free lists and the two
// copy lists from the offsets kernel 1 left in scratch; pushes of freed ids (kernel 2) finish
// before any pop (kernel 3).  In plan-only mode (no tables) only kernel 1 runs.
#include <stdlib.h>

#include <atomic>
#include <mutex>

#include <cooperative_groups.h>

#include "common.cuh"
#include "cluster_scan.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kMaxCluster = 16;

// element flags
constexpr unsigned kAdm = 1u, kPriv = 2u, kFits = 4u, kValid = 8u, kReal = 16u;

struct PlanArgs {
    const int32_t *prompt, *n0, *n1, *n2;
    const uint8_t *flags;
    const int64_t *budget;
    const uint32_t *order;
    int32_t *grant;
    cascade_pools pools;
    cascade_plan plan;
    unsigned long long *pack;          // one decision word per request, slot order (scratch)
    int4 *work_admit, *work_victim;
    int32_t *scalars;
    uint32_t *status;
    int64_t A_act;
    int n;
    int with_tables;
    int prepared;                      // 1: phase 1a was done by plan_prepare_kernel
};

// per-CTA totals published to every CTA of the cluster
struct __align__(16) Exch1 {
    int need, x1, cnt, evictable;
};
struct __align__(16) Exch2 {
    int v, h, c;                      // preemptable holders: blocks, blocks that fit, requests
    int kept_need, kept_cnt, kept_x1, unadm;
    int pad;
    long long tokens;
    long long pad2;
};
struct __align__(16) Exch3 {
    int nv, freed, nev, pad;
};

// Phase 1a for one request (slot r): Eq. 7 bounds and the restore-vs-recompute choice; the per-request outputs
// get their default values and one packed word (n0 | x1 << 14 | tokens_run << 28 | flags << 46) is left for
// the schedule-order phases.  Returns the status bits it found.
__device__ __forceinline__ uint32_t plan_prepare_one(const cascade_params &p, const PlanArgs &a, long long r) {
    const int bt = p.bt;
    uint32_t st = 0;
    const long long P = a.prompt[r], n0 = a.n0[r], n1 = a.n1[r], n2 = a.n2[r];
    const long long b = a.budget[r];
    const int g = a.grant[r];
    const unsigned rf = a.flags[r];
    bool valid = dev_request_valid(bt, P, n0, n1, n2);
    if (valid && a.with_tables) valid = (P + bt - 1) / bt <= a.pools.maxb;
    unsigned long long w = (unsigned long long)kReal << 46;
    int x1 = 0, x2 = 0, run = 0;
    if (!valid) {
        st |= CASCADE_ST_EPRECOND;
        if (g != 0) a.grant[r] = 0;
    } else {
        unsigned f = kReal | kValid;
        if (rf & CASCADE_FLAG_HBM_PRIVATE) f |= kPriv;
        if (dev_restore_time(p, 1, n0) <= b) f |= kFits;
        if (g > 0) {
            int64_t bx1, bx2;
            dev_choose_restore(p, a.A_act, P, n0, n1, n2, b, &bx1, &bx2);
            // a deep fetch is staged first: nothing runs now, HBM is taken at the last hop only
            const long long left = P - (n0 + bx1) * bt;
            x1 = (int)bx1;
            x2 = (int)bx2;
            run = bx2 > 0 ? 0 : (int)(g < left ? g : left);
            f |= kAdm;
        }
        w = (unsigned long long)n0 | ((unsigned long long)x1 << 14) | ((unsigned long long)run << 28) |
            ((unsigned long long)f << 46);
    }
    a.pack[r] = w;
    a.plan.x1[r] = x1;
    a.plan.x2[r] = x2;
    a.plan.tokens_run[r] = run;
    a.plan.action[r] = (valid && n0 > 0) ? CASCADE_ACT_RETAIN : CASCADE_ACT_NONE;
    return st;
}

// Phase 1a as a grid of its own, one thread per request: used for large queues, where the sixteen CTAs of the
// cluster kernel would spend several microseconds on what the whole GPU does in one.
__global__ void __launch_bounds__(256)
plan_prepare_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ PlanArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t st = r < a.n ? plan_prepare_one(p, a, r) : 0u;
    st = __reduce_or_sync(0xffffffffu, st);
    if ((threadIdx.x & 31) == 0 && st) atomicOr(a.status, st);
}

template <int T, int K>
__global__ void __launch_bounds__(T, 1)
plan_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ PlanArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int per = T * K;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();
    __shared__ int ws3[33][3];
    __shared__ long long ws8[32][8];
    __shared__ Exch1 ex1[kMaxCluster];
    __shared__ Exch2 ex2[kMaxCluster];
    __shared__ Exch3 ex3[kMaxCluster];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n;
    const int bt = p.bt;
    uint32_t st = 0;

    long long hbm_cnt = *a.pools.hbm_free_count;
    long long host_cnt = *a.pools.host_free_count;
    if (a.with_tables) {
        if (hbm_cnt < 0 || hbm_cnt > a.pools.hbm_free_cap) {
            st |= CASCADE_ST_EBOUNDS;
            hbm_cnt = hbm_cnt < 0 ? 0 : a.pools.hbm_free_cap;
        }
        if (host_cnt < 0 || host_cnt > a.pools.host_free_cap) {
            st |= CASCADE_ST_EBOUNDS;
            host_cnt = host_cnt < 0 ? 0 : a.pools.host_free_cap;
        }
    }

    // ---- phase 1a, slot order (coalesced): Eq. 7 bounds and the restore-vs-recompute choice; the
    //      per-request outputs get their default values here and one packed word per request
    //      (n0 | x1 << 14 | tokens_run << 28 | flags << 46) is left for the schedule-order phases
    const long long pos0 = (long long)crank * per + (warp * K) * 32 + lane;
    if (!a.prepared) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const long long r = pos0 + k * 32;
            if (r < n) st |= plan_prepare_one(p, a, r);
        }
        cluster.sync();  // the packed words are visible to every CTA of the cluster
    } else {
        // the packed words come from the grid before; only "every CTA has started" is needed, in front of the first
        // store into a neighbour's shared memory: the wait sits there and the gathers below run in the meantime
        cluster.barrier_arrive();
    }

    // ---- phase 1b, schedule order: one 8-byte gather per element --------------------------------
    uint32_t slot[K];
    unsigned fl[K];
    int n0v[K], x1v[K], runv[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long q = pos0 + k * 32;
        slot[k] = q < n ? a.order[q] : 0u;
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long q = pos0 + k * 32;
        const unsigned long long w = q < n ? a.pack[slot[k]] : 0ull;
        fl[k] = (unsigned)(w >> 46);
        n0v[k] = (int)(w & 0x3fff);
        x1v[k] = (int)((w >> 14) & 0x3fff);
        runv[k] = (int)((w >> 28) & 0x3ffff);
    }

    // ---- phase 2: forward scan over the admitted set, capacity cut --------------------------------
    int s_need[K], s_x1[K], s_cnt[K];
    long long evictable = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const bool adm = fl[k] & kAdm;
        s_need[k] = adm ? x1v[k] + (runv[k] + bt - 1) / bt : 0;
        s_x1[k] = adm ? x1v[k] : 0;
        s_cnt[k] = adm ? 1 : 0;
        if ((fl[k] & kValid) && !adm && (fl[k] & kPriv)) evictable += n0v[k];
    }
    int tot[3];
    cta_scan3<T, K>(s_need, s_x1, s_cnt, tot, ws3);
    long long red1[1] = {evictable};
    cta_sum<T, 1>(red1, ws8);
    if (a.prepared) cluster.barrier_wait();
    if (tid < csize) {
        Exch1 x;
        x.need = tot[0];
        x.x1 = tot[1];
        x.cnt = tot[2];
        x.evictable = (int)red1[0];
        cluster.map_shared_rank(ex1, tid)[crank] = x;
    }
    cluster.sync();
    long long off_need = 0, cap = hbm_cnt;
    int off_x1 = 0, off_cnt = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < csize) {
            const Exch1 x = ex1[c];
            cap += x.evictable;
            if (c < crank) { off_need += x.need; off_x1 += x.x1; off_cnt += x.cnt; }
        }
    }
    long long k_need = 0, k_cnt = 0, k_x1 = 0, k_unadm = 0, k_tok = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (!(fl[k] & kAdm)) continue;
        const int nd = x1v[k] + (runv[k] + bt - 1) / bt;
        const long long c_incl = off_need + s_need[k];
        if (c_incl > cap) {
            // HBM cannot hold it even after preempting everything preemptable: cut from the tail
            fl[k] &= ~kAdm;
            x1v[k] = 0;
            runv[k] = 0;
            a.grant[slot[k]] = 0;
            a.plan.x1[slot[k]] = 0;
            a.plan.x2[slot[k]] = 0;
            a.plan.tokens_run[slot[k]] = 0;
            ++k_unadm;
            st |= CASCADE_ST_ENOSPC;
        } else {
            k_need += nd;
            ++k_cnt;
            k_x1 += x1v[k];
            k_tok += runv[k];
            a.work_admit[off_cnt + s_cnt[k] - 1] =
                make_int4((int)slot[k], (int)(c_incl - nd), off_x1 + s_x1[k] - x1v[k], (x1v[k] << 18) | nd);
        }
    }

    // ---- phase 3: preemptable holders, walked backwards ---------------------------------------------
    int s_v[K], s_h[K], s_c[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const bool elig = (fl[k] & kValid) && !(fl[k] & kAdm) && (fl[k] & kPriv) && n0v[k] > 0;
        s_v[k] = elig ? n0v[k] : 0;
        s_h[k] = (elig && (fl[k] & kFits)) ? n0v[k] : 0;
        s_c[k] = elig ? 1 : 0;
    }
    cta_scan3<T, K>(s_v, s_h, s_c, tot, ws3);
    long long red5[5] = {k_need, k_cnt, k_x1, k_unadm, k_tok};
    cta_sum<T, 5>(red5, ws8);
    if (tid < csize) {
        Exch2 x;
        x.v = tot[0];
        x.h = tot[1];
        x.c = tot[2];
        x.kept_need = (int)red5[0];
        x.kept_cnt = (int)red5[1];
        x.kept_x1 = (int)red5[2];
        x.unadm = (int)red5[3];
        x.pad = 0;
        x.tokens = red5[4];
        x.pad2 = 0;
        cluster.map_shared_rank(ex2, tid)[crank] = x;
    }
    cluster.sync();
    long long need_total = 0, V = 0, H = 0, tokens = 0;
    int Cn = 0, off_v = 0, off_h = 0, off_c = 0, n_adm = 0, n_rest = 0, n_unadm = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < csize) {
            const Exch2 x = ex2[c];
            need_total += x.kept_need;
            n_adm += x.kept_cnt;
            n_rest += x.kept_x1;
            n_unadm += x.unadm;
            tokens += x.tokens;
            V += x.v;
            H += x.h;
            Cn += x.c;
            if (c < crank) { off_v += x.v; off_h += x.h; off_c += x.c; }
        }
    }
    long long deficit = need_total - hbm_cnt;
    if (deficit < 0) deficit = 0;
    long long s_nv = 0, s_freed = 0, s_nev = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (!(fl[k] & kReal)) continue;
        uint8_t act = CASCADE_ACT_NONE;
        if (fl[k] & kValid) {
            const int n0 = n0v[k];
            const bool elig = !(fl[k] & kAdm) && (fl[k] & kPriv) && n0 > 0;
            // blocks of preemptable holders visited before this one when the order is walked backwards
            const long long v = V - (off_v + s_v[k]);
            if (elig && v < deficit) {
                // spill only if it can be brought back within the victim's own budget and host has room
                const long long h = H - (off_h + s_h[k]);
                const bool ev = (fl[k] & kFits) && (h + n0 <= host_cnt);
                act = ev ? CASCADE_ACT_EVICT : CASCADE_ACT_DROP;
                a.work_victim[Cn - (off_c + s_c[k])] = make_int4((int)slot[k], (int)v, (int)h, (int)act);
                ++s_nv;
                s_freed += n0;
                if (ev) s_nev += n0;
            } else if (n0 > 0) {
                act = CASCADE_ACT_RETAIN;
            }
        }
        // ---- phase 4: only preempted requests change the action written in phase 1a -----------------
        if (act == CASCADE_ACT_EVICT || act == CASCADE_ACT_DROP) a.plan.action[slot[k]] = act;
    }
    long long red3[3] = {s_nv, s_freed, s_nev};
    cta_sum<T, 3>(red3, ws8);
    if (tid == 0) {
        Exch3 x;
        x.nv = (int)red3[0];
        x.freed = (int)red3[1];
        x.nev = (int)red3[2];
        x.pad = 0;
        cluster.map_shared_rank(ex3, 0)[crank] = x;
    }
    st = __reduce_or_sync(kFull, st);
    if (lane == 0 && st) atomicOr(a.status, st);
    cluster.sync();
    if (crank == 0 && tid == 0) {
        long long nv = 0, freed = 0, nev = 0;
        for (unsigned c = 0; c < csize; ++c) {
            nv += ex3[c].nv;
            freed += ex3[c].freed;
            nev += ex3[c].nev;
        }
        cascade_plan_counts *c = a.plan.counts;
        c->n_restore = n_rest;
        c->n_evict = (int)nev;
        c->n_drop_blocks = (int)(freed - nev);
        c->n_victims = (int)nv;
        c->n_unadmitted = n_unadm;
        c->n_admitted = n_adm;
        c->hbm_need = (int)need_total;
        c->deficit = (int)deficit;
        c->hbm_free_after = (int)(hbm_cnt + freed - need_total);
        c->host_free_after = (int)(host_cnt - nev);
        c->tokens_run = tokens;
        a.scalars[PS_N_ADMIT] = n_adm;
        a.scalars[PS_N_VICTIM] = (int)nv;
        a.scalars[PS_HBM_CNT0] = (int)hbm_cnt;
        a.scalars[PS_HOST_CNT0] = (int)host_cnt;
        a.scalars[PS_TOTAL_FREED] = (int)freed;
        if (a.with_tables) {
            *a.pools.hbm_free_count = (int)(hbm_cnt + freed - need_total);
            *a.pools.host_free_count = (int)(host_cnt - nev);
        }
    }
}

// One warp per preempted request: move its HBM ids to the free stack, and for EVICT take host
// records, fill the evict list and the host table.
__global__ void __launch_bounds__(256)
apply_victims_kernel(const __grid_constant__ PlanArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const int nv = a.scalars[PS_N_VICTIM];
    const long long hbm_cnt = a.scalars[PS_HBM_CNT0], host_cnt = a.scalars[PS_HOST_CNT0];
    uint32_t st = 0;
    for (int i = warp; i < nv; i += n_warps) {
        const int4 it = a.work_victim[i];
        const int slot = it.x;
        const int n0 = min(a.n0[slot], a.pools.maxb);
        int32_t *hrow = a.pools.hbm_tbl + (size_t)slot * a.pools.maxb;
        int32_t *orow = a.pools.host_tbl + (size_t)slot * a.pools.maxb;
        for (int j = lane; j < n0; j += 32) {
            const int32_t g = hrow[j];
            if (it.w == (int)CASCADE_ACT_EVICT) {
                const long long e = (long long)it.z + j;
                const long long hp = host_cnt - 1 - e;
                const int32_t hs = (hp >= 0 && hp < a.pools.host_free_cap) ? a.pools.host_free[hp] : -1;
                if (e < a.plan.evict_cap) {
                    a.plan.evict_src[e] = g;
                    a.plan.evict_dst[e] = hs;
                } else {
                    st |= CASCADE_ST_ELISTCAP;
                }
                orow[j] = hs;
            }
            const long long pp = hbm_cnt + it.y + j;
            if (pp < a.pools.hbm_free_cap) a.pools.hbm_free[pp] = g; else st |= CASCADE_ST_EBOUNDS;
            hrow[j] = -1;
        }
    }
    if (st) atomicOr(a.status, st);
}

// One warp per admitted request: pop HBM ids for its restored and newly computed blocks, fill the
// restore list and the HBM table.
__global__ void __launch_bounds__(256)
apply_admitted_kernel(const __grid_constant__ PlanArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const int na = a.scalars[PS_N_ADMIT];
    const long long top = (long long)a.scalars[PS_HBM_CNT0] + a.scalars[PS_TOTAL_FREED];
    uint32_t st = 0;
    for (int i = warp; i < na; i += n_warps) {
        const int4 it = a.work_admit[i];
        const int slot = it.x;
        const int x1 = it.w >> 18, need = it.w & 0x3ffff;
        const int n0 = a.n0[slot];
        int32_t *hrow = a.pools.hbm_tbl + (size_t)slot * a.pools.maxb;
        const int32_t *orow = a.pools.host_tbl + (size_t)slot * a.pools.maxb;
        for (int jj = lane; jj < need; jj += 32) {
            const int j = n0 + jj;
            if (j >= a.pools.maxb) break;
            const long long pp = top - 1 - ((long long)it.y + jj);
            int32_t g = -1;
            if (pp >= 0 && pp < a.pools.hbm_free_cap) g = a.pools.hbm_free[pp]; else st |= CASCADE_ST_EBOUNDS;
            if (jj < x1) {
                const long long e = (long long)it.z + jj;
                if (e < a.plan.restore_cap) {
                    a.plan.restore_src[e] = orow[j];
                    a.plan.restore_dst[e] = g;
                } else {
                    st |= CASCADE_ST_ELISTCAP;
                }
            }
            hrow[j] = g;
        }
    }
    if (st) atomicOr(a.status, st);
}



template <int T, int K>
cudaError_t launch_plan(const cascade_params &p, const PlanArgs &a, int cluster_size, bool pdl, int device,
                        cudaStream_t stream) {
    // clusters of 16 CTAs need the non-portable size opt-in, once per device
    static CascadeDeviceOnce configured;
    if (!configured.is_set(device)) {
        cudaError_t e = cudaFuncSetAttribute(plan_kernel<T, K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured.set(device);
    }
    return cascade_launch(pdl, cluster_size, dim3(cluster_size), dim3(T), 0, stream, plan_kernel<T, K>, p, a);
}

template <int T>
cudaError_t launch_plan_k(int K, const cascade_params &p, const PlanArgs &a, int C, bool pdl, int device,
                          cudaStream_t s) {
    switch (K) {
        case 1: return launch_plan<T, 1>(p, a, C, pdl, device, s);
        case 2: return launch_plan<T, 2>(p, a, C, pdl, device, s);
        case 4: return launch_plan<T, 4>(p, a, C, pdl, device, s);
        default: return launch_plan<T, 8>(p, a, C, pdl, device, s);
    }
}

}  // namespace

extern "C" int cascade_tier_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget,
                                 const uint32_t *order, int32_t *grant, int n, int32_t D_act, int64_t K_act,
                                 const cascade_pools *pools, const cascade_plan *plan_out, void *stream) {
    CascadeRange nvtx_range("cascade_tier_plan");
    if (!ctx || !r || !pools || !plan_out || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (!plan_out->counts || !pools->hbm_free_count || !pools->host_free_count) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    const bool with_tables = pools->hbm_tbl != nullptr;
    if (n > 0 && (!budget || !order || !grant || !r->prompt || !r->n0 || !r->n1 || !r->n2 || !r->flags ||
                  !plan_out->x1 || !plan_out->x2 || !plan_out->tokens_run || !plan_out->action))
        return CASCADE_EINVAL;
    if (with_tables) {
        if (!pools->host_tbl || !pools->hbm_free || !pools->host_free || pools->maxb < 1 || pools->hbm_free_cap < 0 ||
            pools->host_free_cap < 0 || plan_out->restore_cap < 0 || plan_out->evict_cap < 0)
            return CASCADE_EINVAL;
        if ((plan_out->restore_cap > 0 && (!plan_out->restore_src || !plan_out->restore_dst)) ||
            (plan_out->evict_cap > 0 && (!plan_out->evict_src || !plan_out->evict_dst)))
            return CASCADE_EINVAL;
    }
    cudaStream_t s = (cudaStream_t)stream;
    PlanArgs a;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.flags = r->flags;
    a.budget = budget;
    a.order = order;
    a.grant = grant;
    a.pools = *pools;
    a.plan = *plan_out;
    a.pack = ctx->pack_by_slot;
    a.work_admit = ctx->work_admit;
    a.work_victim = ctx->work_victim;
    a.scalars = ctx->plan_scalars;
    a.status = ctx->status_dev;
    a.A_act = make_load_consts(ctx->params, D_act, K_act).A_act;
    a.n = n;
    a.with_tables = with_tables ? 1 : 0;
    a.prepared = 0;
    int T, C, K;
    if (!cascade_pick_geometry(ctx, n > 0 ? n : 1, &T, &C, &K)) return CASCADE_EINVAL;
    if (n > ctx->plan_prepare_min) {
        a.prepared = 1;
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((n + 255) / 256), dim3(256), 0, s, plan_prepare_kernel,
                                             ctx->params, a));
    }
    cudaError_t e = T == 256 ? launch_plan_k<256>(K, ctx->params, a, C, ctx->pdl, ctx->device, s)
                             : launch_plan_k<512>(K, ctx->params, a, C, ctx->pdl, ctx->device, s);
    CASCADE_CUDA_TRY(ctx, e);
    if (with_tables && n > 0) {
        const int grid = ctx->num_sms * 2;
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(256), 0, s, apply_victims_kernel, a));
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(256), 0, s, apply_admitted_kernel, a));
    }
    return CASCADE_OK;
}

// ---------------------------------------------------------------------------------------------
// cascade_tier_plan_noalloc: the tier plan for callers that must not allocate.
//
// cascade_tier_plan hands per-request offsets from its first kernel to the two table-rewrite
// kernels through scratch that cascade_create obtained with cudaMalloc.  Some users of this
// library cannot make that call at all: a serving engine that has already given every free byte
// of HBM to its KV block pool (a later cudaMalloc can fail or force the pool to shrink), a
// plug-in that runs under a host framework's memory manager and is not allowed to go to the
// driver allocator behind its back, or a loop that may not tolerate the device-wide
// synchronisation an allocation can imply.  For them the same kernels run here on a fixed
// scratch area that is part of the library image: a file-scope device array, present on every GPU
// that loads the library from load until exit, sized for CASCADE_NOALLOC_MAX_REQUESTS requests.
//
// The array's name is only a host-side handle in host code, never a device address, so its
// address is looked up once per device with cudaGetSymbolAddress (with that device current) and
// the resulting pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------
namespace {

struct NoAllocScratch {
    unsigned long long pack[CASCADE_NOALLOC_MAX_REQUESTS];
    int4 work_admit[CASCADE_NOALLOC_MAX_REQUESTS];
    int4 work_victim[CASCADE_NOALLOC_MAX_REQUESTS];
    int32_t scalars[PS_COUNT];
};

// ~320 KiB + a few scalars per GPU; shared by every call on that GPU
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

struct NoAllocDevice {
    NoAllocScratch *scratch;  // device address of g_noalloc_scratch on this device
    int num_sms;
    int max_cluster;          // largest cluster this device co-schedules for the plan geometry
    std::atomic<int> ready;   // published last, with release ordering
};
NoAllocDevice g_noalloc_dev[64];
std::mutex g_noalloc_mutex;   // serialises the first use on a device between host threads

// First use on a device (that device current): resolve the device address of the static array and
// query what the geometry needs.  Queries only; nothing is allocated.
int noalloc_setup(int device, NoAllocDevice **out) {
    if (device < 0 || device >= 64) return CASCADE_EINVAL;
    NoAllocDevice &d = g_noalloc_dev[device];
    if (!d.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!d.ready.load(std::memory_order_relaxed)) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
                cudaGetLastError();
                return CASCADE_ECUDA;
            }
            if (cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
                cudaGetLastError();
                return CASCADE_ECUDA;
            }
            d.max_cluster = cascade_probe_max_cluster();
            const char *e = getenv("CASCADE_MAX_CLUSTER");   // lower it to exercise the fallback geometry
            if (e && atoi(e) > 0 && atoi(e) < d.max_cluster) d.max_cluster = atoi(e);
            d.scratch = reinterpret_cast<NoAllocScratch *>(ptr);
            d.ready.store(1, std::memory_order_release);
        }
    }
    *out = &d;
    return CASCADE_OK;
}

}  // namespace

extern "C" int cascade_tier_plan_noalloc(const cascade_params *p, const cascade_reqs *r, const int64_t *budget,
                                         const uint32_t *order, int32_t *grant, int n, int32_t D_act, int64_t K_act,
                                         const cascade_pools *pools, const cascade_plan *plan_out,
                                         uint32_t *status_dev, void *stream) {
    CascadeRange nvtx_range("cascade_tier_plan_noalloc");
    if (!p || !r || !pools || !plan_out || !status_dev || n < 0) return CASCADE_EINVAL;
    if (n > CASCADE_NOALLOC_MAX_REQUESTS) return CASCADE_ETOOBIG;  // beyond the fixed scratch
    int rc = cascade_validate_params(p);
    if (rc != CASCADE_OK) return rc;
    if (!plan_out->counts || !pools->hbm_free_count || !pools->host_free_count) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    const bool with_tables = pools->hbm_tbl != nullptr;
    if (n > 0 && (!budget || !order || !grant || !r->prompt || !r->n0 || !r->n1 || !r->n2 || !r->flags ||
                  !plan_out->x1 || !plan_out->x2 || !plan_out->tokens_run || !plan_out->action))
        return CASCADE_EINVAL;
    if (with_tables) {
        if (!pools->host_tbl || !pools->hbm_free || !pools->host_free || pools->maxb < 1 || pools->hbm_free_cap < 0 ||
            pools->host_free_cap < 0 || plan_out->restore_cap < 0 || plan_out->evict_cap < 0)
            return CASCADE_EINVAL;
        if ((plan_out->restore_cap > 0 && (!plan_out->restore_src || !plan_out->restore_dst)) ||
            (plan_out->evict_cap > 0 && (!plan_out->evict_src || !plan_out->evict_dst)))
            return CASCADE_EINVAL;
    }
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return CASCADE_ECUDA;
    NoAllocDevice *dev = nullptr;
    rc = noalloc_setup(device, &dev);
    if (rc != CASCADE_OK) return rc;

    cudaStream_t s = (cudaStream_t)stream;
    PlanArgs a;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.flags = r->flags;
    a.budget = budget;
    a.order = order;
    a.grant = grant;
    a.pools = *pools;
    a.plan = *plan_out;
    a.pack = dev->scratch->pack;
    a.work_admit = dev->scratch->work_admit;
    a.work_victim = dev->scratch->work_victim;
    a.scalars = dev->scratch->scalars;
    a.status = status_dev;
    a.A_act = make_load_consts(*p, D_act, K_act).A_act;
    a.n = n;
    a.with_tables = with_tables ? 1 : 0;
    a.prepared = 0;
    // The scalars are rewritten by every call before the rewrite kernels read them and only the
    // work entries written by this call are read back, so nothing has to be cleared; they are
    // zeroed anyway so that a call that launches nothing leaves no stale counts behind.
    if (cudaMemsetAsync(dev->scratch->scalars, 0, sizeof(dev->scratch->scalars), s) != cudaSuccess)
        return CASCADE_ECUDA;
    // same geometry rule as cascade_tier_plan: a device that co-schedules fewer than 16 CTAs gets a
    // smaller cluster with more requests per thread
    cascade_ctx geo = {};
    geo.max_cluster = dev->max_cluster;
    int T, C, K;
    if (!cascade_pick_geometry(&geo, n > 0 ? n : 1, &T, &C, &K)) return CASCADE_ETOOBIG;
    cudaError_t e = T == 256 ? launch_plan_k<256>(K, *p, a, C, false, device, s)
                             : launch_plan_k<512>(K, *p, a, C, false, device, s);
    if (e != cudaSuccess) {
        cudaGetLastError();  // leave no stale error behind for the caller's next runtime call
        return CASCADE_ECUDA;
    }
    if (with_tables && n > 0) {
        const int grid = dev->num_sms * 2;
        apply_victims_kernel<<<grid, 256, 0, s>>>(a);
        if (cudaGetLastError() != cudaSuccess) return CASCADE_ECUDA;
        apply_admitted_kernel<<<grid, 256, 0, s>>>(a);
        if (cudaGetLastError() != cudaSuccess) return CASCADE_ECUDA;
    }
    return CASCADE_OK;
}
