// cascade_tier_plan: restore bound (Eq. 7), restore-vs-recompute choice, HBM capacity check,
// preemption victims with their disposition (Algorithm 1), and deterministic block-id allocation.
//
// Kernel 1 (one CTA of 1024 threads): a per-request phase in slot order (coalesced SoA loads, the
// only int64 divisions of the path, at most two per admitted request), then two block-wide scans
// over the schedule order - a forward scan over the admitted set (cumulative HBM need, restore-list
// offsets) and a backward scan over the preemptable holders (freed-block and evict-list offsets).
// The sequential "pop one request at a time / preempt the largest budget" loops of Algorithm 1
// become prefix sums because admitted requests and victims are prefixes of the order walked
// forwards and backwards.
// Kernels 2 and 3 (many CTAs, one warp per request): rewrite block tables, free lists and the two
// copy lists from the offsets kernel 1 left in scratch; pushes of freed ids (kernel 2) finish
// before any pop (kernel 3).  In plan-only mode (no tables) only kernel 1 runs.
#include "common.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;

// decision word: n0 (14 bits) | x1 (14) | tokens_run (18) | flags
constexpr int kX1Shift = 14, kRunShift = 28;
constexpr unsigned long long kAdm = 1ull << 46, kPriv = 1ull << 47, kFits = 1ull << 48, kValid = 1ull << 49;

struct PlanArgs {
    const int32_t *prompt, *n0, *n1, *n2;
    const uint8_t *flags;
    const int64_t *budget;
    const uint32_t *order;
    int32_t *grant;
    cascade_pools pools;
    cascade_plan plan;
    uint64_t *pack_by_slot, *pack_sorted;
    int4 *work_admit, *work_victim;
    int32_t *scalars;
    uint32_t *status;
    int64_t A_act;
    int n;
    int with_tables;
};

__device__ __forceinline__ int unpack_n0(unsigned long long w) { return int(w & 0x3fff); }
__device__ __forceinline__ int unpack_x1(unsigned long long w) { return int((w >> kX1Shift) & 0x3fff); }
__device__ __forceinline__ int unpack_run(unsigned long long w) { return int((w >> kRunShift) & 0x3ffff); }

// Block-wide exclusive scan of three int32 partials (one per thread); totals returned in tot[3].
__device__ void block_scan3(int &a, int &b, int &c, int *tot, int (*ws)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int ia = a, ib = b, ic = c;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        int ta = __shfl_up_sync(kFull, ia, s), tb = __shfl_up_sync(kFull, ib, s), tc = __shfl_up_sync(kFull, ic, s);
        if (lane >= s) { ia += ta; ib += tb; ic += tc; }
    }
    if (lane == 31) { ws[warp][0] = ia; ws[warp][1] = ib; ws[warp][2] = ic; }
    __syncthreads();
    if (warp == 0) {
        int va = ws[lane][0], vb = ws[lane][1], vc = ws[lane][2];
        int ja = va, jb = vb, jc = vc;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            int ta = __shfl_up_sync(kFull, ja, s), tb = __shfl_up_sync(kFull, jb, s), tc = __shfl_up_sync(kFull, jc, s);
            if (lane >= s) { ja += ta; jb += tb; jc += tc; }
        }
        ws[lane][0] = ja - va; ws[lane][1] = jb - vb; ws[lane][2] = jc - vc;
        if (lane == 31) { ws[kWarps][0] = ja; ws[kWarps][1] = jb; ws[kWarps][2] = jc; }
    }
    __syncthreads();
    a = ws[warp][0] + ia - a;
    b = ws[warp][1] + ib - b;
    c = ws[warp][2] + ic - c;
    tot[0] = ws[kWarps][0]; tot[1] = ws[kWarps][1]; tot[2] = ws[kWarps][2];
    __syncthreads();
}

// Block-wide sum of up to six int64 partials; every thread gets the totals.
template <int M>
__device__ void block_sum(long long (&v)[M], long long (*ws)[6]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) v[m] += __shfl_xor_sync(kFull, v[m], s);
    if (lane == 0)
        for (int m = 0; m < M; ++m) ws[warp][m] = v[m];
    __syncthreads();
#pragma unroll
    for (int m = 0; m < M; ++m) {
        long long t = ws[lane][m];
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) t += __shfl_xor_sync(kFull, t, s);
        v[m] = t;
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads, 1)
plan_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ PlanArgs a) {
    __shared__ int ws3[kWarps + 1][3];
    __shared__ long long ws6[kWarps][6];
    const int tid = threadIdx.x;
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

    // ---- phase 1, slot order: Eq. 7 bounds and the restore-vs-recompute choice ------------------
    for (int r = tid; r < n; r += kThreads) {
        const long long P = a.prompt[r], n0 = a.n0[r], n1 = a.n1[r], n2 = a.n2[r];
        const long long b = a.budget[r];
        const int g = a.grant[r];
        bool valid = dev_request_valid(bt, P, n0, n1, n2);
        if (valid && a.with_tables) valid = (P + bt - 1) / bt <= a.pools.maxb;
        unsigned long long w = 0;
        int x1 = 0, x2 = 0, run = 0;
        if (!valid) {
            st |= CASCADE_ST_EPRECOND;
            if (g != 0) a.grant[r] = 0;
        } else {
            w = kValid | (unsigned long long)n0;
            if (a.flags[r] & CASCADE_FLAG_HBM_PRIVATE) w |= kPriv;
            if (dev_restore_time(p, 1, n0) <= b) w |= kFits;
            if (g > 0) {
                const long long rem = b > 0 ? b : 0;
                // Eq. 7, host tier first
                long long x1max = 0;
                if (n1 > 0) {
                    long long head = rem - p.delta_ns[1];
                    if (head < 0) head = 0;
                    x1max = head / p.blk_ns[1];
                    if (x1max > n1) x1max = n1;
                }
                // deep tier from what is left, only behind a fully restored host segment
                long long x2max = 0;
                if (x1max == n1 && n2 > 0) {
                    long long head = rem - dev_restore_time(p, 1, n1) - p.delta_ns[2];
                    if (head < 0) head = 0;
                    x2max = head / p.blk_ns[2];
                    if (x2max > n2) x2max = n2;
                }
                // smallest predicted completion time; ties restore more
                long long bx1 = 0, bx2 = 0;
                long long bF = dev_comp_q(a.A_act, p.c_attn_q20, P, n0 * bt);
                if (x1max > 0) {
                    const long long F = (dev_restore_time(p, 1, x1max) << 20) +
                                        dev_comp_q(a.A_act, p.c_attn_q20, P, (n0 + x1max) * bt);
                    if (F <= bF) { bF = F; bx1 = x1max; }
                }
                if (x2max > 0) {
                    const long long F = ((dev_restore_time(p, 1, n1) + dev_restore_time(p, 2, x2max)) << 20) +
                                        dev_comp_q(a.A_act, p.c_attn_q20, P, (n0 + n1 + x2max) * bt);
                    if (F <= bF) { bF = F; bx1 = n1; bx2 = x2max; }
                }
                x1 = (int)bx1;
                x2 = (int)bx2;
                // a deep fetch is staged first: nothing runs now, HBM is taken at the last hop only
                const long long left = P - (n0 + bx1) * bt;
                run = bx2 > 0 ? 0 : (int)(g < left ? g : left);
                w |= kAdm | ((unsigned long long)x1 << kX1Shift) | ((unsigned long long)run << kRunShift);
            }
        }
        a.pack_by_slot[r] = w;
        a.plan.x1[r] = x1;
        a.plan.x2[r] = x2;
        a.plan.tokens_run[r] = run;
    }
    __syncthreads();

    // ---- phase 2a, forward over the order: HBM capacity and offsets of the admitted set ---------
    const int ipt = (n + kThreads - 1) / kThreads;
    const int lo = min(n, tid * ipt), hi = min(n, lo + ipt);
    int t_need = 0, t_x1 = 0, t_cnt = 0;
    long long t_evictable = 0;
    for (int q = lo; q < hi; ++q) {
        const unsigned long long w = a.pack_by_slot[a.order[q]];
        a.pack_sorted[q] = w;
        if (w & kValid) {
            if (w & kAdm) {
                const int x1 = unpack_x1(w);
                t_need += x1 + (unpack_run(w) + bt - 1) / bt;
                t_x1 += x1;
                ++t_cnt;
            } else if (w & kPriv) {
                t_evictable += unpack_n0(w);
            }
        }
    }
    int tot3[3];
    block_scan3(t_need, t_x1, t_cnt, tot3, ws3);
    long long red1[1] = {t_evictable};
    block_sum<1>(red1, ws6);
    const long long cap = hbm_cnt + red1[0];

    long long s_need = 0, s_adm = 0, s_tok = 0, s_unadm = 0, s_rest = 0;
    {
        long long c = t_need;
        int rx = t_x1, ci = t_cnt;
        for (int q = lo; q < hi; ++q) {
            unsigned long long w = a.pack_sorted[q];
            if ((w & kValid) && (w & kAdm)) {
                const int x1 = unpack_x1(w), run = unpack_run(w);
                const int nd = x1 + (run + bt - 1) / bt;
                c += nd;
                const uint32_t slot = a.order[q];
                if (c > cap) {
                    // HBM cannot hold it even after preempting everything preemptable: cut from the tail
                    a.grant[slot] = 0;
                    a.plan.x1[slot] = 0;
                    a.plan.x2[slot] = 0;
                    a.plan.tokens_run[slot] = 0;
                    a.pack_sorted[q] = w & (kValid | kPriv | kFits | 0x3fffull);
                    ++s_unadm;
                    st |= CASCADE_ST_ENOSPC;
                } else {
                    s_need += nd;
                    ++s_adm;
                    s_tok += run;
                    s_rest += x1;
                    a.work_admit[ci] = make_int4((int)slot, (int)(c - nd), rx, (x1 << 18) | nd);
                }
                rx += x1;
                ++ci;
            }
        }
    }
    long long red5[5] = {s_need, s_adm, s_tok, s_unadm, s_rest};
    block_sum<5>(red5, ws6);  // also orders the pack_sorted rewrites before phase 2b reads them
    const long long need_total = red5[0];
    long long deficit = need_total - hbm_cnt;
    if (deficit < 0) deficit = 0;

    // ---- phase 2b, backward over the order: victims and their disposition -----------------------
    int t_v = 0, t_h = 0, t_c = 0;
    for (int q = lo; q < hi; ++q) {
        const unsigned long long w = a.pack_sorted[n - 1 - q];
        if ((w & kValid) && !(w & kAdm) && (w & kPriv)) {
            const int n0 = unpack_n0(w);
            if (n0 > 0) {
                t_v += n0;
                ++t_c;
                if (w & kFits) t_h += n0;
            }
        }
    }
    block_scan3(t_v, t_h, t_c, tot3, ws3);
    long long s_nv = 0, s_freed = 0, s_nev = 0;
    {
        long long v = t_v, h = t_h;
        int ci = t_c;
        for (int q = lo; q < hi; ++q) {
            const int pos = n - 1 - q;
            const unsigned long long w = a.pack_sorted[pos];
            const uint32_t slot = a.order[pos];
            uint8_t act = CASCADE_ACT_NONE;
            if (w & kValid) {
                const int n0 = unpack_n0(w);
                const bool elig = !(w & kAdm) && (w & kPriv) && n0 > 0;
                if (elig && v < deficit) {
                    // spill only if it can be brought back within the victim's own budget and host has room
                    const bool ev = (w & kFits) && (h + n0 <= host_cnt);
                    act = ev ? CASCADE_ACT_EVICT : CASCADE_ACT_DROP;
                    a.work_victim[ci] = make_int4((int)slot, (int)v, (int)h, (int)act);
                    ++s_nv;
                    s_freed += n0;
                    if (ev) s_nev += n0;
                } else if (n0 > 0) {
                    act = CASCADE_ACT_RETAIN;
                }
                if (elig) {
                    v += n0;
                    ++ci;
                    if (w & kFits) h += n0;
                }
            }
            a.plan.action[slot] = act;
        }
    }
    long long red3[3] = {s_nv, s_freed, s_nev};
    block_sum<3>(red3, ws6);

    st = __reduce_or_sync(kFull, st);
    if ((tid & 31) == 0 && st) atomicOr(a.status, st);
    if (tid == 0) {
        const long long freed = red3[1], nev = red3[2];
        cascade_plan_counts *c = a.plan.counts;
        c->n_restore = (int)red5[4];
        c->n_evict = (int)nev;
        c->n_drop_blocks = (int)(freed - nev);
        c->n_victims = (int)red3[0];
        c->n_unadmitted = (int)red5[3];
        c->n_admitted = (int)red5[1];
        c->hbm_need = (int)need_total;
        c->deficit = (int)deficit;
        c->hbm_free_after = (int)(hbm_cnt + freed - need_total);
        c->host_free_after = (int)(host_cnt - nev);
        c->tokens_run = red5[2];
        a.scalars[PS_N_ADMIT] = (int)red5[1];
        a.scalars[PS_N_VICTIM] = (int)red3[0];
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

}  // namespace

extern "C" int cascade_tier_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget,
                                 const uint32_t *order, int32_t *grant, int n, int32_t D_act, int64_t K_act,
                                 const cascade_pools *pools, const cascade_plan *plan_out, void *stream) {
    if (!ctx || !r || !pools || !plan_out || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
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
    a.pack_by_slot = ctx->pack_by_slot;
    a.pack_sorted = ctx->pack_sorted;
    a.work_admit = ctx->work_admit;
    a.work_victim = ctx->work_victim;
    a.scalars = ctx->plan_scalars;
    a.status = ctx->status_dev;
    a.A_act = make_load_consts(ctx->params, D_act, K_act).A_act;
    a.n = n;
    a.with_tables = with_tables ? 1 : 0;
    plan_kernel<<<1, kThreads, 0, s>>>(ctx->params, a);
    CASCADE_CUDA_TRY(ctx, cudaGetLastError());
    if (with_tables && n > 0) {
        const int grid = ctx->num_sms * 2;
        apply_victims_kernel<<<grid, 256, 0, s>>>(a);
        CASCADE_CUDA_TRY(ctx, cudaGetLastError());
        apply_admitted_kernel<<<grid, 256, 0, s>>>(a);
        CASCADE_CUDA_TRY(ctx, cudaGetLastError());
    }
    return CASCADE_OK;
}
