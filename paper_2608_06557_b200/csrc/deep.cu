// Deep tier as a real stage, and one copy per shared block.
//
// cascade_stage_plan: first hop of the two-hop path P(2) of Eq. 6 (deep tier -> host DRAM).  Walking
// the order with a running link-time and host-room allowance is a clamped scan, as in the prefetch
// plan: every request before the first one that is cut gets its full choice, the cut one gets what
// is left, nothing behind it gets anything.
//   kernel 1 (thread-block cluster): gather through `order`, each request's own restore choice,
//            prefix sums of hop time / blocks / requests, one exchange of CTA totals through
//            distributed shared memory;
//   kernel 2 (one warp per served request): pop host records, fill the stage list and the host table.
//
// cascade_dedup: one copy per distinct source block of a copy list.  Source ids are dense pool
// indices, so the first occurrence of every id is found with a direct-address table and atomicMin
// (linear work, no sort, result independent of thread order):
//   kernel 1  table[s] = {first: INT_MAX, count: 0} for every id in the list
//   kernel 2  atomicMin(first[s], i), atomicAdd(count[s], 1)
//   kernel 3  per 1024-entry tile: number of kept entries; per slot: table cells -> kept destination
//   kernel 4  per tile: offset from the tile counts, compaction into the output list, surplus ids
//             pushed on the free list, share counts
// Nothing waits on another CTA: every dependency is a kernel boundary.
#include <cooperative_groups.h>

#include "cluster_scan.cuh"
#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kMaxCluster = 16;

// ---------------------------------------------------------------------------------------------------
// stage plan
// ---------------------------------------------------------------------------------------------------
struct StageArgs {
    const int32_t *prompt, *n0, *n1, *n2;
    const int64_t *budget;
    const uint32_t *order;
    const uint8_t *action;
    cascade_pools pools;
    cascade_stage stage;
    int4 *work;
    int32_t *scalars;
    uint32_t *status;
    int64_t A_act;
    int64_t link_budget_ns;
    int64_t hop_delta, hop_blk;
    int host_reserve;
    int n;
    int with_tables;
};

struct __align__(16) StExch1 {
    long long time;
    int blocks, count;
};
struct __align__(16) StExch2 {
    long long used;
    int n_stage, n_req, n_short, pad;
};

__device__ __forceinline__ long long hop_time(const StageArgs &a, long long x) {
    return x == 0 ? 0 : a.hop_delta + x * a.hop_blk;
}

template <int T, int K>
__global__ void __launch_bounds__(T, 1)
stage_kernel(const __grid_constant__ cascade_params p, const __grid_constant__ StageArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int per = T * K;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();
    __shared__ int ws3[33][3];
    __shared__ long long ws8[33][8];
    __shared__ StExch1 ex1[kMaxCluster];
    __shared__ StExch2 ex2[kMaxCluster];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n;
    const int bt = p.bt;
    uint32_t st = 0;
    // "I have started": waited for in front of the first store into another CTA's shared memory (which must exist by
    // then); the barrier's latency hides behind the per-request work
    cluster.barrier_arrive();

    long long host_cnt = *a.pools.host_free_count;
    if (a.with_tables && (host_cnt < 0 || host_cnt > a.pools.host_free_cap)) {
        st |= CASCADE_ST_EBOUNDS;
        host_cnt = host_cnt < 0 ? 0 : a.pools.host_free_cap;
    }

    // ---- per request: does its own choice contain a deep fetch ----------------------------------
    uint32_t slot[K];
    int mv[K], cv[K], zero[K];
    long long tv[K];
    bool real[K];
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
        const long long n2 = a.n2[r];
        if (n2 <= 0) {
            // still has to be a request the plan accepts, but it stages nothing either way
            continue;
        }
        const long long P = a.prompt[r], n0 = a.n0[r], n1 = a.n1[r];
        bool valid = dev_request_valid(bt, P, n0, n1, n2);
        if (valid && a.with_tables) valid = (P + bt - 1) / bt <= a.pools.maxb;
        if (!valid) continue;
        const unsigned act = a.action[r];
        if (act == CASCADE_ACT_EVICT || act == CASCADE_ACT_DROP) continue;
        int64_t x1, x2;
        dev_choose_restore(p, a.A_act, P, n0, n1, n2, a.budget[r], &x1, &x2);
        if (x2 > 0) {
            mv[k] = (int)x2;
            cv[k] = 1;
            tv[k] = hop_time(a, x2);
        }
    }

    // ---- prefix sums over the order, one exchange ------------------------------------------------
    int want[K];
#pragma unroll
    for (int k = 0; k < K; ++k) want[k] = mv[k];
    int tot[3];
    cta_scan3<T, K>(mv, cv, zero, tot, ws3);               // mv, cv now inclusive
    const long long t_total = cta_scan_ll<T, K>(tv, &ws8[0][0]);
    cluster.barrier_wait();
    if (tid < csize) {
        StExch1 x;
        x.time = t_total;
        x.blocks = tot[0];
        x.count = tot[1];
        cluster.map_shared_rank(ex1, tid)[crank] = x;
    }
    cluster.sync();
    long long off_t = 0;
    int off_b = 0, off_c = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < crank && c < csize) {
            const StExch1 x = ex1[c];
            off_t += x.time;
            off_b += x.blocks;
            off_c += x.count;
        }
    }
    const long long link0 = a.link_budget_ns;
    const long long room0 = host_cnt - a.host_reserve;
    long long s_stage = 0, s_req = 0, s_short = 0, s_used = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (!real[k]) continue;
        int b = 0;
        if (want[k] > 0) {
            const long long m = want[k];
            const long long e_t = off_t + tv[k] - hop_time(a, m);   // exclusive
            const long long e_b = (long long)off_b + mv[k] - m;
            const long long left = link0 - e_t;
            const long long by_link = left > a.hop_delta ? (left - a.hop_delta) / a.hop_blk : 0;
            long long by_room = room0 - e_b;
            if (by_room < 0) by_room = 0;
            long long bb = m < by_link ? m : by_link;
            if (by_room < bb) bb = by_room;
            b = (int)bb;
            if (b < m) ++s_short;
            if (b > 0) {
                // every served request before this one got its full choice, so the exclusive sums are exact
                a.work[off_c + cv[k] - 1] = make_int4((int)slot[k], (int)e_b, (int)e_b, b);
                s_stage += b;
                s_used += hop_time(a, b);
                ++s_req;
            }
        }
        a.stage.staged[slot[k]] = b;
    }
    long long red[4] = {s_stage, s_req, s_short, s_used};
    cta_sum<T, 4>(red, ws8);
    if (tid == 0) {
        StExch2 x;
        x.used = red[3];
        x.n_stage = (int)red[0];
        x.n_req = (int)red[1];
        x.n_short = (int)red[2];
        x.pad = 0;
        cluster.map_shared_rank(ex2, 0)[crank] = x;
    }
    st = __reduce_or_sync(kFull, st);
    if (lane == 0 && st) atomicOr(a.status, st);
    cluster.sync();
    if (crank == 0 && tid == 0) {
        int n_stage = 0, n_req = 0, n_short = 0;
        long long used = 0;
        for (unsigned c = 0; c < csize; ++c) {
            n_stage += ex2[c].n_stage;
            n_req += ex2[c].n_req;
            n_short += ex2[c].n_short;
            used += ex2[c].used;
        }
        cascade_stage_counts out;
        out.n_stage = n_stage;
        out.n_requests = n_req;
        out.n_short = n_short;
        out.host_free_after = (int)(host_cnt - n_stage);
        out.link_ns_left = link0 - used;
        *a.stage.counts = out;
        a.scalars[PS_N_ADMIT] = n_req;
        a.scalars[PS_HOST_CNT0] = (int)host_cnt;
        if (a.with_tables) *a.pools.host_free_count = (int)(host_cnt - n_stage);
    }
}

__global__ void __launch_bounds__(256) apply_stage_kernel(const __grid_constant__ StageArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const int n_items = a.scalars[PS_N_ADMIT];
    const long long top = a.scalars[PS_HOST_CNT0];
    uint32_t st = 0;
    for (int i = warp; i < n_items; i += n_warps) {
        const int4 it = a.work[i];
        const int slot = it.x;
        const int lo = a.n0[slot] + a.n1[slot];
        int32_t *orow = a.pools.host_tbl + (size_t)slot * a.pools.maxb;
        const int32_t *drow = a.stage.deep_tbl + (size_t)slot * a.pools.maxb;
        for (int jj = lane; jj < it.w; jj += 32) {
            const int j = lo + jj;
            if (j >= a.pools.maxb) break;
            const long long pp = top - 1 - ((long long)it.y + jj);
            int32_t rec = -1;
            if (pp >= 0 && pp < a.pools.host_free_cap) rec = a.pools.host_free[pp]; else st |= CASCADE_ST_EBOUNDS;
            const long long e = (long long)it.z + jj;
            if (e < a.stage.stage_cap) {
                a.stage.stage_src[e] = drow[j];
                a.stage.stage_dst[e] = rec;
            } else {
                st |= CASCADE_ST_ELISTCAP;
            }
            orow[j] = rec;
        }
    }
    if (st) atomicOr(a.status, st);
}

template <int T, int K>
cudaError_t launch_stage(const cascade_params &p, const StageArgs &a, int cluster_size, bool pdl, cudaStream_t stream) {
    static CascadeDeviceOnce configured;
    int device = 0;
    cudaGetDevice(&device);
    if (!configured.is_set(device)) {
        cudaError_t e = cudaFuncSetAttribute(stage_kernel<T, K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured.set(device);
    }
    return cascade_launch(pdl, cluster_size, dim3(cluster_size), dim3(T), 0, stream, stage_kernel<T, K>, p, a);
}

template <int T>
cudaError_t launch_stage_k(int K, const cascade_params &p, const StageArgs &a, int C, bool pdl, cudaStream_t s) {
    switch (K) {
        case 1: return launch_stage<T, 1>(p, a, C, pdl, s);
        case 2: return launch_stage<T, 2>(p, a, C, pdl, s);
        case 4: return launch_stage<T, 4>(p, a, C, pdl, s);
        default: return launch_stage<T, 8>(p, a, C, pdl, s);
    }
}

// ---------------------------------------------------------------------------------------------------
// one copy per distinct source block
// ---------------------------------------------------------------------------------------------------
constexpr int kDdThreads = 256;
constexpr int kDdRounds = 4;
constexpr int kDdTile = kDdThreads * kDdRounds;   // list entries per CTA
constexpr int kIntMax = 0x7fffffff;

struct DedupArgs {
    cascade_dedup_args u;
    int32_t *first;       // [n_src_ids] smallest list position holding the id
    int32_t *count;       // [n_src_ids] entries holding the id
    int32_t *tile_kept;   // [n_tiles]
    int32_t *sc;          // scalars: [0] list length, [1] free count at entry
    uint32_t *status;
    int n;
    int n_tiles;
};

__device__ __forceinline__ int dd_list_len(const DedupArgs &a) {
    long long m = *a.u.list_count;
    if (m < 0) m = 0;
    if (m > a.u.list_cap) m = a.u.list_cap;
    return (int)m;
}

__device__ __forceinline__ bool dd_entry_valid(const DedupArgs &a, int s, int d) {
    return s >= 0 && s < a.u.n_src_ids && d >= 0 && d < a.u.n_dst_ids;
}

__global__ void __launch_bounds__(kDdThreads) dedup_init_kernel(const __grid_constant__ DedupArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int m = dd_list_len(a);
    uint32_t st = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (*a.u.list_count < 0) st |= CASCADE_ST_EBOUNDS;
        long long f = *a.u.free_count;
        if (f < 0 || f > a.u.free_cap) {
            st |= CASCADE_ST_EBOUNDS;
            f = f < 0 ? 0 : a.u.free_cap;
        }
        a.sc[0] = m;
        a.sc[1] = (int)f;
        a.u.counts->n_shared_requests = 0;
        a.u.counts->max_share = 0;
    }
    for (long long i = (long long)blockIdx.x * kDdThreads + threadIdx.x; i < m; i += (long long)gridDim.x * kDdThreads) {
        const int s = a.u.list_src[i], d = a.u.list_dst[i];
        if (dd_entry_valid(a, s, d)) {
            a.first[s] = kIntMax;
            a.count[s] = 0;
        } else {
            st |= CASCADE_ST_EBOUNDS;
        }
    }
    if (st) atomicOr(a.status, st);
}

__global__ void __launch_bounds__(kDdThreads) dedup_mark_kernel(const __grid_constant__ DedupArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int m = a.sc[0];
    for (long long i = (long long)blockIdx.x * kDdThreads + threadIdx.x; i < m; i += (long long)gridDim.x * kDdThreads) {
        const int s = a.u.list_src[i], d = a.u.list_dst[i];
        if (dd_entry_valid(a, s, d)) {
            atomicMin(&a.first[s], (int)i);
            atomicAdd(&a.count[s], 1);
        }
    }
}

// blocks [0, n_tiles): kept entries per tile; the remaining blocks: one warp per slot rewrites its cells
__global__ void __launch_bounds__(kDdThreads) dedup_tables_kernel(const __grid_constant__ DedupArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int m = a.sc[0];
    if ((int)blockIdx.x < a.n_tiles) {
        const long long base = (long long)blockIdx.x * kDdTile;
        int kept = 0;
#pragma unroll
        for (int k = 0; k < kDdRounds; ++k) {
            const long long i = base + k * kDdThreads + threadIdx.x;
            int flag = 0;
            if (i < m) {
                const int s = a.u.list_src[i], d = a.u.list_dst[i];
                flag = !dd_entry_valid(a, s, d) || a.first[s] == (int)i;
            }
            kept += __syncthreads_count(flag);
        }
        if (threadIdx.x == 0) a.tile_kept[blockIdx.x] = kept;
        return;
    }
    const int lane = threadIdx.x & 31;
    const int warps_per_block = kDdThreads / 32;
    const long long warp0 = ((long long)blockIdx.x - a.n_tiles) * warps_per_block + (threadIdx.x >> 5);
    const long long n_warps = ((long long)gridDim.x - a.n_tiles) * warps_per_block;
    uint32_t st = 0;
    int n_shared = 0;
    for (long long r = warp0; r < a.n; r += n_warps) {
        const long long lo = (long long)a.u.lo_a[r] + (a.u.lo_b ? a.u.lo_b[r] : 0);
        const long long len = (long long)a.u.len_a[r] + (a.u.len_b ? a.u.len_b[r] : 0);
        int shared = 0;
        if (lo >= 0 && len > 0 && lo + len <= a.u.maxb) {
            const int32_t *srow = a.u.src_tbl + (size_t)r * a.u.maxb;
            int32_t *drow = a.u.dst_tbl + (size_t)r * a.u.maxb;
            for (long long j = lo + lane; j < lo + len; j += 32) {
                const int s = srow[j];
                if (s < 0 || s >= a.u.n_src_ids) continue;
                // a source id that is not in this call's list has a stale table entry: check it against the list
                const int h = a.first[s];
                if (h < 0 || h >= m || a.u.list_src[h] != s) continue;
                const int d = a.u.list_dst[h];
                if (d < 0 || d >= a.u.n_dst_ids) continue;
                drow[j] = d;
                if (a.count[s] > 1) shared = 1;
            }
        } else if (len > 0) {
            st |= CASCADE_ST_EPRECOND;
        }
        shared = __any_sync(kFull, shared);
        if (lane == 0) {
            a.u.shared[r] = (uint8_t)shared;
            n_shared += shared;
        }
    }
    if (lane == 0 && n_shared) atomicAdd(&a.u.counts->n_shared_requests, n_shared);
    if (st) atomicOr(a.status, st);
}

__global__ void __launch_bounds__(kDdThreads) dedup_compact_kernel(const __grid_constant__ DedupArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    __shared__ int red[kDdThreads / 32];
    __shared__ int wsum[kDdThreads / 32];
    const int m = a.sc[0];
    const long long fpos0 = a.sc[1];
    const int tile = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long base = (long long)tile * kDdTile;
    if (base >= m && !(tile == 0 && m == 0)) return;
    // kept entries in the tiles before this one
    int part = 0;
    for (int t = tid; t < tile; t += kDdThreads) part += a.tile_kept[t];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) part += __shfl_xor_sync(kFull, part, s);
    if (lane == 0) red[warp] = part;
    __syncthreads();
    int before = 0;
#pragma unroll
    for (int w = 0; w < kDdThreads / 32; ++w) before += red[w];
    uint32_t st = 0;
    int max_share = 0;
    int run = before;                       // kept entries before the current round
#pragma unroll
    for (int k = 0; k < kDdRounds; ++k) {
        const long long i = base + k * kDdThreads + tid;
        int s = -1, d = -1, flag = 0, valid = 0;
        if (i < m) {
            s = a.u.list_src[i];
            d = a.u.list_dst[i];
            valid = dd_entry_valid(a, s, d);
            flag = !valid || a.first[s] == (int)i;
        }
        const unsigned bal = __ballot_sync(kFull, flag);
        const int in_warp = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) wsum[warp] = __popc(bal);
        __syncthreads();
        int woff = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kDdThreads / 32; ++w) {
            const int v = wsum[w];
            if (w < warp) woff += v;
            total += v;
        }
        if (i < m) {
            const long long kept_before = (long long)run + woff + in_warp;
            if (flag) {
                a.u.out_src[kept_before] = s;
                a.u.out_dst[kept_before] = d;
                if (valid) {
                    const int c = a.count[s];
                    a.u.ref[d] = c;
                    max_share = max(max_share, c);
                }
            } else {
                const long long fp = fpos0 + (i - kept_before);
                if (fp < a.u.free_cap) a.u.free_list[fp] = d; else st |= CASCADE_ST_EBOUNDS;
            }
        }
        run += total;
        __syncthreads();
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) max_share = max(max_share, __shfl_xor_sync(kFull, max_share, s));
    if (lane == 0 && max_share) atomicMax(&a.u.counts->max_share, max_share);
    if (st) atomicOr(a.status, st);
    // the tile holding the last entry knows every total
    const bool last = (m == 0) ? tile == 0 : (base < m && m <= base + kDdTile);
    if (last && tid == 0) {
        const int n_unique = run;
        const int n_surplus = m - n_unique;
        a.u.counts->n_in = m;
        a.u.counts->n_unique = n_unique;
        a.u.counts->n_surplus = n_surplus;
        a.u.counts->free_after = (int)(fpos0 + n_surplus);
        *a.u.free_count = (int)(fpos0 + n_surplus);
    }
}

}  // namespace

extern "C" int cascade_stage_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget,
                                  const uint32_t *order, const uint8_t *action, int n, int32_t D_act, int64_t K_act,
                                  int64_t link_budget_ns, int32_t host_reserve, const cascade_pools *pools,
                                  const cascade_stage *stage, void *stream) {
    CascadeRange nvtx_range("cascade_stage_plan");
    if (!ctx || !r || !pools || !stage || n < 0 || n > ctx->max_requests) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (!stage->counts || !pools->host_free_count) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16) || K_act < 0 || K_act > (int64_t(1) << 32)) return CASCADE_ERANGE;
    if (link_budget_ns < 0 || link_budget_ns > (int64_t(1) << 50) || host_reserve < 0) return CASCADE_ERANGE;
    const bool with_tables = stage->deep_tbl != nullptr;
    if (n > 0 && (!budget || !order || !action || !stage->staged || !r->prompt || !r->n0 || !r->n1 || !r->n2))
        return CASCADE_EINVAL;
    if (with_tables) {
        if (!pools->host_tbl || !pools->host_free || pools->maxb < 1 || pools->host_free_cap < 0 ||
            stage->stage_cap < 0 || (stage->stage_cap > 0 && (!stage->stage_src || !stage->stage_dst)))
            return CASCADE_EINVAL;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const cascade_params &p = ctx->params;
    StageArgs a;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.budget = budget;
    a.order = order;
    a.action = action;
    a.pools = *pools;
    a.stage = *stage;
    a.work = ctx->work_admit;
    a.scalars = ctx->plan_scalars;
    a.status = ctx->status_dev;
    a.A_act = make_load_consts(p, D_act, K_act).A_act;
    a.link_budget_ns = link_budget_ns;
    a.hop_delta = p.delta_ns[2] > p.delta_ns[1] ? p.delta_ns[2] - p.delta_ns[1] : 0;
    a.hop_blk = p.blk_ns[2] > p.blk_ns[1] ? p.blk_ns[2] - p.blk_ns[1] : 1;
    a.host_reserve = host_reserve;
    a.n = n;
    a.with_tables = with_tables ? 1 : 0;
    int T, C, K;
    if (!cascade_pick_geometry(ctx, n > 0 ? n : 1, &T, &C, &K)) return CASCADE_EINVAL;
    cudaError_t e = T == 256 ? launch_stage_k<256>(K, p, a, C, ctx->pdl, s) : launch_stage_k<512>(K, p, a, C, ctx->pdl, s);
    CASCADE_CUDA_TRY(ctx, e);
    if (with_tables && n > 0) {
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(ctx->num_sms * 2), dim3(256), 0, s, apply_stage_kernel, a));
    }
    return CASCADE_OK;
}

extern "C" int cascade_dedup(cascade_ctx *ctx, const cascade_dedup_args *u, int n, void *stream) {
    CascadeRange nvtx_range("cascade_dedup");
    if (!ctx || !u || n < 0) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (!u->list_count || !u->free_count || !u->counts || !u->scratch || u->list_cap < 0 || u->free_cap < 0 ||
        u->n_src_ids < 0 || u->n_dst_ids < 0 || u->maxb < 0)
        return CASCADE_EINVAL;
    if (u->list_cap > 0 && (!u->list_src || !u->list_dst || !u->out_src || !u->out_dst || !u->free_list || !u->ref))
        return CASCADE_EINVAL;
    if (u->list_cap > 0 && (u->out_src == u->list_src || u->out_dst == u->list_dst || u->out_src == u->list_dst ||
                            u->out_dst == u->list_src))
        return CASCADE_EINVAL;
    if (n > 0 && (!u->lo_a || !u->len_a || !u->src_tbl || !u->dst_tbl || !u->shared || u->maxb < 1))
        return CASCADE_EINVAL;
    const int n_tiles = u->list_cap > 0 ? (u->list_cap + kDdTile - 1) / kDdTile : 1;
    if (u->scratch_len < 2 * (int64_t)u->n_src_ids + n_tiles + 8) return CASCADE_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    DedupArgs a;
    a.u = *u;
    a.first = u->scratch;
    a.count = u->scratch + u->n_src_ids;
    a.tile_kept = u->scratch + 2 * (size_t)u->n_src_ids;
    a.sc = a.tile_kept + n_tiles;
    a.status = ctx->status_dev;
    a.n = n;
    a.n_tiles = n_tiles;
    int grid = n_tiles * kDdRounds;
    if (grid > ctx->num_sms * 8) grid = ctx->num_sms * 8;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(kDdThreads), 0, s, dedup_init_kernel, a));
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(grid), dim3(kDdThreads), 0, s, dedup_mark_kernel, a));
    int slot_blocks = (n + kDdThreads / 32 - 1) / (kDdThreads / 32);
    if (slot_blocks > ctx->num_sms * 4) slot_blocks = ctx->num_sms * 4;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(n_tiles + slot_blocks), dim3(kDdThreads), 0, s,
                                         dedup_tables_kernel, a));
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(n_tiles), dim3(kDdThreads), 0, s, dedup_compact_kernel, a));
    return CASCADE_OK;
}
