// cascade_schedule: least-remaining-budget-first order (64-bit LSD radix sort) and prefix-sum
// admission (Algorithm 1, phase 2) in ONE kernel launch.
//
// Layout: a thread-block cluster of C CTAs (C = 1, 2, 4, 8) holds the whole queue in shared memory,
// 1024*K elements of 16 bytes (key, slot, want) per CTA.  Each radix pass
//   (a) ranks the 8-bit digits of a warp's 32*K consecutive elements with __match_any_sync and a
//       per-warp 16-bit histogram in shared memory (stable within the warp),
//   (b) scans those histograms across the 32 warps with warp shuffles,
//   (c) exchanges the 256-bin CTA histograms through distributed shared memory and derives, per
//       digit, the global base of this CTA,
//   (d) scatters every element straight into the destination CTA's shared memory (16-byte
//       remote store), so keys never visit global memory between passes.
// Passes whose digit is the same in every key are skipped.  The admission scans run on the sorted
// elements while they are still on chip.  Two cluster barriers per pass are the only waits; they
// are hardware barriers (no spin loops).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 256;
constexpr int kWhistStride = kBins + 2;  // in uint16 units: column reads by 32 lanes hit 32 banks
constexpr unsigned kFull = 0xffffffffu;

struct __align__(16) SortElem {
    uint64_t key;
    uint32_t idx;
    int32_t want;
};

// per-CTA values published to the cluster
struct Exch {
    unsigned long long diff;  // OR of (key ^ key[0]) over this CTA's keys
    long long w1, w2;         // tokens wanted by this CTA's Tier-1 / Tier-2 elements
    int n1;                   // Tier-1 elements in this CTA
    int cnt;                  // elements with a non-zero grant before the batch-size cap
};

struct ScheduleArgs {
    const uint64_t *key;
    const int32_t *prompt, *n0, *n1, *n2;
    uint32_t *order_out;
    int32_t *grant_out;
    cascade_sched_counts *counts;
    long long TB;       // tokens left after the in-flight decodes took theirs
    long long reserve;  // Tier-2 reserve
    int seq_cap;        // max_batch - D_act, >= 0
    int n;
    int bt;
    int per_shift;      // log2(elements per CTA)
};

__device__ __forceinline__ long long warp_incl_scan(long long v, int lane) {
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        long long t = __shfl_up_sync(kFull, v, s);
        if (lane >= s) v += t;
    }
    return v;
}

__device__ __forceinline__ unsigned warp_incl_scan(unsigned v, int lane) {
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        unsigned t = __shfl_up_sync(kFull, v, s);
        if (lane >= s) v += t;
    }
    return v;
}

template <int K>
__global__ void __launch_bounds__(kThreads, 1) schedule_kernel(const __grid_constant__ ScheduleArgs a) {
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();
    constexpr int per = kThreads * K;

    extern __shared__ __align__(16) unsigned char smem[];
    SortElem *elems = reinterpret_cast<SortElem *>(smem);
    uint16_t *whist = reinterpret_cast<uint16_t *>(smem + size_t(per) * sizeof(SortElem));
    uint32_t *hist = reinterpret_cast<uint32_t *>(whist + kWarps * kWhistStride);
    uint32_t *base = hist + kBins;
    long long *wtmp = reinterpret_cast<long long *>(base + kBins);  // 3 * 32 entries
    Exch *exch = reinterpret_cast<Exch *>(wtmp + 3 * kWarps);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;

    if (crank == 0 && tid == 0) {
        a.counts->n_admitted = 0;
        a.counts->tokens_granted = 0;
    }

    // ---- load: key, slot, tokens wanted (prompt minus the matched prefix) ----------------------
    SortElem e[K];
    const unsigned long long key0 = a.key[0];
    unsigned long long diff = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int li = (warp * K + k) * 32 + lane;
        const long long g = (long long)crank * per + li;
        if (g < a.n) {
            const unsigned long long key = a.key[g];
            const long long P = a.prompt[g], h0 = a.n0[g], h1 = a.n1[g], h2 = a.n2[g];
            long long want = 0;
            if (dev_request_valid(a.bt, P, h0, h1, h2)) want = P - (h0 + h1 + h2) * a.bt;
            e[k].key = key;
            e[k].idx = (uint32_t)g;
            e[k].want = (int32_t)want;
            diff |= key ^ key0;
        } else {
            e[k].key = ~0ull;  // padding sorts behind every real key and stays there (stable passes)
            e[k].idx = 0xffffffffu;
            e[k].want = 0;
        }
    }
    {
        unsigned lo = __reduce_or_sync(kFull, (unsigned)diff);
        unsigned hi = __reduce_or_sync(kFull, (unsigned)(diff >> 32));
        if (lane == 0) wtmp[warp] = (long long)(((unsigned long long)hi << 32) | lo);
        __syncthreads();
        if (warp == 0) {
            unsigned long long v = (unsigned long long)wtmp[lane];
            lo = __reduce_or_sync(kFull, (unsigned)v);
            hi = __reduce_or_sync(kFull, (unsigned)(v >> 32));
            if (lane == 0) exch->diff = ((unsigned long long)hi << 32) | lo;
        }
    }
    cluster.sync();
    unsigned long long alld = 0;
    for (unsigned c = 0; c < csize; ++c) alld |= cluster.map_shared_rank(exch, c)->diff;

    // ---- LSD radix sort, 8 bits per pass --------------------------------------------------------
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = pass * 8;
        if (((alld >> shift) & 0xffull) == 0) continue;  // same digit in every key: nothing moves

        // (a) stable rank of each element among equal digits of its warp's chunk
        uint16_t *myhist = whist + warp * kWhistStride;
        for (int i = lane; i < kWhistStride / 2; i += 32) reinterpret_cast<uint32_t *>(myhist)[i] = 0;
        __syncwarp();
        unsigned off[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
            const unsigned peers = __match_any_sync(kFull, d);
            const unsigned lower = peers & lt_mask;
            const unsigned pre = myhist[d];
            __syncwarp();
            if (lower == 0) myhist[d] = (uint16_t)(pre + __popc(peers));
            __syncwarp();
            off[k] = pre + __popc(lower);
        }
        __syncthreads();

        // (b) exclusive scan across warps, one digit column per iteration; warp j owns digits 8j..8j+7
#pragma unroll
        for (int dd = 0; dd < kBins / kWarps; ++dd) {
            const int d = warp * (kBins / kWarps) + dd;
            const unsigned v = whist[lane * kWhistStride + d];
            const unsigned incl = warp_incl_scan(v, lane);
            whist[lane * kWhistStride + d] = (uint16_t)(incl - v);
            if (lane == 31) hist[d] = incl;
        }
        cluster.sync();  // histograms visible cluster-wide; every CTA holds its elements in registers

        // (c) global base of this CTA for each digit
        unsigned total = 0, before = 0, incl = 0;
        if (tid < kBins) {
            for (unsigned c = 0; c < csize; ++c) {
                const unsigned h = cluster.map_shared_rank(hist, c)[tid];
                total += h;
                if (c < crank) before += h;
            }
            incl = warp_incl_scan(total, lane);
            if (lane == 31) reinterpret_cast<unsigned *>(wtmp)[warp] = incl;
        }
        __syncthreads();
        if (tid < kBins) {
            unsigned add = 0;
            for (int w = 0; w < warp; ++w) add += reinterpret_cast<unsigned *>(wtmp)[w];
            base[tid] = incl - total + add + before;
        }
        __syncthreads();

        // (d) scatter into the owning CTA's shared memory
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
            const unsigned pos = base[d] + whist[warp * kWhistStride + d] + off[k];
            SortElem *dst = cluster.map_shared_rank(elems, pos >> a.per_shift) + (pos & (per - 1));
            *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(&e[k]);
        }
        cluster.sync();  // all remote stores have landed
#pragma unroll
        for (int k = 0; k < K; ++k) e[k] = elems[(warp * K + k) * 32 + lane];
    }

    // ---- admission: clamped prefix sums over the sorted elements ---------------------------------
    long long ex[K];
    long long run = 0, s1 = 0, s2 = 0;
    int c1 = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long w = e[k].want;
        const bool real = e[k].idx != 0xffffffffu;
        const bool t2 = (e[k].key >> 63) != 0;
        if (real && !t2) { s1 += w; ++c1; }
        if (real && t2) s2 += w;
        const long long x = warp_incl_scan(w, lane);
        ex[k] = run + x - w;
        run += __shfl_sync(kFull, x, 31);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        s1 += __shfl_xor_sync(kFull, s1, s);
        s2 += __shfl_xor_sync(kFull, s2, s);
        c1 += __shfl_xor_sync(kFull, c1, s);
    }
    if (lane == 0) {
        wtmp[warp] = run;
        wtmp[kWarps + warp] = s1;
        wtmp[2 * kWarps + warp] = s2;
        reinterpret_cast<int *>(base)[warp] = c1;
    }
    __syncthreads();
    if (warp == 0) {
        const long long t = wtmp[lane];
        const long long inc = warp_incl_scan(t, lane);
        long long a1 = wtmp[kWarps + lane], a2 = wtmp[2 * kWarps + lane];
        int ac = reinterpret_cast<int *>(base)[lane];
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            a1 += __shfl_xor_sync(kFull, a1, s);
            a2 += __shfl_xor_sync(kFull, a2, s);
            ac += __shfl_xor_sync(kFull, ac, s);
        }
        wtmp[lane] = inc - t;  // exclusive offset of each warp inside the CTA
        if (lane == 0) {
            exch->w1 = a1;
            exch->w2 = a2;
            exch->n1 = ac;
        }
    }
    cluster.sync();
    long long W1 = 0, W2 = 0, cta_off = 0;
    int N1 = 0;
    for (unsigned c = 0; c < csize; ++c) {
        const Exch *x = cluster.map_shared_rank(exch, c);
        const long long x1 = x->w1, x2 = x->w2;
        W1 += x1;
        W2 += x2;
        N1 += x->n1;
        if (c < crank) cta_off += x1 + x2;
    }
    const long long R2 = min(min(a.reserve, W2), a.TB);
    const long long TB1 = a.TB - R2;
    const long long TB2 = a.TB - min(TB1, W1);  // the reserve plus whatever Tier-1 left
    const long long warp_off = cta_off + wtmp[warp];
    int grant[K];
    unsigned runc = 0;
    unsigned exf[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long w = e[k].want;
        const long long eg = warp_off + ex[k];
        const bool t2 = (e[k].key >> 63) != 0;
        long long g = t2 ? (TB2 - (eg - W1)) : (TB1 - eg);
        g = g < 0 ? 0 : (g > w ? w : g);
        grant[k] = (int)g;
        const unsigned b = __ballot_sync(kFull, g > 0);
        exf[k] = runc + __popc(b & lt_mask);
        runc += __popc(b);
    }
    __syncthreads();  // wtmp is reused below
    if (lane == 0) reinterpret_cast<unsigned *>(wtmp)[warp] = runc;
    __syncthreads();
    if (warp == 0) {
        const unsigned t = reinterpret_cast<unsigned *>(wtmp)[lane];
        const unsigned inc = warp_incl_scan(t, lane);
        reinterpret_cast<unsigned *>(wtmp)[lane] = inc - t;
        if (lane == 31) exch->cnt = (int)inc;
    }
    cluster.sync();
    unsigned cnt_off = 0;
    for (unsigned c = 0; c < crank; ++c) cnt_off += (unsigned)cluster.map_shared_rank(exch, c)->cnt;
    cnt_off += reinterpret_cast<unsigned *>(wtmp)[warp];

    long long tok = 0;
    int adm = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (grant[k] > 0 && (long long)(cnt_off + exf[k]) >= (long long)a.seq_cap) grant[k] = 0;
        if (e[k].idx != 0xffffffffu) {
            const long long g = (long long)crank * per + (warp * K + k) * 32 + lane;
            a.order_out[g] = e[k].idx;
            a.grant_out[e[k].idx] = grant[k];
            tok += grant[k];
            adm += grant[k] > 0;
        }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        tok += __shfl_xor_sync(kFull, tok, s);
        adm += __shfl_xor_sync(kFull, adm, s);
    }
    if (lane == 0 && adm > 0) {
        atomicAdd(reinterpret_cast<unsigned long long *>(&a.counts->tokens_granted), (unsigned long long)tok);
        atomicAdd(&a.counts->n_admitted, adm);
    }
    if (crank == 0 && tid == 0) a.counts->n_tier1 = N1;
    cluster.sync();  // no CTA leaves while a peer may still read its shared memory
}

__global__ void zero_counts_kernel(cascade_sched_counts *c) {
    c->n_tier1 = 0;
    c->n_admitted = 0;
    c->tokens_granted = 0;
}

size_t smem_bytes(int K) {
    return size_t(kThreads) * K * sizeof(SortElem) + size_t(kWarps) * kWhistStride * sizeof(uint16_t) +
           2 * kBins * sizeof(uint32_t) + 3 * kWarps * sizeof(long long) + sizeof(Exch) + 16;
}

template <int K>
cudaError_t launch(const ScheduleArgs &a, int cluster_size, int device, cudaStream_t stream) {
    static bool configured_dev[64] = {};
    bool unknown = false;
    bool &configured = (device >= 0 && device < 64) ? configured_dev[device] : unknown;
    const size_t smem = smem_bytes(K);
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(schedule_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(schedule_kernel<K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster_size, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, schedule_kernel<K>, a);
}

}  // namespace

extern "C" int cascade_schedule(cascade_ctx *ctx, const cascade_reqs *r, const uint64_t *key, int n, int32_t D_act,
                                uint32_t *order_out, int32_t *grant_out, cascade_sched_counts *counts_dev,
                                void *stream) {
    if (!ctx || !r || n < 0 || n > ctx->max_requests || !counts_dev) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16)) return CASCADE_ERANGE;
    cudaStream_t s = (cudaStream_t)stream;
    if (n == 0) {
        zero_counts_kernel<<<1, 1, 0, s>>>(counts_dev);
        CASCADE_CUDA_TRY(ctx, cudaGetLastError());
        return CASCADE_OK;
    }
    if (!key || !order_out || !grant_out || !r->prompt || !r->n0 || !r->n1 || !r->n2) return CASCADE_EINVAL;
    const cascade_params &p = ctx->params;
    // cluster size C and keys per thread K: the smallest K that fits the queue into <= 8 CTAs
    int C = ctx->sort_cluster, K = ctx->sort_items;
    if (K != 1 && K != 2 && K != 4 && K != 8) K = 0;
    if (C != 1 && C != 2 && C != 4 && C != 8 && C != 16) C = 0;
    if (K == 0) {
        const int cmax = C ? C : 8;
        K = 1;
        while (K < 8 && (long long)cmax * kThreads * K < n) K *= 2;
    }
    if (C == 0) {
        C = 1;
        while (C < 16 && (long long)C * kThreads * K < n) C *= 2;
    }
    if ((long long)C * kThreads * K < n) return CASCADE_EINVAL;
    ScheduleArgs a;
    a.key = key;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.order_out = order_out;
    a.grant_out = grant_out;
    a.counts = counts_dev;
    const long long tb = (long long)p.token_budget - D_act;
    a.TB = tb > 0 ? tb : 0;
    a.reserve = p.tier2_reserve;
    const int cap = p.max_batch - D_act;
    a.seq_cap = cap > 0 ? cap : 0;
    a.n = n;
    a.bt = p.bt;
    int sh = 10;
    for (int k = K; k > 1; k >>= 1) ++sh;
    a.per_shift = sh;
    cudaError_t e;
    switch (K) {
        case 1: e = launch<1>(a, C, ctx->device, s); break;
        case 2: e = launch<2>(a, C, ctx->device, s); break;
        case 4: e = launch<4>(a, C, ctx->device, s); break;
        default: e = launch<8>(a, C, ctx->device, s); break;
    }
    CASCADE_CUDA_TRY(ctx, e);
    return CASCADE_OK;
}
