// cascade_schedule: least-remaining-budget-first order (64-bit LSD radix sort) and prefix-sum
// admission (Algorithm 1, phase 2) in ONE kernel launch.
//
// Layout: a thread-block cluster of C CTAs (C = 1..16) holds the whole queue in shared memory,
// T*K elements of 16 bytes (key, slot, want) per CTA (T threads, K elements per thread).  Each
// radix pass
//   (a) ranks the 8-bit digits of a warp's 32*K consecutive elements (stable within the warp) with
//       a per-warp 16-bit histogram in shared memory,
//   (b) scans those histograms across the CTA's warps with segmented warp shuffles and PUSHES the
//       256-bin CTA histogram into every CTA of the cluster (distributed shared memory stores),
//   (c) derives, per digit, the global base of this CTA from the locally received histograms,
//   (d) scatters every element straight into the destination CTA's shared memory (16-byte
//       remote store), so keys never visit global memory between passes.
// Passes whose digit is the same in every key are skipped.  The admission scans run on the sorted
// elements while they are still on chip.
// The two exchanges of a pass are data driven: histograms and elements travel as 16-byte
// asynchronous stores (st.async) that report their bytes to an mbarrier of the receiving CTA, so a
// CTA goes on as soon as ITS inputs have landed instead of waiting at a cluster-wide barrier.  The
// histogram exchange doubles as the guard for buffer reuse: nobody scatters into a CTA before that
// CTA has published the histogram of the elements it already holds in registers.  The mbarrier waits
// are clock-bounded (CASCADE_ST_ETIMEOUT, results then undefined but every CTA still walks the same
// cluster barriers and exits).  CASCADE_SORT_ASYNC=0 selects plain cluster barriers instead.
//
// Small queues (up to 2048 requests by default) skip the radix passes: with every key in each CTA's
// shared memory, the final position of an element is simply the number of (key, slot) pairs below
// it, counted by a few threads per element, and ONE exchange places every element.  The work is
// quadratic but perfectly parallel, and at these sizes the eight passes' sixteen exchanges cost more.
#include <cooperative_groups.h>

#include "common.cuh"
#include "mbarrier.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kBins = 256;
constexpr int kWhistStride = kBins + 2;  // in uint16 units: column reads by 32 lanes hit 32 banks
constexpr int kMaxCluster = 16;
constexpr unsigned kFull = 0xffffffffu;
constexpr long long kWaitLimit = 2000000000LL;  // clocks a CTA waits for its peers' data before giving up
constexpr int kRankMaxKeys = 4096;              // keys the counting path can hold per CTA
constexpr size_t kRankExtra = kRankMaxKeys * sizeof(uint64_t) + 256 * sizeof(int);

struct __align__(16) SortElem {
    uint64_t key;
    uint32_t idx;
    int32_t want;
};

// per-CTA values published to every CTA of the cluster
struct __align__(16) Exch {
    unsigned long long diff;  // OR of (key ^ key[0]) over this CTA's keys
    long long w1, w2;         // tokens wanted by this CTA's Tier-1 / Tier-2 elements
    int n1;                   // Tier-1 elements in this CTA
    int cnt;                  // elements with a non-zero grant before the batch-size cap
};

// what every CTA tells the others after the passes over bits kTopShift..63
struct __align__(16) TieExch {
    unsigned long long first, last;  // bits kTopShift..63 of the CTA's first and last real element
    int count;                       // real elements the CTA holds
    int flags;                       // 1: equal neighbours inside the CTA, 2: a run longer than kMaxRun, or more than
                                     //    an eighth of the CTA's threads hold an element equal to its neighbour
};
constexpr int kMaxRun = 128;
constexpr int kTopShift = 32;   // first-stage order: key bits 32..63 = tier, budget / 512 ns (a multiple of the 8-bit digits)

struct ScheduleArgs {
    const uint64_t *key;
    const int32_t *prompt, *n0, *n1, *n2;
    const int32_t *want_in;   // plan-first admission: the offers cascade_budget left in the context, else NULL
    uint32_t *order_out;
    int32_t *grant_out;
    cascade_sched_counts *counts;
    long long TB;       // tokens left after the in-flight decodes took theirs
    long long reserve;  // Tier-2 reserve
    int seq_cap;        // max_batch - D_act, >= 0
    int n;
    int bt;
    int stage;          // 1: group by digit locally before the remote copy
    int async_sync;     // 1: per-pass exchanges complete on mbarriers (data driven), 0: cluster barriers
    SortElem *runs_out; // run mode: every cluster orders its own 16384-slot stretch of the queue and leaves the ordered
                        // elements here (no admission); NULL otherwise
    const SortElem *sorted_in;  // admission-only kernel: the fully ordered elements
    int top_first;      // 1: order by bits kTopShift..63 first, fix short runs of equal values locally (see the pass loop)
    int rank_per;       // >0: small queue, order by counting (see rank_order below) with this many elements per CTA
    uint32_t *status;
};

template <typename T>
__device__ __forceinline__ T seg_incl_scan(T v, int pos, int width) {
    // inclusive scan inside aligned groups of `width` lanes; pos = lane % width
    for (int s = 1; s < width; s <<= 1) {
        T t = __shfl_up_sync(kFull, v, s, width);
        if (pos >= s) v += t;
    }
    return v;
}

// Admission (Algorithm 1, phase 2) on the sorted elements while they are still on chip: clamped prefix sums of
// the tokens wanted against the Tier-1 / Tier-2 token budgets, the batch-size cap, then `order`, `grant` and the
// counts are written.  e[k] is the element at sorted position crank*per_rt + (warp*K + k)*32 + lane; padding has
// idx 0xffffffff.  Two cluster barriers; every CTA of the cluster must call it.
template <int T, int K>
__device__ __forceinline__ void admit_and_write(const ScheduleArgs &a, const SortElem (&e)[K], int per_rt,
                                                cg::cluster_group &cluster, long long *wtmp, int *itmp, Exch *exall) {
    constexpr int W = T / 32;
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
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
        const long long x = seg_incl_scan(w, lane, 32);
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
        wtmp[32 + warp] = s1;
        wtmp[64 + warp] = s2;
        itmp[warp] = c1;
    }
    __syncthreads();
    if (warp == 0) {
        const bool in = lane < W;
        const long long t = in ? wtmp[lane] : 0;
        const long long inc = seg_incl_scan(t, lane, 32);
        long long a1 = in ? wtmp[32 + lane] : 0, a2 = in ? wtmp[64 + lane] : 0;
        int ac = in ? itmp[lane] : 0;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            a1 += __shfl_xor_sync(kFull, a1, s);
            a2 += __shfl_xor_sync(kFull, a2, s);
            ac += __shfl_xor_sync(kFull, ac, s);
        }
        if (in) wtmp[lane] = inc - t;  // exclusive offset of each warp inside the CTA
        if (lane < csize) {
            Exch *x = cluster.map_shared_rank(exall, lane) + crank;
            x->w1 = a1;
            x->w2 = a2;
            x->n1 = ac;
        }
    }
    cluster.sync();
    long long W1 = 0, W2 = 0, cta_off = 0;
    int N1 = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < csize) {
            const long long x1 = exall[c].w1, x2 = exall[c].w2;
            W1 += x1;
            W2 += x2;
            N1 += exall[c].n1;
            if (c < crank) cta_off += x1 + x2;
        }
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
        const unsigned t = lane < W ? reinterpret_cast<unsigned *>(wtmp)[lane] : 0u;
        const unsigned inc = seg_incl_scan(t, lane, 32);
        if (lane < W) reinterpret_cast<unsigned *>(wtmp)[lane] = inc - t;
        const int tot = (int)__shfl_sync(kFull, inc, 31);
        if (lane < csize) cluster.map_shared_rank(exall, lane)[crank].cnt = tot;
    }
    cluster.sync();
    unsigned cnt_off = reinterpret_cast<unsigned *>(wtmp)[warp];
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c)
        if (c < crank) cnt_off += (unsigned)exall[c].cnt;

    long long tok = 0;
    int adm = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (grant[k] > 0 && (long long)(cnt_off + exf[k]) >= (long long)a.seq_cap) grant[k] = 0;
        if (e[k].idx != 0xffffffffu) {
            const long long g = (long long)crank * per_rt + (warp * K + k) * 32 + lane;
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
}

template <int T, int K>
__global__ void __launch_bounds__(T, 1) schedule_kernel(const __grid_constant__ ScheduleArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int W = T / 32;          // warps per CTA
    constexpr int per = T * K;         // elements per CTA
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();

    extern __shared__ __align__(16) unsigned char smem[];
    SortElem *elems = reinterpret_cast<SortElem *>(smem);
    SortElem *stage = elems + per;
    uint16_t *whist = reinterpret_cast<uint16_t *>(smem + 2 * size_t(per) * sizeof(SortElem));
    uint16_t *allhist = whist + W * kWhistStride;                      // [2][kMaxCluster][kBins]
    uint32_t *base = reinterpret_cast<uint32_t *>(allhist + 2 * kMaxCluster * kBins);
    uint32_t *lbase = base + kBins;
    long long *wtmp = reinterpret_cast<long long *>(lbase + kBins);    // 3 * 32 entries
    Exch *exall = reinterpret_cast<Exch *>(wtmp + 3 * 32);             // [kMaxCluster]
    uint16_t *minehist = reinterpret_cast<uint16_t *>(exall + kMaxCluster);   // [kBins], 16-byte aligned
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(minehist + kBins);  // hist[2], elem[2]
    TieExch *tie_ex = reinterpret_cast<TieExch *>(bars + 4);                              // [kMaxCluster]
    // counting path only (the <256, 1> instance): every key of the queue, then per-thread partial counts
    uint64_t *keys_all = reinterpret_cast<uint64_t *>(tie_ex + kMaxCluster);
    int *partial = reinterpret_cast<int *>(keys_all + kRankMaxKeys);
    const bool by_rank = (K == 1) && a.rank_per > 0;
    const int per_rt = by_rank ? a.rank_per : per;   // elements this CTA holds

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;

    // run mode: this cluster orders the slots [base, base + n_q) only
    const long long base_slot = a.runs_out ? (long long)(blockIdx.x / csize) * ((long long)csize * per) : 0;
    const long long left_q = (long long)a.n - base_slot;
    const int n_q = a.runs_out ? (int)(left_q < 0 ? 0 : (left_q > (long long)csize * per ? (long long)csize * per : left_q)) : a.n;
    if (crank == 0 && tid == 0 && !a.runs_out) {
        a.counts->n_admitted = 0;
        a.counts->tokens_granted = 0;
    }
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbarrier_init(cta_smem_addr(&bars[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // "I have started, my barriers exist": the matching wait sits in front of the first store into another CTA's
    // shared memory, so the barrier's latency hides behind the loads below
    cluster.barrier_arrive();

    // ---- load: key, slot, tokens wanted (prompt minus the matched prefix) ----------------------
    SortElem e[K];
    const unsigned long long key0 = n_q > 0 ? a.key[base_slot] : 0ull;
    unsigned long long diff = 0;
    auto load_elem = [&](int k) {
        const int li = (warp * K + k) * 32 + lane;
        const long long gl = (long long)crank * per_rt + li;   // position inside this cluster's stretch
        const long long g = base_slot + gl;                     // slot of the queue
        if (li < per_rt && gl < n_q) {
            const unsigned long long key = a.key[g];
            const long long P = a.prompt[g], h0 = a.n0[g], h1 = a.n1[g], h2 = a.n2[g];
            long long want = 0;
            if (dev_request_valid(a.bt, P, h0, h1, h2)) want = a.want_in ? a.want_in[g] : P - (h0 + h1 + h2) * a.bt;
            e[k].key = key;
            e[k].idx = (uint32_t)g;
            e[k].want = (int32_t)want;
            diff |= key ^ key0;
        } else {
            e[k].key = ~0ull;  // padding sorts behind every real key and stays there (stable passes)
            e[k].idx = 0xffffffffu;
            e[k].want = 0;
        }
    };
#pragma unroll
    for (int k = 0; k < K; ++k) load_elem(k);
    if (by_rank) {
        if constexpr (K == 1) {
            // ---- order by counting ----------------------------------------------------------------
            // all keys of the queue into shared memory (coalesced, read once per CTA)
            const int n = a.n;
            for (int j = tid; j < n; j += T) keys_all[j] = a.key[j];
            __syncthreads();
            // S = T / per_rt threads share one element: thread t counts, for element t % per_rt, the pairs
            // (key, slot) below it among the slots of segment t / per_rt
            const int S = T / per_rt;
            const int el = tid % per_rt, seg = tid / per_rt;
            const long long gi = (long long)crank * per_rt + el;
            int cnt = 0;
            if (seg < S && gi < n) {
                const unsigned long long ki = keys_all[gi];
                const int seg_len = (n + S - 1) / S;
                const int lo = seg * seg_len, hi = min(n, lo + seg_len);
                const int mid = (int)min((long long)hi, max((long long)lo, gi));   // slots below gi: ties count
                // two keys per 16-byte shared-memory load, eight keys per round: the loads of a round are
                // independent, so their latency overlaps
                auto count_range = [&](int from, int to, bool ties) {
                    int j = from;
                    int c = 0;
                    for (; j < to && (j & 1); ++j) c += ties ? keys_all[j] <= ki : keys_all[j] < ki;
                    const ulonglong2 *pairs = reinterpret_cast<const ulonglong2 *>(keys_all);
                    for (; j + 8 <= to; j += 8) {
                        ulonglong2 v[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) v[u] = pairs[(j >> 1) + u];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            c += ties ? (v[u].x <= ki) + (v[u].y <= ki) : (v[u].x < ki) + (v[u].y < ki);
                        }
                    }
                    for (; j < to; ++j) c += ties ? keys_all[j] <= ki : keys_all[j] < ki;
                    return c;
                };
                cnt = count_range(lo, mid, true);
                cnt += count_range((int)max((long long)mid, min((long long)hi, gi + 1)), hi, false);   // above gi: ties do not count
            }
            partial[tid] = cnt;
            // besides the CTA barrier, the cluster barrier begun at the top: no store into another CTA's shared memory
            // before every CTA of the cluster has started
            __syncthreads();
            cluster.barrier_wait();
            // the element's owner adds the partial counts and sends the element to its final place
            if (tid < per_rt && e[0].idx != 0xffffffffu) {
                int pos = 0;
                for (int q = 0; q < S; ++q) pos += partial[q * per_rt + tid];
                SortElem *dst = cluster.map_shared_rank(elems, pos / per_rt) + (pos % per_rt);
                *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(&e[0]);
            }
            cluster.sync();
            // slots n .. C*per_rt-1 of the sorted layout received nothing: they are padding
            const long long g = (long long)crank * per_rt + tid;
            if (tid < per_rt && g < n) e[0] = elems[tid];
            else { e[0].key = ~0ull; e[0].idx = 0xffffffffu; e[0].want = 0; }
        }
    } else {
    {
        unsigned lo = __reduce_or_sync(kFull, (unsigned)diff);
        unsigned hi = __reduce_or_sync(kFull, (unsigned)(diff >> 32));
        if (lane == 0) wtmp[warp] = (long long)(((unsigned long long)hi << 32) | lo);
        // besides the CTA barrier, the cluster barrier begun at the top: the store below is the first access to another
        // CTA's shared memory, which must not happen before that CTA has started (and initialised its mbarriers)
        __syncthreads();
        cluster.barrier_wait();
        if (warp == 0) {
            unsigned long long v = lane < W ? (unsigned long long)wtmp[lane] : 0ull;
            lo = __reduce_or_sync(kFull, (unsigned)v);
            hi = __reduce_or_sync(kFull, (unsigned)(v >> 32));
            if (lane < csize) cluster.map_shared_rank(exall, lane)[crank].diff = ((unsigned long long)hi << 32) | lo;
        }
    }
    cluster.sync();
    unsigned long long alld = 0;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c)
        if (c < csize) alld |= exall[c].diff;

    // ---- LSD radix sort, 8 bits per pass --------------------------------------------------------
    // With top_first the four passes over the low 32 bits (the arrival id and the budget's lowest nine bits) are left
    // out at first: budgets are nanosecond values, so after four passes over bits 32..63 (tier, budget in steps of
    // 512 ns) equal values are rare and short runs of them are put in (key, slot) order by a fix-up inside the CTA (or
    // between two neighbouring CTAs).  Only when a run is longer than kMaxRun, or when much of a CTA is tied, the queue
    // is loaded again and ordered with all eight passes.
    int ep = 0;          // passes executed so far: selects the mbarrier pair and its phase
    bool dead = false;   // a bounded wait expired: stop exchanging, keep walking the barriers
    int first_pass = a.top_first ? kTopShift / 8 : 0;
    for (int attempt = 0; attempt < 2; ++attempt) {
    const int ep_before = ep;
    for (int pass = first_pass; pass < 8; ++pass) {
        const int shift = pass * 8;
        if (((alld >> shift) & 0xffull) == 0) continue;  // same digit in every key: nothing moves
        if (dead) continue;
        const int q = ep & 1;
        const unsigned phase = (unsigned)(ep >> 1) & 1u;
        uint16_t *hist_in = allhist + q * kMaxCluster * kBins;
        const unsigned hist_bar = cta_smem_addr(&bars[q]), elem_bar = cta_smem_addr(&bars[2 + q]);
        if (a.async_sync && tid == 0) {
            mbarrier_arrive_expect(hist_bar, csize * kBins * (unsigned)sizeof(uint16_t));
            mbarrier_arrive_expect(elem_bar, (unsigned)(per * sizeof(SortElem)));
        }
        ++ep;

        // (a) stable rank of each element among equal digits of its warp's chunk
        uint16_t *myhist = whist + warp * kWhistStride;
        for (int i = lane; i < kWhistStride / 2; i += 32) reinterpret_cast<uint32_t *>(myhist)[i] = 0;
        __syncwarp();
        unsigned off[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
            // lanes holding the same digit: eight ballots, one per bit (cheaper than match.any on
            // high-entropy digits, and its cost does not depend on the data)
            unsigned peers = kFull;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const unsigned bal = __ballot_sync(kFull, (d >> b) & 1u);
                peers &= ((d >> b) & 1u) ? bal : ~bal;
            }
            const unsigned lower = peers & lt_mask;
            const unsigned pre = myhist[d];
            __syncwarp();
            if (lower == 0) myhist[d] = (uint16_t)(pre + __popc(peers));
            __syncwarp();
            off[k] = pre + __popc(lower);
        }
        __syncthreads();

        // (b) one thread per digit walks its column of the W per-warp histograms (exclusive scan in
        //     place) and pushes the CTA's count of that digit to every CTA of the cluster
        unsigned mine = 0;
        if (tid < kBins) {
            unsigned v[W];
#pragma unroll
            for (int w = 0; w < W; ++w) v[w] = whist[w * kWhistStride + tid];
#pragma unroll
            for (int w = 0; w < W; ++w) {
                whist[w * kWhistStride + tid] = (uint16_t)mine;
                mine += v[w];
            }
            if (a.async_sync) {
                minehist[tid] = (uint16_t)mine;
            } else {
#pragma unroll
                for (int c = 0; c < kMaxCluster; ++c)
                    if (c < csize) cluster.map_shared_rank(hist_in, c)[crank * kBins + tid] = (uint16_t)mine;
            }
        }
        if (a.async_sync) {
            // 16-byte pieces of this CTA's histogram go to every CTA and count on its histogram barrier;
            // a CTA goes on as soon as the sixteen histograms it needs have landed
            __syncthreads();
            for (unsigned op = tid; op < csize * (kBins / 8); op += T) {
                const unsigned dst = op / (kBins / 8), piece = op % (kBins / 8);
                const uint4 v = *reinterpret_cast<const uint4 *>(minehist + piece * 8);
                st_async_16(cluster_addr(cta_smem_addr(hist_in + crank * kBins + piece * 8), dst), v,
                            cluster_addr(hist_bar, dst));
            }
            const bool ok = mbarrier_wait_bounded(hist_bar, phase, kWaitLimit);
            if (__syncthreads_or(!ok)) dead = true;
        } else {
            cluster.sync();  // histograms delivered; every CTA holds its elements in registers
        }
        if (dead) continue;

        // (c) per digit: global base of this CTA (high bits) and local base inside this CTA (low 14
        //     bits), both from one packed exclusive scan over the 256 digits
        unsigned packed = 0, before = 0, incl = 0;
        if (tid < kBins) {
            unsigned total = 0;
#pragma unroll
            for (int c = 0; c < kMaxCluster; ++c) {
                if (c < csize) {
                    const unsigned h = hist_in[c * kBins + tid];
                    total += h;
                    if (c < crank) before += h;
                }
            }
            packed = (total << 14) | mine;
            incl = seg_incl_scan(packed, lane, 32);
            if (lane == 31) reinterpret_cast<unsigned *>(wtmp)[warp] = incl;
        }
        __syncthreads();
        if (tid < kBins) {
            unsigned add = 0;
#pragma unroll
            for (int w = 0; w < kBins / 32; ++w) {
                const unsigned t = reinterpret_cast<unsigned *>(wtmp)[w];
                if (w < warp) add += t;
            }
            const unsigned excl = incl - packed + add;
            base[tid] = (excl >> 14) + before;      // first global position of this CTA's run of digit tid
            lbase[tid] = excl & 0x3fffu;            // first local position of that run
        }
        __syncthreads();

        if (a.stage) {
            // (d) group the CTA's elements by digit in a local staging buffer, then copy runs of equal
            //     digits to their owners: consecutive lanes store to consecutive remote addresses
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
                const unsigned lpos = lbase[d] + whist[warp * kWhistStride + d] + off[k];
                *reinterpret_cast<uint4 *>(stage + lpos) = *reinterpret_cast<const uint4 *>(&e[k]);
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const unsigned i = (warp * K + k) * 32 + lane;
                const uint4 v = *reinterpret_cast<const uint4 *>(stage + i);
                const unsigned long long key = ((unsigned long long)v.y << 32) | v.x;
                const unsigned d = (unsigned)(key >> shift) & 0xffu;
                const unsigned pos = base[d] + (i - lbase[d]);
                if (a.async_sync) {
                    st_async_16(cluster_addr(cta_smem_addr(elems + (pos % per)), pos / per), v,
                                cluster_addr(elem_bar, pos / per));
                } else {
                    SortElem *dst = cluster.map_shared_rank(elems, pos / per) + (pos % per);
                    *reinterpret_cast<uint4 *>(dst) = v;
                }
            }
        } else {
            // (d) scatter every element straight to its owner
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
                const unsigned pos = base[d] + whist[warp * kWhistStride + d] + off[k];
                if (a.async_sync) {
                    st_async_16(cluster_addr(cta_smem_addr(elems + (pos % per)), pos / per),
                                *reinterpret_cast<const uint4 *>(&e[k]), cluster_addr(elem_bar, pos / per));
                } else {
                    SortElem *dst = cluster.map_shared_rank(elems, pos / per) + (pos % per);
                    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(&e[k]);
                }
            }
        }
        if (a.async_sync) {
            // this CTA's slice is complete when all of its T*K elements have arrived
            const bool ok = mbarrier_wait_bounded(elem_bar, phase, kWaitLimit);
            if (__syncthreads_or(!ok)) dead = true;
            if (dead) continue;
        } else {
            cluster.sync();  // all remote stores have landed
        }
#pragma unroll
        for (int k = 0; k < K; ++k) e[k] = elems[(warp * K + k) * 32 + lane];
    }
    if (first_pass == 0 || dead) break;   // all eight passes ran (or nothing can be trusted any more)

    // ---- ordered by bits kTopShift..63: look for equal neighbours ---------------------------------------------
    if (ep == ep_before) {   // no pass ran: the elements are still only in registers, in slot order
#pragma unroll
        for (int k = 0; k < K; ++k) elems[(warp * K + k) * 32 + lane] = e[k];
        __syncthreads();
    }
    const long long here_ll = (long long)n_q - (long long)crank * per;
    const int n_here = here_ll < 0 ? 0 : (here_ll > per ? per : (int)here_ll);   // real elements of this CTA
    bool tie = false, long_run = false;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int li = (warp * K + k) * 32 + lane;
        if (li < n_here) {
            const unsigned long long top = e[k].key >> kTopShift;
            if (li > 0 && (elems[li - 1].key >> kTopShift) == top) tie = true;
            if (li >= kMaxRun && (elems[li - kMaxRun].key >> kTopShift) == top) long_run = true;
        }
    }
    // the repair counts inside every run: fine for the odd pair of equal budgets, quadratic when much of the queue is
    // tied (quantised budgets, a burst of identical requests): then the remaining passes are cheaper
    const int tied_threads = __syncthreads_count(tie);
    const bool cta_tie = tied_threads > 0;
    const bool cta_long = __syncthreads_or(long_run) || tied_threads * 8 > T;
    if (warp == 0 && lane < csize) {
        TieExch x;
        x.first = n_here > 0 ? elems[0].key >> kTopShift : 0ull;
        x.last = n_here > 0 ? elems[n_here - 1].key >> kTopShift : 0ull;
        x.count = n_here;
        x.flags = (cta_tie ? 1 : 0) | (cta_long ? 2 : 0);
        cluster.map_shared_rank(tie_ex, lane)[crank] = x;
    }
    cluster.sync();   // also: every CTA is done reading its elements before anybody starts another pass
    bool redo = false, any_tie = false, crossing = false;
#pragma unroll
    for (int c = 0; c < kMaxCluster; ++c) {
        if (c < csize) {
            if (tie_ex[c].flags & 2) redo = true;
            if (tie_ex[c].flags & 1) any_tie = true;
            if (c + 1 < csize && tie_ex[c + 1].count > 0 && tie_ex[c].last == tie_ex[c + 1].first) crossing = true;
        }
    }
    if (!redo) {
        if (crossing || cta_tie) {
            // Runs of equal values are short (no part of a run inside one CTA is longer than kMaxRun, so a run lies
            // in one CTA or in two neighbours): every element of a run counts the members of its run that come before
            // it by (key, slot) and moves there.  A run astride a CTA boundary is read from, and written into, the
            // neighbour's shared memory; then every CTA of the cluster takes part in the two barriers (the decision is
            // the same everywhere: all CTAs hold the same exchanged values).
            const long long g0 = (long long)crank * per;
            auto elem_at = [&](long long gpos) -> SortElem {
                const unsigned c = (unsigned)(gpos / per);
                const int l = (int)(gpos - (long long)c * per);
                return c == crank ? elems[l] : cluster.map_shared_rank(elems, c)[l];
            };
            long long newpos[K];
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int li = (warp * K + k) * 32 + lane;
                newpos[k] = g0 + li;
                if (li >= n_here) continue;
                const unsigned long long top = e[k].key >> kTopShift;
                const long long g = g0 + li;
                // a neighbour in the same CTA decides quickly; only at the CTA's ends the other CTA is looked at
                const bool left_same = li > 0 ? (elems[li - 1].key >> kTopShift) == top
                                              : (crossing && g > 0 && (elem_at(g - 1).key >> kTopShift) == top);
                const bool right_same = li + 1 < n_here ? (elems[li + 1].key >> kTopShift) == top
                                                        : (crossing && g + 1 < n_q && (elem_at(g + 1).key >> kTopShift) == top);
                if (!left_same && !right_same) continue;
                // without a run astride a boundary nobody looks into another CTA's shared memory: its owner may be
                // rewriting it, or may have left already
                const long long lo_min = crossing ? 0 : g0, hi_max = crossing ? (long long)n_q - 1 : g0 + n_here - 1;
                long long lo = g, hi = g;
                while (lo > lo_min && g - lo < 2 * kMaxRun && (elem_at(lo - 1).key >> kTopShift) == top) --lo;
                while (hi < hi_max && hi - g < 2 * kMaxRun && (elem_at(hi + 1).key >> kTopShift) == top) ++hi;
                int r = 0;
                for (long long j = lo; j <= hi; ++j) {
                    const SortElem o = elem_at(j);
                    r += (o.key < e[k].key) || (o.key == e[k].key && o.idx < e[k].idx);
                }
                newpos[k] = lo + r;
            }
            if (crossing) cluster.sync(); else __syncthreads();   // every read of the old order is done
#pragma unroll
            for (int k = 0; k < K; ++k) {
                if ((warp * K + k) * 32 + lane >= n_here) continue;
                const unsigned c = (unsigned)(newpos[k] / per);
                const int l = (int)(newpos[k] - (long long)c * per);
                SortElem *dst = c == crank ? elems + l : cluster.map_shared_rank(elems, c) + l;
                *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(&e[k]);
            }
            if (crossing) cluster.sync(); else __syncthreads();   // every element is at its place
#pragma unroll
            for (int k = 0; k < K; ++k) e[k] = elems[(warp * K + k) * 32 + lane];
        }
        break;
    }
    // a run longer than the local repair takes: start again from the queue as it was loaded, this time with every pass
    first_pass = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) load_elem(k);
    }  // attempts
    if (dead && tid == 0) atomicOr(a.status, CASCADE_ST_ETIMEOUT);
    }  // radix path

    if (a.runs_out) {
        // run mode: the ordered stretch goes to global memory (coalesced), the merge and the admission follow in
        // their own kernels
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const long long gl = (long long)crank * per + (warp * K + k) * 32 + lane;
            if (gl < n_q) a.runs_out[base_slot + gl] = e[k];
        }
        return;
    }
    admit_and_write<T, K>(a, e, per_rt, cluster, wtmp, reinterpret_cast<int *>(base), exall);
    // every remote store of this kernel is followed by a cluster barrier and nothing reads remote
    // shared memory, so a CTA may leave as soon as it is done
}

// ---- queues beyond 32768 requests: ordered runs of 16384, merged by rank, then admission ---------------------
// One cluster cannot hold more than 16 x 4096 elements and its radix passes slow down with the elements per
// thread (6.2 us per pass at 65536 against 2.3 us at 16384).  Larger queues are cut into stretches of 16384 slots;
// one cluster per stretch orders it with the kernel above (all stretches at the same time), every element then
// finds its place among all elements as its position in its own run plus the number of keys below it in the
// other runs (binary searches through L2; runs in front count equal keys too: stable by slot), and one
// cluster reads the merged order back for the admission scans.
constexpr int kRunLen = 16384;

__global__ void __launch_bounds__(256) merge_runs_kernel(const SortElem *__restrict__ runs, SortElem *__restrict__ sorted,
                                                         int n) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const SortElem me = runs[i];
    const int r = i / kRunLen;
    int pos = i - r * kRunLen;
    // the searches through the other runs advance in step: their loads (L2 latency each) do not depend on one another,
    // so a round of the loop costs one latency instead of one per run
    constexpr int kMaxRuns = CASCADE_MAX_REQUESTS / kRunLen;
    int lo[kMaxRuns], len[kMaxRuns];
    bool more = false;
#pragma unroll
    for (int q = 0; q < kMaxRuns; ++q) {
        lo[q] = 0;
        len[q] = (q == r || q * kRunLen >= n) ? 0 : min(kRunLen, n - q * kRunLen);
        more |= len[q] > 0;
    }
    while (more) {
        unsigned long long v[kMaxRuns];
#pragma unroll
        for (int q = 0; q < kMaxRuns; ++q)
            if (len[q] > 0) v[q] = runs[(size_t)q * kRunLen + lo[q] + (len[q] >> 1)].key;
        more = false;
#pragma unroll
        for (int q = 0; q < kMaxRuns; ++q) {
            if (len[q] > 0) {
                const int half = len[q] >> 1;
                const bool below = q < r ? v[q] <= me.key : v[q] < me.key;   // runs in front count equal keys too
                lo[q] = below ? lo[q] + half + 1 : lo[q];
                len[q] = below ? len[q] - half - 1 : half;
                more |= len[q] > 0;
            }
        }
    }
#pragma unroll
    for (int q = 0; q < kMaxRuns; ++q) pos += lo[q];
    sorted[pos] = me;
}

template <int T, int K>
__global__ void __launch_bounds__(T, 1) admit_kernel(const __grid_constant__ ScheduleArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int per = T * K;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    __shared__ long long wtmp[3 * 32];
    __shared__ int itmp[32];
    __shared__ Exch exall[kMaxCluster];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (crank == 0 && tid == 0) {
        a.counts->n_admitted = 0;
        a.counts->tokens_granted = 0;
    }
    cluster.barrier_arrive();
    SortElem e[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long g = (long long)crank * per + (warp * K + k) * 32 + lane;
        if (g < a.n) e[k] = a.sorted_in[g];
        else { e[k].key = ~0ull; e[k].idx = 0xffffffffu; e[k].want = 0; }
    }
    cluster.barrier_wait();   // every CTA has started (and the counts are zero) before anybody writes to a neighbour
    admit_and_write<T, K>(a, e, per, cluster, wtmp, itmp, exall);
}

// ---- merge-rank ordering: queues that fit one CTA's shared memory as bare keys (up to 16384) -------------
// The radix passes above pay two cluster-wide exchanges per digit.  Here every CTA first orders ITS OWN
// T*K elements with the same stable radix passes run entirely inside the CTA (no exchange), then the sorted
// key lists of all CTAs are gathered into every CTA's shared memory (one exchange), each element finds its
// global position as the sum, over the lists, of the number of keys below it (binary searches in shared memory;
// lists of CTAs in front count equal keys too, which keeps the order stable by slot), and ONE more exchange
// sends every element to its place.  Two exchanges in total instead of sixteen.
constexpr int kMergeMaxKeys = 16384;

template <int T, int K>
__global__ void __launch_bounds__(T, 1) schedule_merge_kernel(const __grid_constant__ ScheduleArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    constexpr int W = T / 32;
    constexpr int per = T * K;
    static_assert((per & (per - 1)) == 0, "the searches assume lists of a power-of-two length");
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned crank = cluster.block_rank();
    const unsigned csize = cluster.num_blocks();

    extern __shared__ __align__(16) unsigned char smem[];
    SortElem *elems = reinterpret_cast<SortElem *>(smem);                              // [per]
    uint64_t *keys_all = reinterpret_cast<uint64_t *>(elems + per);                    // [csize][per], sorted lists
    uint16_t *whist = reinterpret_cast<uint16_t *>(keys_all + kMergeMaxKeys);          // [W][kWhistStride]
    uint32_t *lbase = reinterpret_cast<uint32_t *>(whist + W * kWhistStride);          // [kBins]
    long long *wtmp = reinterpret_cast<long long *>(lbase + kBins);                    // 3 * 32 entries
    Exch *exall = reinterpret_cast<Exch *>(wtmp + 3 * 32);                             // [kMaxCluster]
    int *itmp = reinterpret_cast<int *>(exall + kMaxCluster);                          // [32]
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(itmp + 32);      // keys, elements

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int n = a.n;
    // elements of the final order that land in this CTA
    const long long mine_ll = (long long)n - (long long)crank * per;
    const int n_mine = mine_ll < 0 ? 0 : (mine_ll > per ? per : (int)mine_ll);

    if (crank == 0 && tid == 0) {
        a.counts->n_admitted = 0;
        a.counts->tokens_granted = 0;
    }
    const unsigned keys_bar = cta_smem_addr(&bars[0]), elem_bar = cta_smem_addr(&bars[1]);
    if (tid == 0) {
        mbarrier_init(keys_bar, 1);
        mbarrier_init(elem_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbarrier_arrive_expect(keys_bar, (csize - 1) * (unsigned)(per * sizeof(uint64_t)));
        mbarrier_arrive_expect(elem_bar, (unsigned)(n_mine * sizeof(SortElem)));
    }
    cluster.barrier_arrive();   // waited for in front of the first store into another CTA's shared memory

    // ---- load: key, slot, tokens wanted -------------------------------------------------------------
    SortElem e[K];
    unsigned long long diff = 0, key_first = 0;
    {
        const long long g0 = (long long)crank * per;
        key_first = g0 < n ? a.key[g0] : 0ull;
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int li = (warp * K + k) * 32 + lane;
        const long long g = (long long)crank * per + li;
        if (g < n) {
            const unsigned long long key = a.key[g];
            const long long P = a.prompt[g], h0 = a.n0[g], h1 = a.n1[g], h2 = a.n2[g];
            long long want = 0;
            if (dev_request_valid(a.bt, P, h0, h1, h2)) want = a.want_in ? a.want_in[g] : P - (h0 + h1 + h2) * a.bt;
            e[k].key = key;
            e[k].idx = (uint32_t)g;
            e[k].want = (int32_t)want;
            diff |= key ^ key_first;
        } else {
            e[k].key = ~0ull;  // padding sorts behind every real key of this CTA and stays there (stable passes)
            e[k].idx = 0xffffffffu;
            e[k].want = 0;
        }
    }
    // bits in which this CTA's keys differ: passes over other digits would move nothing
    {
        unsigned lo = __reduce_or_sync(kFull, (unsigned)diff);
        unsigned hi = __reduce_or_sync(kFull, (unsigned)(diff >> 32));
        if (lane == 0) wtmp[warp] = (long long)(((unsigned long long)hi << 32) | lo);
        __syncthreads();
        unsigned long long v = 0;
#pragma unroll
        for (int w = 0; w < W; ++w) v |= (unsigned long long)wtmp[w];
        diff = v;
        __syncthreads();
    }

    // ---- local order: stable LSD radix passes inside the CTA ---------------------------------------------
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = pass * 8;
        if (((diff >> shift) & 0xffull) == 0) continue;
        // (a) stable rank of each element among equal digits of its warp's 32*K elements
        uint16_t *myhist = whist + warp * kWhistStride;
        for (int i = lane; i < kWhistStride / 2; i += 32) reinterpret_cast<uint32_t *>(myhist)[i] = 0;
        __syncwarp();
        unsigned off[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
            unsigned peers = kFull;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const unsigned bal = __ballot_sync(kFull, (d >> b) & 1u);
                peers &= ((d >> b) & 1u) ? bal : ~bal;
            }
            const unsigned lower = peers & lt_mask;
            const unsigned pre = myhist[d];
            __syncwarp();
            if (lower == 0) myhist[d] = (uint16_t)(pre + __popc(peers));
            __syncwarp();
            off[k] = pre + __popc(lower);
        }
        __syncthreads();
        // (b) per digit: exclusive scan of the warps' counts in place, CTA total, then the scan over the digits
        unsigned mine = 0, incl = 0;
        if (tid < kBins) {
            unsigned v[W];
#pragma unroll
            for (int w = 0; w < W; ++w) v[w] = whist[w * kWhistStride + tid];
#pragma unroll
            for (int w = 0; w < W; ++w) {
                whist[w * kWhistStride + tid] = (uint16_t)mine;
                mine += v[w];
            }
            incl = seg_incl_scan(mine, lane, 32);
            if (lane == 31) reinterpret_cast<unsigned *>(wtmp)[warp] = incl;
        }
        __syncthreads();
        if (tid < kBins) {
            unsigned add = 0;
#pragma unroll
            for (int w = 0; w < kBins / 32; ++w) {
                const unsigned t = reinterpret_cast<unsigned *>(wtmp)[w];
                if (w < warp) add += t;
            }
            lbase[tid] = incl - mine + add;
        }
        __syncthreads();
        // (c) every element to its place, then back into registers in position order
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const unsigned d = (unsigned)(e[k].key >> shift) & 0xffu;
            const unsigned pos = lbase[d] + whist[warp * kWhistStride + d] + off[k];
            *reinterpret_cast<uint4 *>(elems + pos) = *reinterpret_cast<const uint4 *>(&e[k]);
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < K; ++k) e[k] = elems[(warp * K + k) * 32 + lane];
    }

    // ---- gather the sorted key lists of all CTAs -----------------------------------------------------------
    uint64_t *my_list = keys_all + (size_t)crank * per;
#pragma unroll
    for (int k = 0; k < K; ++k) my_list[(warp * K + k) * 32 + lane] = e[k].key;
    // first access to other CTAs' shared memory: they must all have started and initialised their barriers
    __syncthreads();
    cluster.barrier_wait();
    for (unsigned op = tid; op < (csize - 1) * (per / 2); op += T) {
        unsigned dst = op / (per / 2);
        const unsigned piece = op % (per / 2);
        dst += dst >= crank;   // everybody but myself
        const uint4 v = *reinterpret_cast<const uint4 *>(my_list + piece * 2);
        st_async_16(cluster_addr(cta_smem_addr(my_list + piece * 2), dst), v, cluster_addr(keys_bar, dst));
    }
    bool dead = !mbarrier_wait_bounded(keys_bar, 0, kWaitLimit);
    if (__syncthreads_or(dead)) dead = true;

    // ---- global position: keys below mine in every list --------------------------------------------------
    if (!dead) {
        unsigned pos[K];
#pragma unroll
        for (int k = 0; k < K; ++k) pos[k] = (warp * K + k) * 32 + lane;   // own list: the local position
        // four lists at a time: their searches advance in step, so the shared-memory latency of a round is paid once
        // for the four of them (the own list is searched along and left out of the sum; csize is a power of two)
        constexpr int G = 4;
        for (unsigned c0 = 0; c0 < csize; c0 += G) {
            unsigned p[G][K];
            const uint64_t *list[G];
            bool ties[G], counted[G];
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const unsigned c = c0 + j < csize ? c0 + j : csize - 1;
                list[j] = keys_all + (size_t)c * per;
                ties[j] = c < crank;       // equal keys of CTAs in front hold lower slots: they come first
                counted[j] = c0 + j < csize && c != crank;
#pragma unroll
                for (int k = 0; k < K; ++k) p[j][k] = 0;
            }
#pragma unroll
            for (int s = per / 2; s > 0; s >>= 1) {
#pragma unroll
                for (int j = 0; j < G; ++j) {
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        const uint64_t v = list[j][p[j][k] + s - 1];
                        p[j][k] += (ties[j] ? v <= e[k].key : v < e[k].key) ? s : 0;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < G; ++j) {
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const uint64_t v = list[j][p[j][k]];
                    p[j][k] += (ties[j] ? v <= e[k].key : v < e[k].key) ? 1 : 0;
                    if (counted[j]) pos[k] += p[j][k];
                }
            }
        }
        // ---- every real element to its place (padding stays behind: nobody reads the slots past n) ----------
#pragma unroll
        for (int k = 0; k < K; ++k) {
            if (e[k].idx == 0xffffffffu) continue;
            st_async_16(cluster_addr(cta_smem_addr(elems + (pos[k] % per)), pos[k] / per),
                        *reinterpret_cast<const uint4 *>(&e[k]), cluster_addr(elem_bar, pos[k] / per));
        }
        dead = !mbarrier_wait_bounded(elem_bar, 0, kWaitLimit);
    }
    if (__syncthreads_or(dead)) dead = true;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int li = (warp * K + k) * 32 + lane;
        if (!dead && li < n_mine) e[k] = elems[li];
        else { e[k].key = ~0ull; e[k].idx = 0xffffffffu; e[k].want = 0; }
    }
    if (dead && tid == 0) atomicOr(a.status, CASCADE_ST_ETIMEOUT);
    admit_and_write<T, K>(a, e, per, cluster, wtmp, itmp, exall);
}

__global__ void zero_counts_kernel(cascade_sched_counts *c) {
    c->n_tier1 = 0;
    c->n_admitted = 0;
    c->tokens_granted = 0;
}

size_t smem_bytes(int T, int K) {
    return (T == 256 && K == 1 ? kRankExtra : 0) + 2 * size_t(T) * K * sizeof(SortElem) + size_t(T / 32) * kWhistStride * sizeof(uint16_t) +
           2 * size_t(kMaxCluster) * kBins * sizeof(uint16_t) + 2 * kBins * sizeof(uint32_t) +
           3 * 32 * sizeof(long long) + kMaxCluster * sizeof(Exch) + kBins * sizeof(uint16_t) + 4 * 8 +
           kMaxCluster * sizeof(TieExch) + 16;
}

template <int T, int K>
cudaError_t launch(const ScheduleArgs &a, int cluster_size, int device, bool pdl, cudaStream_t stream, int n_clusters = 1) {
    static CascadeDeviceOnce configured;
    const size_t smem = smem_bytes(T, K);
    if (!configured.is_set(device)) {
        cudaError_t e = cudaFuncSetAttribute(schedule_kernel<T, K>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(schedule_kernel<T, K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured.set(device);
    }
    return cascade_launch(pdl, cluster_size, dim3(cluster_size * n_clusters), dim3(T), smem, stream, schedule_kernel<T, K>, a);
}

size_t merge_smem_bytes(int T, int K) {
    return size_t(T) * K * sizeof(SortElem) + size_t(kMergeMaxKeys) * sizeof(uint64_t) +
           size_t(T / 32) * kWhistStride * sizeof(uint16_t) + kBins * sizeof(uint32_t) + 3 * 32 * sizeof(long long) +
           kMaxCluster * sizeof(Exch) + 32 * sizeof(int) + 2 * 8 + 16;
}

template <int K>
cudaError_t launch_merge(const ScheduleArgs &a, int cluster_size, int device, bool pdl, cudaStream_t stream) {
    static CascadeDeviceOnce configured;
    const size_t smem = merge_smem_bytes(256, K);
    if (!configured.is_set(device)) {
        cudaError_t e = cudaFuncSetAttribute(schedule_merge_kernel<256, K>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(schedule_merge_kernel<256, K>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured.set(device);
    }
    return cascade_launch(pdl, cluster_size, dim3(cluster_size), dim3(256), smem, stream, schedule_merge_kernel<256, K>, a);
}

cudaError_t launch_merge_k(int K, const ScheduleArgs &a, int C, int device, bool pdl, cudaStream_t s) {
    switch (K) {
        case 1: return launch_merge<1>(a, C, device, pdl, s);
        case 2: return launch_merge<2>(a, C, device, pdl, s);
        case 4: return launch_merge<4>(a, C, device, pdl, s);
        default: return launch_merge<8>(a, C, device, pdl, s);
    }
}

template <int T>
cudaError_t launch_k(int K, const ScheduleArgs &a, int C, int device, bool pdl, cudaStream_t s) {
    switch (K) {
        case 1: return launch<T, 1>(a, C, device, pdl, s);
        case 2: return launch<T, 2>(a, C, device, pdl, s);
        case 4: return launch<T, 4>(a, C, device, pdl, s);
        default: return launch<T, 8>(a, C, device, pdl, s);
    }
}

}  // namespace

// Largest cluster the device will co-schedule for the ordering kernel (its shared-memory footprint is
// the largest of the cluster kernels); 16 on a full B200, less on partitioned or smaller parts.
int cascade_probe_max_cluster() {
    cudaFuncSetAttribute(schedule_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(256, 8));
    cudaFuncSetAttribute(schedule_kernel<256, 1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(16, 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes(256, 8);
    int size = 0;
    if (cudaOccupancyMaxPotentialClusterSize(&size, schedule_kernel<256, 1>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 8;  // the portable maximum
    }
    // restore the kernel's own footprint for later launches
    cudaFuncSetAttribute(schedule_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(256, 1));
    return size < 1 ? 1 : (size > 16 ? 16 : size);
}

extern "C" int cascade_schedule(cascade_ctx *ctx, const cascade_reqs *r, const uint64_t *key, int n, int32_t D_act,
                                uint32_t *order_out, int32_t *grant_out, cascade_sched_counts *counts_dev,
                                void *stream) {
    CascadeRange nvtx_range("cascade_schedule");
    if (!ctx || !r || n < 0 || n > ctx->max_requests || !counts_dev) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (D_act < 0 || D_act > (1 << 16)) return CASCADE_ERANGE;
    cudaStream_t s = (cudaStream_t)stream;
    if (n == 0) {
        zero_counts_kernel<<<1, 1, 0, s>>>(counts_dev);
        CASCADE_CUDA_TRY(ctx, cudaGetLastError());
        return CASCADE_OK;
    }
    if (!key || !order_out || !grant_out || !r->prompt || !r->n0 || !r->n1 || !r->n2) return CASCADE_EINVAL;
    const cascade_params &p = ctx->params;
    int T, C, K;
    if (!cascade_pick_geometry(ctx, n, &T, &C, &K)) return CASCADE_EINVAL;
    ScheduleArgs a;
    a.key = key;
    a.prompt = r->prompt;
    a.n0 = r->n0;
    a.n1 = r->n1;
    a.n2 = r->n2;
    a.want_in = p.plan_first ? ctx->want_by_slot : nullptr;
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
    a.stage = ctx->sort_stage >= 0 ? ctx->sort_stage : (K >= 4);
    a.async_sync = ctx->sort_async;
    // the comparison policies order by small integers (tokens left, ...): equal values are the rule there
    a.top_first = ctx->sort_top_first && p.policy == CASCADE_POLICY_BUDGET;
    a.rank_per = 0;
    if (n <= ctx->rank_sort_max && n <= kRankMaxKeys) {
        // counting path: the widest cluster the device schedules, 256 threads, 32..256 elements per CTA
        const int c = ctx->max_cluster > 0 ? (ctx->max_cluster < 16 ? ctx->max_cluster : 16) : 16;
        int per_rank = (n + c - 1) / c;
        per_rank = per_rank <= 32 ? 32 : (per_rank <= 64 ? 64 : (per_rank <= 128 ? 128 : 256));
        if ((long long)per_rank * c >= n && per_rank <= 256) {
            T = 256;
            K = 1;
            C = 1;
            while (C * per_rank < n) C *= 2;      // cluster sizes stay powers of two; CTAs past the data hold padding
            a.rank_per = per_rank;
        }
    }
    a.status = ctx->status_dev;
    a.runs_out = nullptr;
    a.sorted_in = nullptr;
    if (ctx->sort_runs && ctx->multi_sort && n > (ctx->multi_sort == 2 ? kRunLen : 2 * kRunLen)) {
        // stretches of 16384 slots ordered by one cluster each, merged by rank, admission by one cluster
        const int n_runs = (n + kRunLen - 1) / kRunLen;
        ScheduleArgs r = a;
        r.runs_out = reinterpret_cast<SortElem *>(ctx->sort_runs);
        r.stage = ctx->sort_stage >= 0 ? ctx->sort_stage : 1;
        CASCADE_CUDA_TRY(ctx, (launch<256, 4>(r, 16, ctx->device, ctx->pdl, s, n_runs)));
        SortElem *sorted = reinterpret_cast<SortElem *>(ctx->sort_sorted);
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((n + 255) / 256), dim3(256), 0, s, merge_runs_kernel,
                                             (const SortElem *)r.runs_out, sorted, n));
        ScheduleArgs c = a;
        c.sorted_in = sorted;
        static CascadeDeviceOnce configured;
        if (!configured.is_set(ctx->device)) {
            CASCADE_CUDA_TRY(ctx, cudaFuncSetAttribute(admit_kernel<512, 8>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
            configured.set(ctx->device);
        }
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 16, dim3(16), dim3(512), 0, s, admit_kernel<512, 8>, c));
        return CASCADE_OK;
    }
    // queues beyond the counting path whose bare keys fit one CTA's shared memory: local order + merge by rank
    // (measured: a gain while every thread holds one element, i.e. up to 4096 requests; beyond that the searches
    // cost more than the exchanges they save, unless CASCADE_MERGE_SORT=2 forces it)
    const bool merge = ctx->merge_sort && a.rank_per == 0 && T == 256 && (long long)C * T * K <= kMergeMaxKeys &&
                       (K == 1 || ctx->merge_sort == 2);
    cudaError_t e = merge      ? launch_merge_k(K, a, C, ctx->device, ctx->pdl, s)
                    : T == 256 ? launch_k<256>(K, a, C, ctx->device, ctx->pdl, s)
                               : launch_k<512>(K, a, C, ctx->device, ctx->pdl, s);
    CASCADE_CUDA_TRY(ctx, e);
    return CASCADE_OK;
}
