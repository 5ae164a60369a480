/*
 * libcascade: the per-iteration, budget-driven scheduling and KV-tier step of the Cascade
 * serving loop as hand-written CUDA kernels for sm_100a (NVIDIA B200), behind a C ABI.
 *
 * One iteration = five stream-ordered calls on ONE stream, no host synchronisation between them:
 *
 *   cascade_budget     per-request latency budget and 64-bit priority key      (Eq. 3, Eq. 4, Eq. 5)
 *   cascade_schedule   least-remaining-budget-first order + admission          (Algorithm 1, phase 2)
 *   cascade_tier_plan  restore bound, restore/retain/recompute, preemption     (Eq. 6, Eq. 7, Algorithm 1)
 *   cascade_kv_evict   paged HBM blocks  -> contiguous host records            (preemption under HBM pressure)
 *   cascade_kv_restore contiguous host records -> paged HBM blocks             (TriggerPrefetch of Algorithm 1)
 *
 * Optional steps on the same stream: cascade_prefetch_plan (prefetch for queued requests), cascade_stage_plan +
 * cascade_kv_stage (first hop of a deep-tier fetch), cascade_dedup (one copy per shared block), cascade_kv_move
 * (evict and restore in one call).
 *
 * Conventions
 *   - Every time is an int64 number of nanoseconds, every token / block count an int32, every
 *     cost coefficient a Q20 fixed-point int64 (value * 2^20).  All results are exact integers.
 *   - Unless a parameter says "host", a pointer is a DEVICE pointer owned by the caller; a pinned,
 *     mapped host allocation (cudaHostAlloc / torch pin_memory) counts as device-accessible.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - The library allocates device memory only in cascade_create.  The five hot calls allocate
 *     nothing, never synchronise the host and use no stream of their own (the one exception, by its
 *     nature, is cascade_kv_move_staged: it drives the copy engines from the host).
 *   - One context per stream.  A context is not thread-safe, and its calls must not run on two streams at
 *     the same time either (order them with events if they are issued to different streams): the kernels
 *     of one context share scratch, the plan's work lists and the copy kernels' work counters.
 *   - Return value: 0 on success, a negative CASCADE_E* code for errors found on the host before
 *     anything is launched.  Conditions found on the device never trap; they OR a CASCADE_ST_* bit
 *     into the context's sticky status word, read with cascade_status.
 */
#ifndef CASCADE_H
#define CASCADE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CASCADE_MAX_CLASSES 8
#define CASCADE_MAX_REQUESTS 65536 /* largest queue one context can order */

/* host-side return codes */
#define CASCADE_OK 0
#define CASCADE_EINVAL (-1) /* NULL pointer, negative or oversized count, bad alignment            */
#define CASCADE_ERANGE (-2) /* a parameter outside the overflow-safe bounds listed below           */
#define CASCADE_ECUDA (-3)  /* a CUDA runtime call failed; its code is kept in cascade_status_t    */
#define CASCADE_ENOMEM (-4) /* cascade_create could not allocate its scratch                       */
#define CASCADE_ETOOBIG (-5) /* a size beyond a fixed maximum of the entry point (see the _noalloc call) */

/* device-side sticky status bits */
#define CASCADE_ST_EBOUNDS 1u   /* a block id or list length outside its pool: that item was skipped   */
#define CASCADE_ST_ENOSPC 2u    /* HBM could not hold the admitted set: it was cut from the tail       */
#define CASCADE_ST_ETIMEOUT 4u  /* a bounded wait inside a kernel expired                              */
#define CASCADE_ST_EPRECOND 8u  /* a request outside the input bounds: it was parked / ignored         */
#define CASCADE_ST_ELISTCAP 16u /* a copy list was too short: entries beyond its capacity were dropped */

/* request flags */
#define CASCADE_FLAG_HBM_PRIVATE 1u /* the request's n0 HBM blocks are its own and may be preempted */
#define CASCADE_FLAG_RUNNING 2u     /* informational: partially prefilled                            */

/* per-request action written by cascade_tier_plan */
#define CASCADE_ACT_NONE 0u   /* holds no HBM block                                  */
#define CASCADE_ACT_RETAIN 1u /* keeps its HBM blocks                                */
#define CASCADE_ACT_EVICT 2u  /* preempted, KV spilled to host (on the evict list)   */
#define CASCADE_ACT_DROP 3u   /* preempted, KV discarded (recomputed on re-execution) */

/*
 * Cost model and policy parameters (host struct, copied at cascade_create).
 * The paper's TTFT estimator is an offline-trained model with no printed form; this library
 * uses an integer polynomial:
 *   iter_q(D,K)   = c_iter + D*c_dseq + K*c_dkv            one engine iteration with D decodes over K KV tokens
 *   A(D,K)        = c_tok + (iter_q(D,K) >> chunk_shift)   per prefill token
 *   comp_q(A,P,s) = A*(P-s) + c_attn*(P*P - s*s)           prefill of prompt tokens [s,P)
 *   T_k(x)        = x ? delta_ns[k] + x*blk_ns[k] : 0      Eq. 6 in blocks, k = 1 host DRAM, 2 deep tier
 * Overflow-safe bounds (checked, CASCADE_ERANGE): 1 <= bt <= 4096, 0 <= chunk_shift <= 20,
 * 1 <= max_batch <= 65536, 0 <= max_ctx_avg <= 2^20, (max_batch-1)*max_ctx_avg <= 2^32,
 * 0 <= gamma_q16 <= 2^17, 1 <= n_classes <= 8, 0 <= token_budget <= 2^30, 0 <= tier2_reserve,
 * 0 <= c_tok_q20 <= 2^40, 0 <= c_attn_q20 <= 2^20, 0 <= c_iter_q20 <= 2^50, 0 <= c_dseq_q20 <= 2^40,
 * 0 <= c_dkv_q20 <= 2^28, 0 <= delta_ns[k] <= 2^30, 1 <= blk_ns[k] <= 2^27, 0 <= ttft_ns, tpot_ns <= 2^40.
 * Per call: 0 <= D_act <= 2^16, 0 <= K_act <= 2^32.
 */
typedef struct cascade_params {
    int32_t bt;            /* tokens per KV block                                              */
    int32_t chunk_shift;   /* prefill chunk = 2^chunk_shift tokens                             */
    int32_t max_batch;     /* B_max: sequences per engine iteration, decodes included          */
    int32_t max_ctx_avg;   /* KV tokens per decode sequence assumed in the maximum-load regime */
    int32_t gamma_q16;     /* guardband gamma of Eq. 3, times 2^16                             */
    int32_t n_classes;
    int32_t token_budget;  /* tokens per engine iteration (decodes take one each)              */
    int32_t tier2_reserve; /* tokens of every iteration kept for the Tier-2 queue              */
    int64_t c_tok_q20, c_attn_q20, c_iter_q20, c_dseq_q20, c_dkv_q20;
    int64_t delta_ns[3];   /* Eq. 6: fixed overheads summed over path P(k); [0] unused         */
    int64_t blk_ns[3];     /* Eq. 6: time per block summed over path P(k); [0] unused          */
    int64_t ttft_ns[CASCADE_MAX_CLASSES]; /* class TTFT targets                                */
    int64_t tpot_ns[CASCADE_MAX_CLASSES]; /* class TPOT targets; 0 disables the decode term    */
    int32_t policy;        /* CASCADE_POLICY_*: what the queue is ordered by (0 = the paper's method)     */
    int32_t plan_first;    /* 0 | 1: plan-first admission, see below                                       */
} cascade_params;

/* Ordering policies.  BUDGET is the method: least remaining budget first with the Tier-1 / Tier-2 split.
 * The others are the comparison policies of the paper's evaluation, one queue, same key packing:
 * FCFS orders by arrival time, EDF by the TTFT deadline arrival + ttft_ns[cls], SJF by the tokens left
 * to prefill.  budget_out is the latency budget under every policy (the tier plan needs it). */
/* plan_first = 1: every request's own restore choice (the Eq. 7 bounds and the restore-vs-recompute
 * comparison of cascade_tier_plan, taken from its budget alone) is made before admission, and admission
 * offers it exactly the tokens that choice leaves to compute, prompt - (n0 + x1)*bt, instead of assuming
 * the whole matched prefix is reused; a request that chooses a deep-tier fetch asks for nothing this
 * iteration.  Every admitted request then runs exactly its grant.  cascade_budget stores the offers in the
 * context, so cascade_schedule must follow cascade_budget on the same context and request arrays. */
#define CASCADE_POLICY_BUDGET 0
#define CASCADE_POLICY_FCFS 1
#define CASCADE_POLICY_EDF 2
#define CASCADE_POLICY_SJF 3

/*
 * The request queue as a structure of arrays (host struct of device pointers, n entries each).
 * Per-request bounds (a violation parks the request and sets CASCADE_ST_EPRECOND):
 * 1 <= prompt <= 2^17, 0 <= pred_out <= 2^20, n0,n1,n2 >= 0, n0+n1+n2 <= 2^13,
 * (n0+n1+n2)*bt < prompt, cls < n_classes, |now - arrival| <= 2^50.
 */
typedef struct cascade_reqs {
    const int64_t *arrival_ns; /* arrival timestamp a_r                                         */
    const int32_t *prompt;     /* prompt length in tokens                                       */
    const int32_t *pred_out;   /* predicted output length in tokens                             */
    const int32_t *n0;         /* matched prefix blocks resident in HBM (table positions 0..n0) */
    const int32_t *n1;         /* next matched blocks held in host DRAM                         */
    const int32_t *n2;         /* next matched blocks held in the deep tier (priced only)       */
    const uint32_t *id;        /* arrival id; ties in budget are broken by its low 23 bits      */
    const uint8_t *cls;        /* SLO class                                                     */
    const uint8_t *flags;      /* CASCADE_FLAG_*                                                */
} cascade_reqs;

/* written to device memory by cascade_schedule */
typedef struct cascade_sched_counts {
    int32_t n_tier1;        /* requests in the Tier-1 queue (budget of Eq. 4 positive) */
    int32_t n_admitted;     /* requests with grant > 0                                 */
    int64_t tokens_granted; /* sum of grants                                           */
} cascade_sched_counts;

/* written to device memory by cascade_tier_plan */
typedef struct cascade_plan_counts {
    int32_t n_restore;       /* entries of the restore list (blocks)            */
    int32_t n_evict;         /* entries of the evict list (blocks)              */
    int32_t n_drop_blocks;   /* HBM blocks freed without a copy                 */
    int32_t n_victims;       /* requests preempted (EVICT or DROP)              */
    int32_t n_unadmitted;    /* requests un-admitted by the HBM capacity check  */
    int32_t n_admitted;      /* requests still admitted after the plan          */
    int32_t hbm_need;        /* new HBM blocks the admitted set takes           */
    int32_t deficit;         /* blocks that had to be freed                     */
    int32_t hbm_free_after;  /* HBM free-list length after the plan             */
    int32_t host_free_after; /* host free-list length after the plan            */
    int64_t tokens_run;      /* tokens the admitted set computes this iteration */
} cascade_plan_counts;

/*
 * Block tables and free lists (host struct of device pointers).  Read AND updated by
 * cascade_tier_plan.  Tables are row-major [n][maxb] int32, -1 = no block: hbm_tbl[r][j] is the
 * HBM block holding tokens [j*bt,(j+1)*bt) of request r, host_tbl[r][j] its host record.
 * Free lists are stacks: the next id handed out is list[count-1].  hbm_free must have room for
 * every block that can be freed (capacity = number of HBM blocks is always enough).
 * hbm_tbl == NULL selects plan-only mode: decisions and counts are produced from the two counts
 * alone; no table, free list, count or copy list is touched.
 */
typedef struct cascade_pools {
    int32_t *hbm_tbl;
    int32_t *host_tbl;
    int32_t maxb;
    int32_t *hbm_free;
    int32_t *hbm_free_count; /* device scalar, updated */
    int32_t hbm_free_cap;
    int32_t *host_free;
    int32_t *host_free_count; /* device scalar, updated */
    int32_t host_free_cap;
} cascade_pools;

/* Outputs of cascade_tier_plan (host struct of device pointers; arrays of n, lists of *_cap). */
typedef struct cascade_plan {
    int32_t *x1;         /* host blocks to restore now                          */
    int32_t *x2;         /* deep-tier blocks to stage (priced and planned only) */
    int32_t *tokens_run; /* prompt tokens computed this iteration               */
    uint8_t *action;     /* CASCADE_ACT_*                                       */
    int32_t *restore_src; /* host record ids, in schedule order                 */
    int32_t *restore_dst; /* HBM block ids                                      */
    int32_t restore_cap;
    int32_t *evict_src;   /* HBM block ids, in preemption order                 */
    int32_t *evict_dst;   /* host record ids                                    */
    int32_t evict_cap;
    cascade_plan_counts *counts; /* device */
} cascade_plan;

/*
 * Geometry of the paged HBM pool.  Byte address of chunk c (0..n_chunks-1, one per layer and K/V
 * plane) of block b: c*chunk_stride + b*block_stride.  A layer-major pool has block_stride =
 * chunk_bytes and chunk_stride = n_blocks*chunk_bytes; a block-major pool has chunk_stride =
 * chunk_bytes and block_stride = n_chunks*chunk_bytes.  The host pool (or a device staging buffer
 * standing in for it) is always record-major: record h occupies [h*bb, (h+1)*bb) with
 * bb = n_chunks*chunk_bytes, its chunks back to back.
 * chunk_bytes, both strides and both pool base addresses must be multiples of 16.
 */
typedef struct cascade_kv_layout {
    int64_t n_blocks;
    int32_t n_chunks;
    int32_t reserved;
    int64_t chunk_bytes;
    int64_t chunk_stride;
    int64_t block_stride;
} cascade_kv_layout;

typedef struct cascade_status_t {
    uint32_t bits;       /* OR of CASCADE_ST_* seen since the last clear */
    int32_t cuda_error;  /* last failing cudaError_t, 0 if none          */
} cascade_status_t;

typedef struct cascade_ctx cascade_ctx;

/* Creates a context on `device` for queues of up to max_requests (<= CASCADE_MAX_REQUESTS, and
 * <= 4096 times the largest thread-block cluster the device co-schedules: 16 on a full B200).
 * Validates the parameters against the bounds above.  Allocates scratch (about 44 bytes per request, 76 for
 * contexts of more than 16384 requests), four side streams and seven events for the copy-engine path.
 * `p` and `out` are host pointers.  The calling thread's current device is left as it was; the hot calls
 * launch on the current device, so make `device` current (and pass one of its streams) when calling them:
 * a call made while another device is current returns CASCADE_EINVAL and launches nothing. */
int cascade_create(cascade_ctx **out, const cascade_params *p, int max_requests, int device);
void cascade_destroy(cascade_ctx *ctx);
/* Replaces the parameters (same validation); takes effect for calls made afterwards. */
int cascade_set_params(cascade_ctx *ctx, const cascade_params *p);

/*
 * Latency budget and priority key of every request (one thread per request).
 *   L      = ((L_act + L_max) * gamma) / 2                      Eq. 3, with L_rho = T_1(n1) + T_2(n2) +
 *            comp_q(A(rho), prompt, (n0+n1+n2)*bt) for the actual load rho = (D_act, K_act) and the
 *            maximum load (max(D_act, max_batch-1), max(K_act, (max_batch-1)*max_ctx_avg))
 *   B      = ttft_ns[cls] - L                                   Eq. 4;  B > 0 -> Tier-1 queue, else Tier-2
 *   B_rem  = B - (now_ns - arrival_ns)                          Eq. 5
 *   budget = B_rem - pred_out * max(0, t_dec - tpot_ns[cls])    decode-overrun penalty, 0 if tpot_ns == 0
 *   key    = tier2 << 63 | (clamp(budget, -2^39, 2^39-1) + 2^39) << 23 | (id & 0x7FFFFF)
 * budget_out[n] and key_out[n] are written (caller-owned device arrays).
 * Errors: CASCADE_EINVAL (NULL pointer, n < 0, n > max_requests), CASCADE_ERANGE (D_act or K_act outside the
 * bounds above), CASCADE_ECUDA (launch failed).  On the device: a request outside the input bounds, with a class
 * index >= n_classes or with |now - arrival| > 2^50 gets budget -2^62 and the key (1 << 63 | id), i.e. the very
 * end of the Tier-2 queue, and sets CASCADE_ST_EPRECOND.
 */
int cascade_budget(cascade_ctx *ctx, const cascade_reqs *r, int n, int64_t now_ns, int32_t D_act, int64_t K_act,
                   int64_t *budget_out, uint64_t *key_out, void *stream);

/*
 * The TTFT estimator's four operating regimes for every request (Section "TTFT Latency Estimator"):
 *   lat4_out[4*r + 0]  zero load, full recomputation            (L^zero_recomp)
 *   lat4_out[4*r + 1]  actual load, full recomputation          (L^act_recomp)
 *   lat4_out[4*r + 2]  actual load, tier-aware prefix reuse     (L^actual of Eq. 3)
 *   lat4_out[4*r + 3]  maximum load, tier-aware prefix reuse    (L^max of Eq. 3)
 * in ns, from the same integer model cascade_budget uses.  A request outside the input bounds gets
 * four zeros and CASCADE_ST_EPRECOND.  Diagnostic: not part of the per-iteration path.
 */
int cascade_latency_regimes(cascade_ctx *ctx, const cascade_reqs *r, int n, int32_t D_act, int64_t K_act,
                            int64_t *lat4_out, void *stream);

/*
 * Queue maintenance (the paper has no counterpart; "the only per-iteration write is the priority key" there
 * because its queue lives in host memory): overwrite m slots of the device-resident request arrays.
 *   dst     the queue's arrays (device), cap entries each
 *   src     the new values, m entries each, compact; device-accessible: pinned mapped host memory is read in
 *           place over the host link, which for a few hundred slots is cheaper than staging copies
 *   slots   m destination indices (device-accessible), each < cap; others are skipped (CASCADE_ST_EBOUNDS);
 *           indices must be distinct
 * Stream-ordered like every other call; m = 0 is a no-op.
 */
int cascade_reqs_update(cascade_ctx *ctx, const cascade_reqs *dst, int cap, const cascade_reqs *src,
                        const int32_t *slots, int m, void *stream);

/*
 * Least-remaining-budget-first order and admission (Algorithm 1, phase 2).
 *   order_out[n]  slot indices sorted ascending by key (stable: equal keys keep slot order)
 *   grant_out[n]  tokens granted to each slot this iteration (0 = not admitted): the Tier-1 queue
 *                 is served in order from token_budget - D_act minus the Tier-2 reserve, the Tier-2
 *                 queue from the reserve plus what Tier-1 left; each request is offered
 *                 prompt - (n0+n1+n2)*bt tokens; at most max_batch - D_act requests are admitted.
 *   counts_dev    device struct, written.
 * n = 0 writes zero counts.  A request outside the input bounds is offered nothing.
 * Errors: CASCADE_EINVAL (NULL pointer, n out of range), CASCADE_ERANGE (D_act), CASCADE_ECUDA.  On the device:
 * CASCADE_ST_ETIMEOUT if a bounded wait between the CTAs of the cluster expires (results then undefined).
 */
int cascade_schedule(cascade_ctx *ctx, const cascade_reqs *r, const uint64_t *key, int n, int32_t D_act,
                     uint32_t *order_out, int32_t *grant_out, cascade_sched_counts *counts_dev, void *stream);

/*
 * Tier plan for the admitted set.
 *   - Eq. 7 bound per tier from the request's budget (host first, deep tier from what is left),
 *     then the candidate (nothing / host bound / host + deep bound) with the smallest predicted
 *     completion time  (T_1(x1)+T_2(x2)) + comp(prompt, (n0+x1+x2)*bt); ties restore more.
 *   - HBM capacity: admitted requests whose cumulative block need exceeds free + preemptable are
 *     un-admitted from the tail (`grant` is zeroed for them; CASCADE_ST_ENOSPC).
 *   - Preemption: non-admitted CASCADE_FLAG_HBM_PRIVATE holders, last in the order first, until the
 *     deficit is covered; EVICT when T_1(n0) <= budget and the host pool has room, else DROP.
 *   - Block ids: freed HBM ids are pushed, then admitted requests pop ids for restored and newly
 *     computed blocks; tables, free lists, counts and the two copy lists are updated.
 * `grant` is read and updated.  `pools` and `plan_out` are host structs (copied during the call).
 * The evict list must be executed before the restore list (a freed block may be reused at once).
 * Errors: CASCADE_EINVAL (NULL pointer, n out of range, tables without free lists, negative capacities),
 * CASCADE_ERANGE (D_act, K_act), CASCADE_ECUDA.  On the device: CASCADE_ST_ENOSPC (admitted set cut),
 * CASCADE_ST_EPRECOND (a request outside the input bounds, or whose prompt needs more than maxb table cells:
 * its grant is zeroed and it is never a victim), CASCADE_ST_ELISTCAP (a copy list shorter than the plan:
 * the counts still say how many entries there should have been), CASCADE_ST_EBOUNDS (a free-list count
 * outside [0, capacity]: clamped).
 */
int cascade_tier_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget, const uint32_t *order,
                      int32_t *grant, int n, int32_t D_act, int64_t K_act, const cascade_pools *pools,
                      const cascade_plan *plan_out, void *stream);

/* written to device memory by cascade_prefetch_plan */
typedef struct cascade_prefetch_counts {
    int32_t n_prefetch;      /* blocks appended to the restore list                  */
    int32_t n_requests;      /* queued requests that got at least one block          */
    int32_t hbm_free_after;  /* HBM free-list length afterwards                      */
    int32_t n_restore_total; /* restore-list length afterwards (plan + prefetch)     */
    int64_t link_ns_left;    /* link time left after the admitted set's own restores */
} cascade_prefetch_counts;

/*
 * Budget-bounded prefetch for requests that stay queued: the paper's prefix prefetcher "prefetching
 * required prefix KV states within their budget bounds" (overview of the system; Eq. 6, Eq. 7) applied
 * ahead of admission.  Call it after cascade_tier_plan and before cascade_kv_restore.
 *   Link time left this iteration = link_budget_ns - sum of T_1(x1) over the admitted requests.
 *   Walking `order`, every request that is valid, not admitted (grant <= 0), not preempted by this
 *   iteration's plan (action EVICT / DROP) and holds host blocks (n1 > 0) gets
 *       m = min(n1, Eq. 7 bound from its budget), or 0 if restoring m blocks is predicted slower than
 *           recomputing them,
 *       b = min(m, blocks that still fit the link time left, free HBM blocks above hbm_reserve),
 *   and uses up T_1(b) of link time and b HBM blocks.
 * Outputs: pf_out[n] (blocks prefetched per slot); for each such block an HBM id is popped from
 * hbm_free, written to hbm_tbl[r][n0 + j] and the pair (host_tbl[r][n0 + j], id) is appended to the
 * plan's restore list; plan->counts->n_restore and *hbm_free_count are updated so that the following
 * cascade_kv_restore moves the prefetched blocks together with the admitted set's.  The caller folds
 * pf_out into next iteration's hit profile (n0 += pf, n1 -= pf).  With pools->hbm_tbl == NULL only
 * pf_out and the counts are produced.  0 <= link_budget_ns <= 2^50, hbm_reserve >= 0.
 */
int cascade_prefetch_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget, const uint32_t *order,
                          const int32_t *grant, const uint8_t *action, int n, int32_t D_act, int64_t K_act,
                          int64_t link_budget_ns, int32_t hbm_reserve, const cascade_pools *pools,
                          const cascade_plan *plan, int32_t *pf_out, cascade_prefetch_counts *counts_dev,
                          void *stream);

/*
 * Restore: for i < count, copy host record src_ids[i] into HBM block dst_ids[i]
 * (n_chunks pieces of chunk_bytes scattered into the paged layout).
 *   src_pool       record-major pool: pinned mapped host memory (read over the host link) or a
 *                  device staging buffer; src_is_device says which (tuning hint only)
 *   src_blocks     number of records in src_pool (ids outside are skipped, CASCADE_ST_EBOUNDS)
 *   n_copies_dev   device scalar holding the count, or NULL to use n_copies_max itself
 *   n_copies_max   upper bound of the count (list capacity)
 * Destination ids must be distinct within a call.
 * Errors: CASCADE_EINVAL (NULL pointer, negative count, chunk_bytes < 16, a size, stride or pool address that is
 * not a multiple of 16), CASCADE_ECUDA.  On the device: CASCADE_ST_EBOUNDS (that pair is skipped),
 * CASCADE_ST_ETIMEOUT (a bounded wait on a copy in flight expired: the CTA stops issuing work, waits, bounded
 * again, for the loads it already issued, and returns).
 */
int cascade_kv_restore(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, const void *src_pool,
                       int64_t src_blocks, int src_is_device, const int32_t *src_ids, const int32_t *dst_ids,
                       const int32_t *n_copies_dev, int n_copies_max, void *stream);

/* Evict: for i < count, copy HBM block src_ids[i] into host record dst_ids[i]; arguments as above. */
int cascade_kv_evict(cascade_ctx *ctx, const cascade_kv_layout *hbm, const void *hbm_pool, void *dst_pool,
                     int64_t dst_blocks, int dst_is_device, const int32_t *src_ids, const int32_t *dst_ids,
                     const int32_t *n_copies_dev, int n_copies_max, void *stream);

/*
 * Evict and restore in one call, with the host link used in both directions at once ("Budget-aware
 * preemption": a victim's KV is spilled and its freed HBM blocks are handed out again in the same iteration).
 * Same result as cascade_kv_evict on the evict list followed by cascade_kv_restore on the restore list (the
 * order the tier plan requires): a restore whose HBM block is also evicted by this call waits, block by
 * block, until that block has been read out.  Both lists as in the two calls above; the host pool must be
 * pinned, mapped host memory (or device memory).  Precondition: no restore reads a host record that an eviction
 * of the same call writes (the tier plan never produces that: evictions take records off the free list); such a
 * pair is not ordered here.  cascade_kv_move_staged orders it.
 *   scratch   caller-owned device array of cascade_kv_move_scratch_len(n_evict_max, n_restore_max) int32;
 *             contents irrelevant before the call.  After the call scratch[i], i < restore count, is the
 *             number of pieces of restore i that were NOT written: 0 = that block is complete, > 0 = a
 *             bounded wait ran out or an id was outside its pool (the matching status bit is set as well).
 * Residency rule: the evict side and the restore side are two grids of at most half the SMs each.  The
 * restore grid is a programmatic dependent of the evict grid, so the hardware starts it only when every
 * CTA of the evict grid is running or done; a waiting restore CTA therefore only ever waits for CTAs that
 * already hold an SM and that never wait themselves.  The call is safe beside other long-running kernels
 * (it only gets slower).  With programmatic launch off (CASCADE_PDL=0) the two grids run one after the other.
 * The per-block waits are clock-bounded all the same: on expiry CASCADE_ST_ETIMEOUT is set and that piece
 * is not written.
 */
int64_t cascade_kv_move_scratch_len(int n_evict_max, int n_restore_max);
int cascade_kv_move(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, void *host_pool,
                    int64_t host_blocks, const int32_t *evict_src, const int32_t *evict_dst,
                    const int32_t *n_evict_dev, int n_evict_max, const int32_t *restore_src,
                    const int32_t *restore_dst, const int32_t *n_restore_dev, int n_restore_max, int32_t *scratch,
                    void *stream);

/*
 * Evict and restore through the GPU's copy engines (the "asynchronous prefix prefetcher" driven from the host;
 * the rate this path reaches is the B^eff of Eq. 6 for large blocks).  Same result as cascade_kv_evict followed
 * by cascade_kv_restore; same list arguments as cascade_kv_move.  Unlike every other hot call this one
 * SYNCHRONISES THE HOST with `stream` once, because the copy engines are programmed by the host and the lists
 * live in device memory:
 *   1. a kernel publishes the two counts and the live list entries into `mailbox`, the host waits for it;
 *   2. evictions: the paged blocks are gathered into `staging` on `stream` (HBM to HBM), then one
 *      cudaMemcpyAsync per run of consecutive host records drains them to the host pool on a side stream;
 *   3. restores: one cudaMemcpyAsync per run of consecutive host records fills `staging` on a second side
 *      stream, then the staged blocks are scattered into the paged pool on `stream` (behind every gather);
 *   4. `stream` is made to wait for both side streams, so work issued on it afterwards sees the complete result.
 * The call returns when everything has been enqueued, not when it has run.  Both directions of the link are
 * busy at once; if a restore reads a host record that this call's evictions write, the fills wait for the drains.
 *   staging         caller-owned device buffer of staging_blocks * block bytes, 16-byte aligned, at least one
 *                   block per non-empty list (CASCADE_EINVAL otherwise, found after the host wait);
 *                   split between the two directions in proportion to the lists; with fewer blocks than
 *                   the lists hold the batches queue up for space (correct, slower)
 *   mailbox         caller-owned PINNED, mapped host array of cascade_kv_mailbox_len(n_evict_max, n_restore_max)
 *                   int32; after the call: [0] eviction count, [1] restore count, then the four lists
 * Faster than the zero-copy kernels for blocks of a megabyte and more (the copy engines move 55 - 57 GB/s per
 * direction and 96 - 100 GB/s both ways on a PCIe Gen5 x16 link), slower for small blocks (a few microseconds
 * of host and engine work per copy).  With a staging buffer that holds both lists the drains and the fills are
 * queued alternately, so both directions stay busy however long the lists are; with a smaller one the lists are
 * worked off one after the other in batches that wait for space (correct, slower).
 * Cannot be captured in a CUDA graph (host synchronisation).
 * Errors: as cascade_kv_move, plus CASCADE_ENOMEM (host bookkeeping could not grow).  Ids outside a pool:
 * that pair is skipped, CASCADE_ST_EBOUNDS.
 */
int64_t cascade_kv_mailbox_len(int n_evict_max, int n_restore_max);
int cascade_kv_move_staged(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, void *host_pool,
                           int64_t host_blocks, const int32_t *evict_src, const int32_t *evict_dst,
                           const int32_t *n_evict_dev, int n_evict_max, const int32_t *restore_src,
                           const int32_t *restore_dst, const int32_t *n_restore_dev, int n_restore_max, void *staging,
                           int64_t staging_blocks, int32_t *mailbox, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * Deep tier as a real stage, and one copy per shared block.
 *
 * Section "Memory management and HBM allocation": a deep-tier hit travels deep tier -> host DRAM -> HBM
 * (path P(2) of Eq. 6) and HBM is taken only at the last hop.  Here the first hop is a plan step of its
 * own (cascade_stage_plan) with a copy (cascade_kv_stage); the staged blocks become host blocks of the
 * request and the ordinary restore path of a later iteration is the last hop.  Section "Prefix hit
 * detection": several requests can match the same cached blocks; cascade_dedup makes a copy list carry
 * each such block once and counts the sharers.
 * ------------------------------------------------------------------------------------------------- */

/* written to device memory by cascade_stage_plan */
typedef struct cascade_stage_counts {
    int32_t n_stage;         /* entries of the stage list (blocks)                         */
    int32_t n_requests;      /* requests that staged at least one block                    */
    int32_t n_short;         /* requests that got fewer blocks than their choice asked for */
    int32_t host_free_after; /* host free-list length afterwards                           */
    int64_t link_ns_left;    /* deep-link time left                                        */
} cascade_stage_counts;

/* Inputs and outputs of cascade_stage_plan (host struct of device pointers). */
typedef struct cascade_stage {
    const int32_t *deep_tbl; /* [n][maxb]: deep_tbl[r][j] = deep-tier record of table position j, for
                                j in [n0+n1, n0+n1+n2); NULL = counts and `staged` only              */
    int32_t *stage_src;      /* deep-tier record ids, in schedule order                              */
    int32_t *stage_dst;      /* host record ids                                                      */
    int32_t stage_cap;
    int32_t *staged;         /* [n]: blocks staged per slot                                          */
    cascade_stage_counts *counts; /* device */
} cascade_stage;

/*
 * First hop of the two-hop path P(2).  Call it after cascade_tier_plan (it reads `action`; the host free
 * list must already reflect this iteration's evictions).  Walking `order`, every request that is valid,
 * holds deep blocks (n2 > 0), was not preempted by this iteration's plan and whose own restore choice
 * (the Eq. 7 bounds and the restore-vs-recompute comparison of cascade_tier_plan, from its budget alone)
 * contains a deep fetch of x2 > 0 blocks gets
 *     b = min(x2, blocks that still fit the deep link's time, host records free above host_reserve)
 * where one hop of x blocks costs what P(2) adds to P(1) in Eq. 6:
 *     max(0, delta_ns[2]-delta_ns[1]) + x * max(1, blk_ns[2]-blk_ns[1]),
 * and uses up that time and b host records.  For each such block a host record is popped from
 * pools->host_free, written to pools->host_tbl[r][n0+n1+j], and the pair (deep_tbl[r][n0+n1+j], record)
 * is appended to the stage list; *pools->host_free_count is updated.  No HBM block, table or list is
 * touched.  The caller folds `staged` into the next iteration's hit profile (n1 += staged, n2 -= staged).
 * Admission does not matter: with plan_first = 1 a request that chooses a deep fetch asks for no tokens
 * and stays queued while its blocks are staged.  0 <= link_budget_ns <= 2^50, host_reserve >= 0.
 * Only pools->host_tbl, maxb, host_free, host_free_count and host_free_cap are used.
 */
int cascade_stage_plan(cascade_ctx *ctx, const cascade_reqs *r, const int64_t *budget, const uint32_t *order,
                       const uint8_t *action, int n, int32_t D_act, int64_t K_act, int64_t link_budget_ns,
                       int32_t host_reserve, const cascade_pools *pools, const cascade_stage *stage, void *stream);

/*
 * Stage copy: for i < count, copy deep-tier record src_ids[i] into host record dst_ids[i].  Both pools are
 * record-major with records of block_bytes (a multiple of 16) and device-accessible: the deep pool is
 * pinned, mapped host memory standing in for the storage tier, or device memory.  Count arguments as in
 * cascade_kv_restore.  Ids outside a pool are skipped (CASCADE_ST_EBOUNDS).
 */
int cascade_kv_stage(cascade_ctx *ctx, const void *deep_pool, int64_t deep_blocks, void *host_pool,
                     int64_t host_blocks, int64_t block_bytes, const int32_t *src_ids, const int32_t *dst_ids,
                     const int32_t *n_copies_dev, int n_copies_max, void *stream);

/* written to device memory by cascade_dedup */
typedef struct cascade_dedup_counts {
    int32_t n_in;              /* list entries read                                        */
    int32_t n_unique;          /* entries of the output list                               */
    int32_t n_surplus;         /* destination ids handed back to the free list             */
    int32_t n_shared_requests; /* slots with at least one block shared with another entry  */
    int32_t max_share;         /* largest number of entries merged into one copy           */
    int32_t free_after;        /* free-list length afterwards                              */
} cascade_dedup_counts;

/* Arguments of cascade_dedup (host struct of device pointers). */
typedef struct cascade_dedup_args {
    const int32_t *lo_a, *lo_b;   /* [n] each, lo_b may be NULL: first table cell of slot r = lo_a[r] + lo_b[r] */
    const int32_t *len_a, *len_b; /* [n] each, len_b may be NULL: number of cells = len_a[r] + len_b[r]          */
    const int32_t *src_tbl;       /* [n][maxb] table holding the source ids of those cells                       */
    int32_t *dst_tbl;             /* [n][maxb] table holding their destination ids (rewritten)                   */
    int32_t maxb;
    const int32_t *list_src, *list_dst; /* the copy list                                                         */
    const int32_t *list_count;    /* device scalar: its length (a value above list_cap means list_cap)           */
    int32_t list_cap;
    int32_t *out_src, *out_dst;   /* the merged list, list_cap entries each; must not alias the input list       */
    int32_t n_src_ids, n_dst_ids; /* sizes of the source and destination pools (ids are 0 .. size-1)             */
    int32_t *free_list;           /* stack of free destination ids; surplus ids are pushed                       */
    int32_t *free_count;          /* device scalar, updated                                                      */
    int32_t free_cap;
    int32_t *ref;                 /* [n_dst_ids]: ref[d] = entries merged into kept destination d (written)      */
    uint8_t *shared;              /* [n]: 1 if a cell of the slot's range is shared with another entry           */
    int32_t *scratch;             /* caller-owned, scratch_len int32; contents irrelevant before and after       */
    int64_t scratch_len;          /* >= 2*n_src_ids + (list_cap + 1023)/1024 + 8                                 */
    cascade_dedup_counts *counts; /* device */
} cascade_dedup_args;

/*
 * One copy per distinct source block of a copy list: for shared prefixes that several requests restore
 * (list = the tier plan's restore list, source table = host_tbl, destination table = hbm_tbl, free list =
 * the HBM free list, cells [n0, n0 + x1 + prefetched)) or stage (list = the stage list, source table =
 * deep_tbl, destination table = host_tbl, free list = the host free list, cells [n0+n1, n0+n1+staged)) in
 * the same iteration.  Call it between the plan that wrote the list and the copy.
 *   - The first entry of every source id is kept; out_src/out_dst hold the kept entries in their
 *     original order and counts->n_unique their number (a device scalar usable as a copy count).
 *   - Every later entry of that source hands its destination id back: pushed on free_list in list order.
 *   - Every table cell in the slots' ranges whose source id has a kept entry is pointed at that entry's
 *     destination; ref[destination] = number of entries merged; shared[r] says whether slot r now shares
 *     a block (the caller then clears CASCADE_FLAG_HBM_PRIVATE for it: a shared block is never a victim).
 *   - An entry with an id outside its pool is passed through unchanged (CASCADE_ST_EBOUNDS); a slot whose
 *     range leaves its table row is skipped (CASCADE_ST_EPRECOND).
 * Source ids index a direct-address table in `scratch` (no sort): the cost is linear in the list length.
 */
int cascade_dedup(cascade_ctx *ctx, const cascade_dedup_args *a, int n, void *stream);

/*
 * One iteration in one call: what a serving loop issues between two engine iterations (Algorithm 1 as a
 * whole: re-budget every queued request, order, admit, plan, move).  Validates once and launches, in stream
 * order on `stream`,
 *     cascade_reqs_update   (if upd_m > 0)
 *     cascade_budget -> cascade_schedule -> cascade_tier_plan
 *     cascade_kv_move       (if layout != NULL; counts taken from plan->counts on the device)
 * with exactly the arguments of those calls; results and errors are theirs.  Nothing here synchronises the
 * host.  A caller that does not capture the iteration in a CUDA graph pays one crossing of its foreign-function
 * interface instead of four or five.  All members are host values; pointers are device pointers as in the
 * single calls.
 */
typedef struct cascade_step_args {
    const cascade_reqs *reqs;      /* the queue */
    int32_t n;                     /* queued requests */
    int32_t D_act;                 /* decode sequences in flight */
    int64_t K_act;                 /* their KV tokens */
    int64_t now_ns;
    const cascade_reqs *upd_src;   /* queue maintenance, see cascade_reqs_update; ignored when upd_m == 0 */
    const int32_t *upd_slots;
    int32_t upd_m;
    int32_t upd_cap;
    int64_t *budget;               /* outputs of cascade_budget */
    uint64_t *key;
    uint32_t *order;               /* outputs of cascade_schedule */
    int32_t *grant;
    cascade_sched_counts *sched_counts;
    const cascade_pools *pools;    /* cascade_tier_plan */
    const cascade_plan *plan;
    const cascade_kv_layout *layout; /* NULL: no copies */
    void *hbm_pool;
    void *host_pool;
    int64_t host_blocks;
    int32_t *move_scratch;         /* cascade_kv_move_scratch_len(plan->evict_cap, plan->restore_cap) int32 */
} cascade_step_args;
int cascade_step(cascade_ctx *ctx, const cascade_step_args *args, void *stream);

/* Waits for `stream`, copies the status word to *host_out and, if clear != 0, resets it. */
int cascade_status(cascade_ctx *ctx, cascade_status_t *host_out, int clear, void *stream);

/*
 * Tier plan without any allocation.  (The paper has no counterpart: this entry point exists for
 * the library's users, not for the method.)
 *
 * Same computation, same arguments and same results as cascade_tier_plan, but no context: the
 * per-request offsets that the first plan kernel hands to the two table-rewrite kernels live in a
 * fixed scratch area compiled into the library (about 320 KiB of device memory on every GPU that
 * loads the library, held from load to exit) instead of memory obtained in cascade_create.  It is
 * meant for callers that cannot call cudaMalloc: an engine that has already handed all free HBM to
 * its KV block pool, code running under a host framework that owns the allocator, or a loop that
 * cannot accept the device-wide synchronisation an allocation may cause.  The call itself makes no
 * cudaMalloc / cudaFree and calls no allocating library routine.
 *
 *   p            parameters (host), validated on every call as in cascade_create
 *   status_dev   caller-owned device word; CASCADE_ST_* bits are OR-ed into it (never cleared here)
 *   n            at most CASCADE_NOALLOC_MAX_REQUESTS, otherwise CASCADE_ETOOBIG is returned and
 *                nothing is launched
 *   all other arguments as in cascade_tier_plan; the device used is the calling thread's current one.
 *
 * The first call on each device looks up the device address of the scratch area (no allocation, but
 * a runtime query): make that first call outside any stream capture.  Every call on a GPU shares
 * the one scratch area and it keeps the previous call's contents; the entry point rewrites what it
 * reads, but two calls whose kernels can overlap on the GPU (different streams, or one process
 * with several host threads) race on it: issue them on one stream or order them with events.
 */
#define CASCADE_NOALLOC_MAX_REQUESTS 8192
int cascade_tier_plan_noalloc(const cascade_params *p, const cascade_reqs *r, const int64_t *budget,
                              const uint32_t *order, int32_t *grant, int n, int32_t D_act, int64_t K_act,
                              const cascade_pools *pools, const cascade_plan *plan_out, uint32_t *status_dev,
                              void *stream);

/* Library version (major*10000 + minor*100 + patch). */
int cascade_version(void);

#ifdef __cplusplus
}
#endif
#endif
