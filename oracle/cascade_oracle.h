/*
 * Cascade scheduling + KV-tier step: CPU oracle (TEST INFRASTRUCTURE, not product code).
 *
 * A plain, slow, single-threaded statement of what one iteration of the budget-driven
 * scheduling and KV-tier step computes.  It shares no code with the CUDA library and is
 * used only by the tests, the smoke check and the bench's CPU-baseline leg.
 *
 * Every time is an int64 number of nanoseconds, every token/block count an int32 and
 * every cost coefficient a Q20 fixed-point int64 (value * 2^20), so each input has
 * exactly one correct output.
 *
 * The struct layouts below are private to the oracle (they are mirrored by
 * oracle/__init__.py with ctypes); the CUDA library has its own header.
 */
#ifndef CASCADE_ORACLE_H
#define CASCADE_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_MAX_CLASSES 8

/* request flags */
#define ORC_FLAG_HBM_PRIVATE 1u /* the n0 HBM blocks belong to this request alone */
#define ORC_FLAG_RUNNING     2u /* informational */

/* per-request action written by the tier plan */
#define ORC_ACT_NONE   0u
#define ORC_ACT_RETAIN 1u
#define ORC_ACT_EVICT  2u
#define ORC_ACT_DROP   3u

/* status bits (OR-ed) */
#define ORC_ST_EBOUNDS  1u
#define ORC_ST_ENOSPC   2u
#define ORC_ST_EPRECOND 8u
#define ORC_ST_ELISTCAP 16u

typedef struct orc_params {
    int32_t bt;            /* tokens per KV block                                            */
    int32_t chunk_shift;   /* prefill chunk = 2^chunk_shift tokens                           */
    int32_t max_batch;     /* B_max: sequences per engine iteration, decodes included        */
    int32_t max_ctx_avg;   /* KV tokens assumed per decode sequence in the max-load regime   */
    int32_t gamma_q16;     /* guardband gamma * 2^16 (Eq. 3)                                 */
    int32_t n_classes;     /* <= ORC_MAX_CLASSES                                             */
    int32_t token_budget;  /* tokens per engine iteration                                    */
    int32_t tier2_reserve; /* tokens of each iteration kept for the Tier-2 queue             */
    int64_t c_tok_q20;     /* prefill cost per token, ns * 2^20                              */
    int64_t c_attn_q20;    /* prefill attention cost per token^2 (already halved), ns * 2^20 */
    int64_t c_iter_q20;    /* fixed cost of one engine iteration, ns * 2^20                  */
    int64_t c_dseq_q20;    /* cost per decode sequence in the iteration, ns * 2^20           */
    int64_t c_dkv_q20;     /* cost per decode KV token in the iteration, ns * 2^20           */
    int64_t delta_ns[3];   /* Eq. 6: sum of per-transfer overheads on path P(k); [0] unused  */
    int64_t blk_ns[3];     /* Eq. 6: time per block on path P(k); [0] unused                 */
    int64_t ttft_ns[ORC_MAX_CLASSES]; /* class TTFT targets                                  */
    int64_t tpot_ns[ORC_MAX_CLASSES]; /* class TPOT targets; 0 disables the decode term      */
    int32_t policy;        /* ordering: 0 least remaining budget, 1 FCFS, 2 EDF, 3 SJF (comparison policies) */
    int32_t plan_first;    /* 1: admission offers each request the tokens its own restore choice leaves to compute */
} orc_params;

#define ORC_POLICY_BUDGET 0
#define ORC_POLICY_FCFS 1
#define ORC_POLICY_EDF 2
#define ORC_POLICY_SJF 3

/* counts written by orc_schedule */
typedef struct orc_sched_counts {
    int32_t n_tier1;        /* requests whose key has the Tier-2 bit clear */
    int32_t n_admitted;     /* requests with grant > 0                     */
    int64_t tokens_granted; /* sum of grants                               */
} orc_sched_counts;

/* counts written by orc_tier_plan */
typedef struct orc_plan_counts {
    int32_t n_restore;      /* entries of the restore list (blocks)          */
    int32_t n_evict;        /* entries of the evict list (blocks)            */
    int32_t n_drop_blocks;  /* HBM blocks freed without a copy               */
    int32_t n_victims;      /* requests preempted (EVICT or DROP)            */
    int32_t n_unadmitted;   /* requests un-admitted by the HBM capacity scan */
    int32_t n_admitted;     /* requests still admitted after the plan        */
    int32_t hbm_need;       /* new HBM blocks the admitted set takes         */
    int32_t deficit;        /* blocks that had to be freed                   */
    int32_t hbm_free_after; /* HBM free-list length after the plan           */
    int32_t host_free_after;/* host free-list length after the plan          */
    int64_t tokens_run;     /* sum of tokens_run over admitted requests      */
} orc_plan_counts;

/* Steps B1-B6: per-request latency budget and 64-bit priority key (Eqs. 3-5).
 * Returns status bits (ORC_ST_EPRECOND when a request breaks an input bound). */
uint32_t orc_budget(const orc_params *p, int n,
                    const int64_t *arrival_ns, const int32_t *prompt, const int32_t *pred_out,
                    const int32_t *n0, const int32_t *n1, const int32_t *n2,
                    const uint32_t *id, const uint8_t *cls,
                    int64_t now_ns, int32_t D_act, int64_t K_act,
                    int64_t *budget_out, uint64_t *key_out);

/* Steps S1-S3: least-remaining-budget-first order and token-budget admission
 * (Algorithm 1, phase 2). */
uint32_t orc_schedule(const orc_params *p, int n,
                      const uint64_t *key, const int32_t *prompt,
                      const int32_t *n0, const int32_t *n1, const int32_t *n2,
                      int32_t D_act,
                      uint32_t *order_out, int32_t *grant_out, orc_sched_counts *counts,
                      const int64_t *budget /* plan_first only */, int64_t K_act /* plan_first only */);

/* Steps P1-P6 and K1: restore bound (Eq. 7), restore-vs-recompute choice, HBM
 * capacity, preemption victims and their disposition, block-id allocation.
 * hbm_tbl/host_tbl may be NULL together ("plan-only"): decisions and counts are
 * produced, no table, free list or copy list is touched. */
uint32_t orc_tier_plan(const orc_params *p, int n,
                       const int32_t *prompt, const int32_t *n0, const int32_t *n1, const int32_t *n2,
                       const uint8_t *flags,
                       const int64_t *budget, const uint32_t *order, int32_t *grant /* in/out */,
                       int32_t D_act, int64_t K_act,
                       int32_t *hbm_tbl, int32_t *host_tbl, int32_t maxb,
                       int32_t *hbm_free, int32_t *hbm_free_count, int32_t hbm_free_cap,
                       int32_t *host_free, int32_t *host_free_count, int32_t host_free_cap,
                       int32_t *x1_out, int32_t *x2_out, int32_t *tokens_run_out, uint8_t *action_out,
                       int32_t *restore_src, int32_t *restore_dst, int32_t restore_cap,
                       int32_t *evict_src, int32_t *evict_dst, int32_t evict_cap,
                       orc_plan_counts *counts);

/* counts written by orc_prefetch_plan */
typedef struct orc_prefetch_counts {
    int32_t n_prefetch;      /* blocks appended to the restore list                   */
    int32_t n_requests;      /* queued requests that got at least one block           */
    int32_t hbm_free_after;  /* HBM free-list length afterwards                       */
    int32_t n_restore_total; /* restore-list length afterwards (plan + prefetch)      */
    int64_t link_ns_left;    /* link time left after the admitted set's own restores  */
} orc_prefetch_counts;

/* Budget-bounded prefetch for queued requests (see the .cpp).  Tables NULL = plan-only. */
uint32_t orc_prefetch_plan(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                           const int32_t *n2, const int64_t *budget, const uint32_t *order, const int32_t *grant,
                           const uint8_t *action, const int32_t *x1, int32_t D_act, int64_t K_act,
                           int64_t link_budget_ns, int32_t hbm_reserve, int32_t *hbm_tbl, const int32_t *host_tbl,
                           int32_t maxb, int32_t *hbm_free, int32_t *hbm_free_count, int32_t hbm_free_cap,
                           int32_t *restore_src, int32_t *restore_dst, int32_t restore_cap, int32_t *n_restore,
                           int32_t *pf_out, orc_prefetch_counts *counts);

/* counts written by orc_stage_plan */
typedef struct orc_stage_counts {
    int32_t n_stage;         /* entries of the stage list (blocks)                          */
    int32_t n_requests;      /* requests that staged at least one block                     */
    int32_t n_short;         /* requests that got fewer blocks than their choice asked for  */
    int32_t host_free_after; /* host free-list length afterwards                            */
    int64_t link_ns_left;    /* deep-link time left                                         */
} orc_stage_counts;

/* First hop of the two-hop path P(2) (deep tier -> host DRAM -> HBM), see the .cpp.
 * Tables NULL = counts and staged_out only. */
uint32_t orc_stage_plan(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                        const int32_t *n2, const int64_t *budget, const uint32_t *order, const uint8_t *action,
                        int32_t D_act, int64_t K_act, int64_t link_budget_ns, int32_t host_reserve,
                        int32_t *host_tbl, const int32_t *deep_tbl, int32_t maxb, const int32_t *host_free,
                        int32_t *host_free_count, int32_t host_free_cap, int32_t *stage_src, int32_t *stage_dst,
                        int32_t stage_cap, int32_t *staged_out, orc_stage_counts *counts);

/* counts written by orc_dedup */
typedef struct orc_dedup_counts {
    int32_t n_in;              /* list entries read                                         */
    int32_t n_unique;          /* entries of the output list                                */
    int32_t n_surplus;         /* destination ids handed back to the free list              */
    int32_t n_shared_requests; /* slots with at least one block shared with another entry   */
    int32_t max_share;         /* largest number of entries merged into one copy            */
    int32_t free_after;        /* free-list length afterwards                               */
} orc_dedup_counts;

/* One copy per distinct source block.  The list (src[i], dst[i]) is read in order; the first entry
 * of every source id is kept (output list, same relative order), each later entry gives its
 * destination id back to the free list (pushed in list order) and every table cell in the ranges
 * [lo[r], lo[r] + len[r]) whose source id has a kept entry is pointed at that entry's destination.
 * ref[d] = number of entries merged into destination d, shared_out[r] = 1 if any cell of r's range
 * is merged with another entry.  Entries with an id outside its pool are kept untouched (EBOUNDS). */
uint32_t orc_dedup(int n, const int32_t *lo_a, const int32_t *lo_b, const int32_t *len_a, const int32_t *len_b,
                   const int32_t *src_tbl, int32_t *dst_tbl, int32_t maxb, const int32_t *list_src,
                   const int32_t *list_dst, int32_t list_count, int32_t list_cap, int32_t *out_src, int32_t *out_dst,
                   int32_t n_src_ids, int32_t n_dst_ids, int32_t *free_list, int32_t *free_count, int32_t free_cap,
                   int32_t *ref, uint8_t *shared_out, orc_dedup_counts *counts);

/* Record-major pool to record-major pool (deep tier -> host DRAM), one record per list entry. */
uint32_t orc_kv_stage(const uint8_t *deep_pool, int64_t deep_blocks, uint8_t *host_pool, int64_t host_blocks,
                      int64_t block_bytes, const int32_t *src_ids, const int32_t *dst_ids, int n_copies);

/* Step K2: paged copies.  HBM pool: chunk c of block b starts at
 * c*chunk_stride + b*block_stride.  Host pool: record h starts at h*n_chunks*chunk_bytes,
 * its chunks stored back to back.  Ids outside a pool are skipped and flagged. */
uint32_t orc_kv_restore(uint8_t *hbm_pool, int64_t hbm_blocks, int32_t n_chunks, int64_t chunk_bytes,
                        int64_t chunk_stride, int64_t block_stride,
                        const uint8_t *host_pool, int64_t host_blocks,
                        const int32_t *src_ids, const int32_t *dst_ids, int n_copies);
uint32_t orc_kv_evict(const uint8_t *hbm_pool, int64_t hbm_blocks, int32_t n_chunks, int64_t chunk_bytes,
                      int64_t chunk_stride, int64_t block_stride,
                      uint8_t *host_pool, int64_t host_blocks,
                      const int32_t *src_ids, const int32_t *dst_ids, int n_copies);

/* The estimator's four operating regimes for every request, lat4_out[4*r + i] in ns:
 * 0 zero load, full recomputation; 1 actual load, full recomputation; 2 actual load with tier-aware
 * prefix reuse; 3 maximum load with prefix reuse.  Regimes 2 and 3 are the L_actual and L_max of Eq. 3. */
uint32_t orc_latency_regimes(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                             const int32_t *n2, int32_t D_act, int64_t K_act, int64_t *lat4_out);

/* Pieces of the model exposed so the tests can pin them one by one. */
int64_t orc_restore_time(const orc_params *p, int k, int64_t x_blocks);            /* Eq. 6 */
int64_t orc_max_restorable(const orc_params *p, int k, int64_t rem_ns, int64_t nk); /* Eq. 7 */
int64_t orc_plan_cost_q20(const orc_params *p, int32_t D_act, int64_t K_act, int32_t prompt,
                          int32_t n0, int32_t x1, int32_t x2);                      /* F(x1,x2) */

#ifdef __cplusplus
}
#endif
#endif
