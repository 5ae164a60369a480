/*
 * Cascade scheduling + KV-tier step: CPU oracle (TEST INFRASTRUCTURE, not product code).
 *
 * Plain single-threaded C++17, sequential loops, std::stable_sort, memcpy.  No blocking,
 * fusion or reordering: each function takes the steps in the order the method states them
 * so that it can be checked against the paper by eye.  Only tests, the smoke check and the
 * bench's CPU-baseline leg may call this file; the CUDA library never does.
 *
 * What the paper fixes and what it leaves open:
 *   - Eq. 3 (effective latency), Eq. 4 (budget), Eq. 5 (remaining budget), Eq. 6 (restore
 *     time), Eq. 7 (max restorable volume) and Algorithm 1 (queue tiers, least-remaining-
 *     budget-first order, pop-while-capacity batch formation, largest-budget preemption)
 *     are followed literally.
 *   - The paper's latency estimator is an "offline-trained predictive model" with no printed
 *     form.  The integer polynomial used here (iter_q / A / comp_q below) is this build's
 *     reading; so are the token-granular admission scan, the Tier-2 reserve in tokens, the
 *     decode-overrun penalty and the three-candidate restore-vs-recompute choice.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py (hand-worked values,
 * closed forms, invariants, brute force on tiny inputs).  The paper's system-level results
 * (goodput, violation rate, fairness index) need its traces and simulator: parity unpinned.
 */
#include "cascade_oracle.h"

#include <algorithm>
#include <cstring>
#include <numeric>
#include <vector>

namespace {

constexpr int64_t kBudgetClamp = int64_t(1) << 39; /* key holds budget in [-2^39, 2^39) ns   */
constexpr uint32_t kIdMask = 0x7FFFFFu;            /* key holds the low 23 bits of the id     */
constexpr int64_t kInvalidBudget = -(int64_t(1) << 62);

struct Load {
    int64_t D; /* decode sequences sharing the iteration */
    int64_t K; /* their KV tokens                        */
};

/* Cost of one engine iteration that carries D decode sequences over K KV tokens (Q20 ns). */
int64_t iter_q(const orc_params *p, Load l) { return p->c_iter_q20 + l.D * p->c_dseq_q20 + l.K * p->c_dkv_q20; }

/* Cost per prefill token: its own linear cost plus its 1/chunk share of the iteration (Q20 ns). */
int64_t tok_q(const orc_params *p, Load l) { return p->c_tok_q20 + (iter_q(p, l) >> p->chunk_shift); }

/* Prefill compute for prompt tokens [s, P) when s tokens are already in the KV cache (Q20 ns). */
int64_t comp_q(const orc_params *p, int64_t A, int64_t P, int64_t s) {
    return A * (P - s) + p->c_attn_q20 * (P * P - s * s);
}

/* Eq. 6 in blocks: fixed overheads of the path plus per-block time; nothing to move costs nothing. */
int64_t restore_time(const orc_params *p, int k, int64_t x) {
    return x == 0 ? 0 : p->delta_ns[k] + x * p->blk_ns[k];
}

/* Eq. 7 in blocks: [rem - sum(delta)]^+ / per-block time, floored and capped at the nk blocks held. */
int64_t max_restorable(const orc_params *p, int k, int64_t rem, int64_t nk) {
    if (nk == 0) return 0;
    int64_t head = rem - p->delta_ns[k];
    if (head < 0) head = 0;
    return std::min<int64_t>(nk, head / p->blk_ns[k]);
}

/* The two load regimes of Eq. 3: actual load, and B_max - 1 concurrent decodes (never below actual). */
Load load_act(int32_t D_act, int64_t K_act) { return Load{D_act, K_act}; }
Load load_max(const orc_params *p, int32_t D_act, int64_t K_act) {
    int64_t Dm = std::max<int64_t>(D_act, p->max_batch - 1);
    int64_t Km = std::max<int64_t>(K_act, int64_t(p->max_batch - 1) * p->max_ctx_avg);
    return Load{Dm, Km};
}

/* Input bounds every step relies on (prompt <= 2^17, hits <= 2^13 blocks, at least one
 * prompt token left to compute). */
bool request_valid(const orc_params *p, int64_t P, int64_t n0, int64_t n1, int64_t n2) {
    if (P < 1 || P > (int64_t(1) << 17)) return false;
    if (n0 < 0 || n1 < 0 || n2 < 0) return false;
    if (n0 + n1 + n2 > (int64_t(1) << 13)) return false;
    return (n0 + n1 + n2) * p->bt < P;
}

int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* F(x1, x2): predicted completion time (Q20 ns, exact) when x1 host blocks and x2 deep blocks
 * are restored and the rest of the prompt is recomputed under the actual load. */
int64_t plan_cost_q20(const orc_params *p, Load act, int64_t P, int64_t n0, int64_t x1, int64_t x2) {
    int64_t transfer = restore_time(p, 1, x1) + restore_time(p, 2, x2);
    return (transfer << 20) + comp_q(p, tok_q(p, act), P, (n0 + x1 + x2) * p->bt);
}

/* P1 + P2: the Eq. 7 bounds (host first, deep tier from what is left and only behind a fully restored
 * host segment), then the endpoint candidate with the smallest predicted completion time; ties restore more. */
void choose_restore(const orc_params *p, Load act, int64_t P, int64_t n0, int64_t n1, int64_t n2, int64_t budget,
                    int64_t *x1, int64_t *x2) {
    const int64_t rem = std::max<int64_t>(0, budget);
    const int64_t x1max = max_restorable(p, 1, rem, n1);
    int64_t x2max = 0;
    if (x1max == n1 && n2 > 0) {
        const int64_t rem2 = rem - restore_time(p, 1, n1);
        x2max = max_restorable(p, 2, rem2, n2);
    }
    int64_t bx1 = 0, bx2 = 0;
    int64_t bF = plan_cost_q20(p, act, P, n0, 0, 0);
    if (x1max > 0) {
        const int64_t F = plan_cost_q20(p, act, P, n0, x1max, 0);
        if (F <= bF) { bF = F; bx1 = x1max; bx2 = 0; }
    }
    if (x2max > 0) {
        const int64_t F = plan_cost_q20(p, act, P, n0, n1, x2max);
        if (F <= bF) { bF = F; bx1 = n1; bx2 = x2max; }
    }
    *x1 = bx1;
    *x2 = bx2;
}

}  // namespace

extern "C" {

int64_t orc_restore_time(const orc_params *p, int k, int64_t x_blocks) { return restore_time(p, k, x_blocks); }

int64_t orc_max_restorable(const orc_params *p, int k, int64_t rem_ns, int64_t nk) {
    return max_restorable(p, k, rem_ns, nk);
}

int64_t orc_plan_cost_q20(const orc_params *p, int32_t D_act, int64_t K_act, int32_t prompt, int32_t n0, int32_t x1,
                          int32_t x2) {
    return plan_cost_q20(p, load_act(D_act, K_act), prompt, n0, x1, x2);
}

uint32_t orc_budget(const orc_params *p, int n, const int64_t *arrival_ns, const int32_t *prompt,
                    const int32_t *pred_out, const int32_t *n0, const int32_t *n1, const int32_t *n2,
                    const uint32_t *id, const uint8_t *cls, int64_t now_ns, int32_t D_act, int64_t K_act,
                    int64_t *budget_out, uint64_t *key_out) {
    uint32_t status = 0;
    const Load act = load_act(D_act, K_act);
    const Load mx = load_max(p, D_act, K_act);
    for (int r = 0; r < n; ++r) {
        const int64_t P = prompt[r];
        const int64_t O = pred_out[r];
        const int64_t elapsed = now_ns - arrival_ns[r];
        bool ok = request_valid(p, P, n0[r], n1[r], n2[r]);
        ok = ok && O >= 0 && O <= (int64_t(1) << 20);
        ok = ok && cls[r] < p->n_classes;
        ok = ok && elapsed <= (int64_t(1) << 50) && elapsed >= -(int64_t(1) << 50);
        if (!ok) {
            /* flagged; parked at the very end of the Tier-2 queue */
            status |= ORC_ST_EPRECOND;
            budget_out[r] = kInvalidBudget;
            key_out[r] = (uint64_t(1) << 63) | uint64_t(id[r] & kIdMask);
            continue;
        }
        /* B1: tokens of the prompt already cached in some tier */
        const int64_t s_hit = int64_t(n0[r] + n1[r] + n2[r]) * p->bt;
        /* B2: tier-priced transfer of the matched non-HBM prefix plus the compute of the rest,
         *     under the actual and under the maximum load */
        const int64_t tp = restore_time(p, 1, n1[r]) + restore_time(p, 2, n2[r]);
        const int64_t L_act = tp + (comp_q(p, tok_q(p, act), P, s_hit) >> 20);
        const int64_t L_max = tp + (comp_q(p, tok_q(p, mx), P, s_hit) >> 20);
        /* B3 (Eq. 3): L = (L_act + L_max)/2 * gamma, floored */
        const int64_t L = ((L_act + L_max) * p->gamma_q16) >> 17;
        /* B4 (Eq. 4, Eq. 5): budget against the class TTFT target; queue tier; remaining budget */
        const int64_t B = p->ttft_ns[cls[r]] - L;
        const int tier = (B > 0) ? 1 : 2;
        const int64_t B_rem = B - elapsed;
        /* B5: decode-overrun penalty from the predicted output length */
        const Load act1{act.D + 1, act.K + P};
        const Load mx1{mx.D + 1, mx.K + P};
        const int64_t chunk_q = p->c_tok_q20 << p->chunk_shift;
        const int64_t tdec_act = (iter_q(p, act1) + chunk_q) >> 20;
        const int64_t tdec_max = (iter_q(p, mx1) + chunk_q) >> 20;
        const int64_t tdec = ((tdec_act + tdec_max) * p->gamma_q16) >> 17;
        const int64_t tpot = p->tpot_ns[cls[r]];
        int64_t pen = 0;
        if (tpot != 0) pen = O * std::max<int64_t>(0, tdec - tpot);
        const int64_t budget = B_rem - pen;
        /* B6: 64-bit key = (tier-2 bit, clamped budget, arrival id).  The comparison policies keep the
         *     same packing with one queue: arrival time (FCFS), TTFT deadline (EDF), tokens left to
         *     prefill (SJF). */
        int64_t v = budget;
        bool tier2 = tier == 2;
        if (p->policy == ORC_POLICY_FCFS) { v = -elapsed; tier2 = false; }
        if (p->policy == ORC_POLICY_EDF) { v = p->ttft_ns[cls[r]] - elapsed; tier2 = false; }
        if (p->policy == ORC_POLICY_SJF) { v = P - s_hit; tier2 = false; }
        int64_t u = std::min(std::max(v, -kBudgetClamp), kBudgetClamp - 1) + kBudgetClamp;
        budget_out[r] = budget;
        key_out[r] = (uint64_t(tier2) << 63) | (uint64_t(u) << 23) | uint64_t(id[r] & kIdMask);
    }
    return status;
}

uint32_t orc_latency_regimes(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                             const int32_t *n2, int32_t D_act, int64_t K_act, int64_t *lat4_out) {
    uint32_t status = 0;
    const Load idle{0, 0};
    const Load act = load_act(D_act, K_act);
    const Load mx = load_max(p, D_act, K_act);
    for (int r = 0; r < n; ++r) {
        const int64_t P = prompt[r];
        if (!request_valid(p, P, n0[r], n1[r], n2[r])) {
            status |= ORC_ST_EPRECOND;
            for (int i = 0; i < 4; ++i) lat4_out[4 * r + i] = 0;
            continue;
        }
        const int64_t s_hit = int64_t(n0[r] + n1[r] + n2[r]) * p->bt;
        const int64_t tp = restore_time(p, 1, n1[r]) + restore_time(p, 2, n2[r]);
        lat4_out[4 * r + 0] = comp_q(p, tok_q(p, idle), P, 0) >> 20;          /* zero load, recompute all    */
        lat4_out[4 * r + 1] = comp_q(p, tok_q(p, act), P, 0) >> 20;           /* actual load, recompute all  */
        lat4_out[4 * r + 2] = tp + (comp_q(p, tok_q(p, act), P, s_hit) >> 20); /* actual load, tiered reuse   */
        lat4_out[4 * r + 3] = tp + (comp_q(p, tok_q(p, mx), P, s_hit) >> 20);  /* maximum load, tiered reuse  */
    }
    return status;
}

uint32_t orc_schedule(const orc_params *p, int n, const uint64_t *key, const int32_t *prompt, const int32_t *n0,
                      const int32_t *n1, const int32_t *n2, int32_t D_act, uint32_t *order_out, int32_t *grant_out,
                      orc_sched_counts *counts, const int64_t *budget, int64_t K_act) {
    /* S1: ascending by key; equal keys keep slot order */
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return key[a] < key[b]; });

    /* S2: tokens each request would compute if its whole matched prefix is reused */
    std::vector<int64_t> want(n);
    for (int r = 0; r < n; ++r) {
        if (!request_valid(p, prompt[r], n0[r], n1[r], n2[r])) {
            want[r] = 0;
        } else if (p->plan_first) {
            /* the request's own restore choice decides what is left to compute; a deep fetch is staged
             * first, so such a request asks for nothing this iteration */
            int64_t x1, x2;
            choose_restore(p, load_act(D_act, K_act), prompt[r], n0[r], n1[r], n2[r], budget[r], &x1, &x2);
            want[r] = x2 > 0 ? 0 : int64_t(prompt[r]) - (n0[r] + x1) * p->bt;
        } else {
            want[r] = int64_t(prompt[r]) - int64_t(n0[r] + n1[r] + n2[r]) * p->bt;
        }
    }
    /* every in-flight decode sequence takes one token of the iteration */
    const int64_t TB = std::max<int64_t>(0, int64_t(p->token_budget) - D_act);
    int n_t1 = 0;
    int64_t W2 = 0;
    for (int i = 0; i < n; ++i) {
        uint32_t r = order[i];
        if (key[r] >> 63)
            W2 += want[r];
        else
            ++n_t1;
    }
    const int64_t R2 = std::min<int64_t>(std::min<int64_t>(p->tier2_reserve, W2), TB);
    /* Tier-1 queue: pop in order, give each request what is left of the Tier-1 share */
    int64_t left = TB - R2;
    int64_t used1 = 0;
    for (int i = 0; i < n_t1; ++i) {
        uint32_t r = order[i];
        int64_t g = std::min(want[r], left);
        grant_out[r] = int32_t(g);
        left -= g;
        used1 += g;
    }
    /* Tier-2 queue: the reserve plus whatever Tier-1 left */
    left = TB - used1;
    for (int i = n_t1; i < n; ++i) {
        uint32_t r = order[i];
        int64_t g = std::min(want[r], left);
        grant_out[r] = int32_t(g);
        left -= g;
    }
    /* S3: at most max_batch sequences per iteration, decodes included */
    const int64_t seq_cap = std::max<int64_t>(0, int64_t(p->max_batch) - D_act);
    int64_t rank = 0;
    int32_t n_adm = 0;
    int64_t tokens = 0;
    for (int i = 0; i < n; ++i) {
        uint32_t r = order[i];
        if (grant_out[r] > 0) {
            if (rank >= seq_cap) grant_out[r] = 0;
            ++rank;
        }
        if (grant_out[r] > 0) {
            ++n_adm;
            tokens += grant_out[r];
        }
    }
    for (int i = 0; i < n; ++i) order_out[i] = order[i];
    counts->n_tier1 = n_t1;
    counts->n_admitted = n_adm;
    counts->tokens_granted = tokens;
    return 0;
}

uint32_t orc_tier_plan(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                       const int32_t *n2, const uint8_t *flags, const int64_t *budget, const uint32_t *order,
                       int32_t *grant, int32_t D_act, int64_t K_act, int32_t *hbm_tbl, int32_t *host_tbl,
                       int32_t maxb, int32_t *hbm_free, int32_t *hbm_free_count, int32_t hbm_free_cap,
                       int32_t *host_free, int32_t *host_free_count, int32_t host_free_cap, int32_t *x1_out,
                       int32_t *x2_out, int32_t *tokens_run_out, uint8_t *action_out, int32_t *restore_src,
                       int32_t *restore_dst, int32_t restore_cap, int32_t *evict_src, int32_t *evict_dst,
                       int32_t evict_cap, orc_plan_counts *counts) {
    uint32_t status = 0;
    const bool with_tables = hbm_tbl != nullptr;
    const Load act = load_act(D_act, K_act);

    int64_t hbm_cnt = *hbm_free_count;
    int64_t host_cnt = *host_free_count;
    if (with_tables) {
        if (hbm_cnt < 0 || hbm_cnt > hbm_free_cap) {
            status |= ORC_ST_EBOUNDS;
            hbm_cnt = std::min<int64_t>(std::max<int64_t>(hbm_cnt, 0), hbm_free_cap);
        }
        if (host_cnt < 0 || host_cnt > host_free_cap) {
            status |= ORC_ST_EBOUNDS;
            host_cnt = std::min<int64_t>(std::max<int64_t>(host_cnt, 0), host_free_cap);
        }
    }

    /* requests the plan may touch: inside the input bounds and, with tables, inside a table row */
    std::vector<uint8_t> valid(n);
    for (int r = 0; r < n; ++r) {
        bool ok = request_valid(p, prompt[r], n0[r], n1[r], n2[r]);
        if (ok && with_tables) ok = ceil_div(prompt[r], p->bt) <= maxb;
        valid[r] = ok;
        if (!ok) {
            status |= ORC_ST_EPRECOND;
            grant[r] = 0;
        }
    }

    /* P1 + P2 for every admitted request */
    std::vector<int32_t> need(n, 0);
    for (int r = 0; r < n; ++r) {
        x1_out[r] = 0;
        x2_out[r] = 0;
        tokens_run_out[r] = 0;
        action_out[r] = ORC_ACT_NONE;
        if (!valid[r] || grant[r] <= 0) continue;
        const int64_t P = prompt[r];
        int64_t bx1, bx2;
        choose_restore(p, act, P, n0[r], n1[r], n2[r], budget[r], &bx1, &bx2);
        x1_out[r] = int32_t(bx1);
        x2_out[r] = int32_t(bx2);
        /* a deep fetch is staged first: nothing runs this iteration, HBM is taken only at the last hop */
        const int64_t have = (n0[r] + bx1) * int64_t(p->bt);
        const int64_t run = (bx2 > 0) ? 0 : std::min<int64_t>(grant[r], P - have);
        tokens_run_out[r] = int32_t(run);
        need[r] = int32_t(bx1 + (ceil_div(have + run, p->bt) - (n0[r] + bx1)));
    }

    /* P3: HBM capacity.  Only blocks of non-admitted private holders can be freed. */
    int64_t evictable = 0;
    for (int r = 0; r < n; ++r)
        if (valid[r] && grant[r] <= 0 && (flags[r] & ORC_FLAG_HBM_PRIVATE)) evictable += n0[r];
    const int64_t cap = hbm_cnt + evictable;
    int64_t c = 0, need_total = 0;
    int32_t n_unadmitted = 0;
    for (int i = 0; i < n; ++i) {
        const uint32_t r = order[i];
        if (!valid[r] || grant[r] <= 0) continue;
        c += need[r];
        if (c > cap) {
            grant[r] = 0;
            x1_out[r] = x2_out[r] = tokens_run_out[r] = 0;
            need[r] = 0;
            ++n_unadmitted;
            status |= ORC_ST_ENOSPC;
        } else {
            need_total += need[r];
        }
    }
    const int64_t deficit = std::max<int64_t>(0, need_total - hbm_cnt);

    /* P4 + P5: victims, walking the order backwards (last to be served first) */
    std::vector<uint32_t> victims;
    {
        int64_t v = 0; /* blocks of eligible requests visited so far    */
        int64_t h = 0; /* blocks of victims that fit, visited so far     */
        for (int i = n - 1; i >= 0; --i) {
            const uint32_t r = order[i];
            const bool eligible = valid[r] && grant[r] <= 0 && (flags[r] & ORC_FLAG_HBM_PRIVATE) && n0[r] > 0;
            if (!eligible) continue;
            if (v < deficit) {
                /* spill only if it could be brought back within the victim's own budget, and host has room */
                const bool fits = restore_time(p, 1, n0[r]) <= budget[r];
                if (fits && h + n0[r] <= host_cnt)
                    action_out[r] = ORC_ACT_EVICT;
                else
                    action_out[r] = ORC_ACT_DROP;
                if (fits) h += n0[r];
                victims.push_back(r);
            }
            v += n0[r];
        }
    }
    for (int r = 0; r < n; ++r)
        if (valid[r] && action_out[r] == ORC_ACT_NONE && n0[r] > 0) action_out[r] = ORC_ACT_RETAIN;

    /* P6 / K1: block ids.  Free lists are stacks; all pushes precede all pops. */
    int32_t n_restore = 0, n_evict = 0, n_drop = 0;
    int64_t hbm_pos = hbm_cnt, host_pos = host_cnt;
    auto hbm_push = [&](int32_t v) {
        if (with_tables) {
            if (hbm_pos < hbm_free_cap) hbm_free[hbm_pos] = v; else status |= ORC_ST_EBOUNDS;
        }
        ++hbm_pos;
    };
    auto hbm_pop = [&]() -> int32_t {
        --hbm_pos;
        if (!with_tables) return -1;
        if (hbm_pos < hbm_free_cap) return hbm_free[hbm_pos];
        status |= ORC_ST_EBOUNDS;
        return -1;
    };
    for (uint32_t r : victims) {
        for (int j = 0; j < n0[r]; ++j) {
            const int32_t g = with_tables ? hbm_tbl[int64_t(r) * maxb + j] : -1;
            if (action_out[r] == ORC_ACT_EVICT) {
                --host_pos;
                if (with_tables) {
                    const int32_t hslot = host_free[host_pos];
                    if (n_evict < evict_cap) { evict_src[n_evict] = g; evict_dst[n_evict] = hslot; }
                    else status |= ORC_ST_ELISTCAP;
                    host_tbl[int64_t(r) * maxb + j] = hslot;
                }
                ++n_evict;
            } else {
                ++n_drop;
            }
            hbm_push(g);
            if (with_tables) hbm_tbl[int64_t(r) * maxb + j] = -1;
        }
    }
    int32_t n_admitted = 0;
    int64_t tokens_run = 0;
    for (int i = 0; i < n; ++i) {
        const uint32_t r = order[i];
        if (!valid[r] || grant[r] <= 0) continue;
        ++n_admitted;
        tokens_run += tokens_run_out[r];
        for (int j = n0[r]; j < n0[r] + need[r]; ++j) {
            const int32_t g = hbm_pop();
            if (j < n0[r] + x1_out[r]) {
                if (with_tables) {
                    if (n_restore < restore_cap) { restore_src[n_restore] = host_tbl[int64_t(r) * maxb + j]; restore_dst[n_restore] = g; }
                    else status |= ORC_ST_ELISTCAP;
                }
                ++n_restore;
            }
            if (with_tables) hbm_tbl[int64_t(r) * maxb + j] = g;
        }
    }
    if (with_tables) {
        *hbm_free_count = int32_t(hbm_pos);
        *host_free_count = int32_t(host_pos);
    }
    counts->n_restore = n_restore;
    counts->n_evict = n_evict;
    counts->n_drop_blocks = n_drop;
    counts->n_victims = int32_t(victims.size());
    counts->n_unadmitted = n_unadmitted;
    counts->n_admitted = n_admitted;
    counts->hbm_need = int32_t(need_total);
    counts->deficit = int32_t(deficit);
    counts->hbm_free_after = int32_t(hbm_pos);
    counts->host_free_after = int32_t(host_pos);
    counts->tokens_run = tokens_run;
    return status;
}

/* Budget-bounded prefetch for requests that stay queued (the prefix prefetcher acting ahead of
 * admission).  Walks the order; every valid request that was neither admitted nor preempted and
 * holds host blocks gets, while link time and free HBM last:
 *   m = its Eq. 7 bound for the host tier, if restoring m blocks beats recomputing them;
 *   b = min(m, blocks that still fit the link budget, free HBM blocks above the reserve).
 * Link time already spent this iteration: the sum of T_1(x1) over the admitted requests. */
uint32_t orc_prefetch_plan(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                           const int32_t *n2, const int64_t *budget, const uint32_t *order, const int32_t *grant,
                           const uint8_t *action, const int32_t *x1, int32_t D_act, int64_t K_act,
                           int64_t link_budget_ns, int32_t hbm_reserve, int32_t *hbm_tbl, const int32_t *host_tbl,
                           int32_t maxb, int32_t *hbm_free, int32_t *hbm_free_count, int32_t hbm_free_cap,
                           int32_t *restore_src, int32_t *restore_dst, int32_t restore_cap, int32_t *n_restore,
                           int32_t *pf_out, orc_prefetch_counts *counts) {
    uint32_t status = 0;
    const bool with_tables = hbm_tbl != nullptr;
    const Load act = load_act(D_act, K_act);
    int64_t hbm_pos = *hbm_free_count;
    if (with_tables && (hbm_pos < 0 || hbm_pos > hbm_free_cap)) {
        status |= ORC_ST_EBOUNDS;
        hbm_pos = std::min<int64_t>(std::max<int64_t>(hbm_pos, 0), hbm_free_cap);
    }
    int64_t link_left = link_budget_ns;
    for (int r = 0; r < n; ++r) {
        pf_out[r] = 0;
        bool ok = request_valid(p, prompt[r], n0[r], n1[r], n2[r]);
        if (ok && with_tables) ok = ceil_div(prompt[r], p->bt) <= maxb;
        if (ok && grant[r] > 0) link_left -= restore_time(p, 1, x1[r]);
    }
    int64_t avail = hbm_pos - hbm_reserve;
    int32_t n_pf = 0, n_req = 0, rest = *n_restore;
    const int64_t link_start = link_left;
    for (int i = 0; i < n; ++i) {
        const uint32_t r = order[i];
        bool ok = request_valid(p, prompt[r], n0[r], n1[r], n2[r]);
        if (ok && with_tables) ok = ceil_div(prompt[r], p->bt) <= maxb;
        if (!ok || grant[r] > 0 || n1[r] <= 0) continue;
        if (action[r] == ORC_ACT_EVICT || action[r] == ORC_ACT_DROP) continue;
        /* Eq. 7 bound, then restore-vs-recompute */
        const int64_t rem = std::max<int64_t>(0, budget[r]);
        int64_t m = max_restorable(p, 1, rem, n1[r]);
        if (m > 0 && plan_cost_q20(p, act, prompt[r], n0[r], m, 0) > plan_cost_q20(p, act, prompt[r], n0[r], 0, 0)) m = 0;
        if (m == 0) continue;
        /* what the link and HBM still allow */
        int64_t b = m;
        const int64_t by_link = link_left > p->delta_ns[1] ? (link_left - p->delta_ns[1]) / p->blk_ns[1] : 0;
        b = std::min(b, by_link);
        b = std::min(b, std::max<int64_t>(avail, 0));
        if (b <= 0) continue;
        link_left -= restore_time(p, 1, b);
        avail -= b;
        pf_out[r] = int32_t(b);
        n_pf += int32_t(b);
        ++n_req;
        for (int64_t j = 0; j < b; ++j) {
            --hbm_pos;
            if (!with_tables) continue;
            const int32_t g = hbm_pos < hbm_free_cap ? hbm_free[hbm_pos] : -1;
            const int64_t t = int64_t(r) * maxb + n0[r] + j;
            if (rest < restore_cap) { restore_src[rest] = host_tbl[t]; restore_dst[rest] = g; }
            else status |= ORC_ST_ELISTCAP;
            ++rest;
            hbm_tbl[t] = g;
        }
    }
    if (with_tables) {
        *hbm_free_count = int32_t(hbm_pos);
        *n_restore = rest;
    }
    counts->n_prefetch = n_pf;
    counts->n_requests = n_req;
    counts->hbm_free_after = int32_t(hbm_pos);
    counts->n_restore_total = with_tables ? rest : *n_restore + n_pf;
    counts->link_ns_left = link_start;
    return status;
}

/* First hop of P(2): deep tier -> host DRAM.  Walking the order, every valid request that this
 * iteration's plan did not preempt and whose own restore choice (Eq. 7 bounds, then the cheapest
 * candidate, from its budget) contains a deep fetch x2 > 0 gets host records for its first x2 deep
 * blocks while the deep link's time budget and the host pool (above a reserve) last.  One hop costs
 * what P(2) adds to P(1) in Eq. 6.  HBM is not touched (Section 4.4, memory management: HBM is taken
 * at the last hop only): the staged blocks become host blocks of the request and a later iteration
 * restores them. */
uint32_t orc_stage_plan(const orc_params *p, int n, const int32_t *prompt, const int32_t *n0, const int32_t *n1,
                        const int32_t *n2, const int64_t *budget, const uint32_t *order, const uint8_t *action,
                        int32_t D_act, int64_t K_act, int64_t link_budget_ns, int32_t host_reserve,
                        int32_t *host_tbl, const int32_t *deep_tbl, int32_t maxb, const int32_t *host_free,
                        int32_t *host_free_count, int32_t host_free_cap, int32_t *stage_src, int32_t *stage_dst,
                        int32_t stage_cap, int32_t *staged_out, orc_stage_counts *counts) {
    uint32_t status = 0;
    const bool with_tables = host_tbl != nullptr;
    const Load act = load_act(D_act, K_act);
    int64_t host_pos = *host_free_count;
    if (with_tables && (host_pos < 0 || host_pos > host_free_cap)) {
        status |= ORC_ST_EBOUNDS;
        host_pos = std::min<int64_t>(std::max<int64_t>(host_pos, 0), host_free_cap);
    }
    const int64_t hop_delta = std::max<int64_t>(0, p->delta_ns[2] - p->delta_ns[1]);
    const int64_t hop_blk = std::max<int64_t>(1, p->blk_ns[2] - p->blk_ns[1]);
    int64_t room = host_pos - host_reserve;
    int64_t link_left = link_budget_ns;
    int32_t n_stage = 0, n_req = 0, n_short = 0;
    for (int r = 0; r < n; ++r) staged_out[r] = 0;
    for (int i = 0; i < n; ++i) {
        const uint32_t r = order[i];
        bool ok = request_valid(p, prompt[r], n0[r], n1[r], n2[r]);
        if (ok && with_tables) ok = ceil_div(prompt[r], p->bt) <= maxb;
        if (!ok || n2[r] <= 0) continue;
        const bool preempted = action[r] == ORC_ACT_EVICT || action[r] == ORC_ACT_DROP;
        if (preempted) continue;
        int64_t bx1, bx2;
        choose_restore(p, act, prompt[r], n0[r], n1[r], n2[r], budget[r], &bx1, &bx2);
        if (bx2 <= 0) continue;
        const int64_t by_link = link_left > hop_delta ? (link_left - hop_delta) / hop_blk : 0;
        const int64_t b = std::min(bx2, std::min(by_link, std::max<int64_t>(room, 0)));
        if (b < bx2) ++n_short;
        if (b <= 0) continue;
        link_left -= hop_delta + b * hop_blk;
        room -= b;
        staged_out[r] = int32_t(b);
        ++n_req;
        for (int64_t j = 0; j < b; ++j) {
            --host_pos;
            if (with_tables) {
                const int64_t t = int64_t(r) * maxb + n0[r] + n1[r] + j;
                const int32_t rec = host_pos < host_free_cap ? host_free[host_pos] : -1;
                if (n_stage < stage_cap) { stage_src[n_stage] = deep_tbl[t]; stage_dst[n_stage] = rec; }
                else status |= ORC_ST_ELISTCAP;
                host_tbl[t] = rec;
            }
            ++n_stage;
        }
    }
    if (with_tables) *host_free_count = int32_t(host_pos);
    counts->n_stage = n_stage;
    counts->n_requests = n_req;
    counts->n_short = n_short;
    counts->host_free_after = int32_t(host_pos);
    counts->link_ns_left = link_left;
    return status;
}

/* One copy per distinct source block of a copy list (shared prefixes restored or staged by several
 * requests in one iteration). */
uint32_t orc_dedup(int n, const int32_t *lo_a, const int32_t *lo_b, const int32_t *len_a, const int32_t *len_b,
                   const int32_t *src_tbl, int32_t *dst_tbl, int32_t maxb, const int32_t *list_src,
                   const int32_t *list_dst, int32_t list_count, int32_t list_cap, int32_t *out_src, int32_t *out_dst,
                   int32_t n_src_ids, int32_t n_dst_ids, int32_t *free_list, int32_t *free_count, int32_t free_cap,
                   int32_t *ref, uint8_t *shared_out, orc_dedup_counts *counts) {
    uint32_t status = 0;
    int64_t m = list_count;
    if (m < 0 || m > list_cap) {
        if (m < 0) status |= ORC_ST_EBOUNDS;   /* a count above the capacity is a list the producer already cut */
        m = std::min<int64_t>(std::max<int64_t>(m, 0), list_cap);
    }
    int64_t fpos = *free_count;
    if (fpos < 0 || fpos > free_cap) {
        status |= ORC_ST_EBOUNDS;
        fpos = std::min<int64_t>(std::max<int64_t>(fpos, 0), free_cap);
    }
    /* kept[s] = destination of the first entry with source s; merged[s] = entries with source s */
    std::vector<int32_t> kept(size_t(std::max(n_src_ids, 0)), -1), merged(size_t(std::max(n_src_ids, 0)), 0);
    int32_t n_unique = 0, n_surplus = 0, max_share = 0;
    for (int64_t i = 0; i < m; ++i) {
        const int32_t s = list_src[i], d = list_dst[i];
        if (s < 0 || s >= n_src_ids || d < 0 || d >= n_dst_ids) {
            status |= ORC_ST_EBOUNDS;
            out_src[n_unique] = s;
            out_dst[n_unique] = d;
            ++n_unique;
            continue;
        }
        if (merged[s] == 0) {
            kept[s] = d;
            out_src[n_unique] = s;
            out_dst[n_unique] = d;
            ++n_unique;
        } else {
            if (fpos < free_cap) free_list[fpos] = d; else status |= ORC_ST_EBOUNDS;
            ++fpos;
            ++n_surplus;
        }
        ++merged[s];
    }
    for (int64_t i = 0; i < m; ++i) {
        const int32_t s = list_src[i];
        if (s < 0 || s >= n_src_ids || kept[s] < 0) continue;
        ref[kept[s]] = merged[s];
        max_share = std::max(max_share, merged[s]);
    }
    int32_t n_shared = 0;
    for (int r = 0; r < n; ++r) {
        const int64_t lo = int64_t(lo_a[r]) + (lo_b ? lo_b[r] : 0);
        const int64_t len = int64_t(len_a[r]) + (len_b ? len_b[r] : 0);
        uint8_t shared = 0;
        if (lo >= 0 && len > 0 && lo + len <= maxb) {
            for (int64_t j = lo; j < lo + len; ++j) {
                const int32_t s = src_tbl[int64_t(r) * maxb + j];
                if (s < 0 || s >= n_src_ids || merged[s] == 0) continue;
                dst_tbl[int64_t(r) * maxb + j] = kept[s];
                if (merged[s] > 1) shared = 1;
            }
        } else if (len > 0) {
            status |= ORC_ST_EPRECOND;
        }
        shared_out[r] = shared;
        n_shared += shared;
    }
    *free_count = int32_t(fpos);
    counts->n_in = int32_t(m);
    counts->n_unique = n_unique;
    counts->n_surplus = n_surplus;
    counts->n_shared_requests = n_shared;
    counts->max_share = max_share;
    counts->free_after = int32_t(fpos);
    return status;
}

uint32_t orc_kv_stage(const uint8_t *deep_pool, int64_t deep_blocks, uint8_t *host_pool, int64_t host_blocks,
                      int64_t block_bytes, const int32_t *src_ids, const int32_t *dst_ids, int n_copies) {
    uint32_t status = 0;
    for (int i = 0; i < n_copies; ++i) {
        const int64_t s = src_ids[i], d = dst_ids[i];
        if (s < 0 || s >= deep_blocks || d < 0 || d >= host_blocks) {
            status |= ORC_ST_EBOUNDS;
            continue;
        }
        std::memcpy(host_pool + d * block_bytes, deep_pool + s * block_bytes, size_t(block_bytes));
    }
    return status;
}

uint32_t orc_kv_restore(uint8_t *hbm_pool, int64_t hbm_blocks, int32_t n_chunks, int64_t chunk_bytes,
                        int64_t chunk_stride, int64_t block_stride, const uint8_t *host_pool, int64_t host_blocks,
                        const int32_t *src_ids, const int32_t *dst_ids, int n_copies) {
    uint32_t status = 0;
    const int64_t bb = int64_t(n_chunks) * chunk_bytes;
    for (int i = 0; i < n_copies; ++i) {
        const int64_t s = src_ids[i], d = dst_ids[i];
        if (s < 0 || s >= host_blocks || d < 0 || d >= hbm_blocks) {
            status |= ORC_ST_EBOUNDS;
            continue;
        }
        for (int c = 0; c < n_chunks; ++c)
            std::memcpy(hbm_pool + c * chunk_stride + d * block_stride, host_pool + s * bb + c * chunk_bytes,
                        size_t(chunk_bytes));
    }
    return status;
}

uint32_t orc_kv_evict(const uint8_t *hbm_pool, int64_t hbm_blocks, int32_t n_chunks, int64_t chunk_bytes,
                      int64_t chunk_stride, int64_t block_stride, uint8_t *host_pool, int64_t host_blocks,
                      const int32_t *src_ids, const int32_t *dst_ids, int n_copies) {
    uint32_t status = 0;
    const int64_t bb = int64_t(n_chunks) * chunk_bytes;
    for (int i = 0; i < n_copies; ++i) {
        const int64_t s = src_ids[i], d = dst_ids[i];
        if (s < 0 || s >= hbm_blocks || d < 0 || d >= host_blocks) {
            status |= ORC_ST_EBOUNDS;
            continue;
        }
        for (int c = 0; c < n_chunks; ++c)
            std::memcpy(host_pool + d * bb + c * chunk_bytes, hbm_pool + c * chunk_stride + s * block_stride,
                        size_t(chunk_bytes));
    }
    return status;
}

}  // extern "C"
