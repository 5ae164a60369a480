"""Pins for the oracle's tier plan: Eq. 6, Eq. 7, restore-vs-recompute, HBM capacity,
preemption victims (Algorithm 1) and block-id allocation."""
import json
import os

import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))
S = wl.S
PRIV = wl.FLAG_HBM_PRIVATE


def test_restore_time_is_affine_eq6():
    p = oracle.make_params(wl.default_params())
    assert oracle.restore_time(p, 1, 0) == 0 and oracle.restore_time(p, 2, 0) == 0
    assert oracle.restore_time(p, 1, 1) == 10_000 + 40_000
    assert oracle.restore_time(p, 1, 128) == 5_130_000          # the worked host-hit example
    assert oracle.restore_time(p, 2, 3) == 110_000 + 3 * 340_000
    for k in (1, 2):
        for x in (1, 5, 1000):
            assert oracle.restore_time(p, k, x + 1) - oracle.restore_time(p, k, x) == [0, 40_000, 340_000][k]


def test_max_restorable_inverts_restore_time_eq7():
    """Eq. 7 is Eq. 6 solved for the volume: T_k(M) <= rem < T_k(M+1) whenever 0 < M < n_k,
    M = 0 when the fixed overheads alone exceed the budget."""
    p = oracle.make_params(wl.default_params())
    rng = np.random.default_rng(2)
    for k, delta in ((1, 10_000), (2, 110_000)):
        assert oracle.max_restorable(p, k, delta, 50) == 0
        assert oracle.max_restorable(p, k, delta - 1, 50) == 0
        assert oracle.max_restorable(p, k, -5, 50) == 0
        assert oracle.max_restorable(p, k, 10**12, 0) == 0
        assert oracle.max_restorable(p, k, 10**12, 50) == 50
        for rem in rng.integers(0, 30_000_000, 500):
            nk = int(rng.integers(1, 100))
            M = oracle.max_restorable(p, k, int(rem), nk)
            assert 0 <= M <= nk
            if M > 0:
                assert oracle.restore_time(p, k, M) <= rem
            if M < nk:
                assert oracle.restore_time(p, k, M + 1) > rem


def py_cost_q20(d, D, K, P, n0, x1, x2):
    """Completion-time estimate in exact Python integers (Eq. 6 transfer + prefill of the rest)."""
    it = d["c_iter_q20"] + D * d["c_dseq_q20"] + K * d["c_dkv_q20"]
    A = d["c_tok_q20"] + (it >> d["chunk_shift"])
    T = lambda k, x: 0 if x == 0 else d["delta_ns"][k] + x * d["blk_ns"][k]
    s = (n0 + x1 + x2) * d["bt"]
    return ((T(1, x1) + T(2, x2)) << 20) + A * (P - s) + d["c_attn_q20"] * (P * P - s * s)


@pytest.mark.parametrize("ex", GOLD["plan"], ids=lambda e: e["name"])
def test_worked_plans(ex):
    base = next(b for b in GOLD["budget"] if b["name"] == ex["request"])
    d = wl.default_params(gamma_q16=base["gamma_q16"], ttft_ns=[base["ttft_ns"]], tpot_ns=[base["tpot_ns"]],
                          blk_ns=[0, ex["blk_ns_1"], 340_000])
    p = oracle.make_params(d)
    n0, n1, n2 = base["n"]
    D, K, P = base["D_act"], base["K_act"], base["prompt"]
    assert oracle.max_restorable(p, 1, ex["budget"], n1) == ex["x1max"]
    assert oracle.plan_cost_q20(p, D, K, P, n0, 0, 0) >> 20 == ex["F_recompute_ns"]
    assert oracle.plan_cost_q20(p, D, K, P, n0, ex["x1max"], 0) >> 20 == ex["F_restore_ns"]
    reqs = dict(prompt=[P], n0=[n0], n1=[n1], n2=[n2], flags=[0])
    grant = np.array([512], np.int32)
    pools = oracle.Pools(None, None, None, 1 << 30, None, 1 << 30)
    out = oracle.tier_plan(p, reqs, np.array([ex["budget"]], np.int64), np.array([0], np.uint32), grant, D, K, pools)
    assert (int(out["x1"][0]), int(out["x2"][0])) == (ex["x1"], ex["x2"])
    assert out["counts"]["n_restore"] == ex["x1"]


def test_choice_equals_brute_force_minimum():
    """The endpoint candidates must give the same (x1, x2) as minimising the completion time
    over every budget-feasible pair, ties going to the larger restore."""
    rng = np.random.default_rng(8)
    checked_partial = checked_deep = checked_none = 0
    for trial in range(1500):
        blk1 = int(rng.choice([500, 40_000, 400_000, 2_000_000]))
        blk2 = int(rng.choice([900, 340_000, 3_000_000]))
        d = wl.default_params(blk_ns=[0, blk1, blk2], delta_ns=[0, int(rng.integers(0, 200_000)),
                                                               int(rng.integers(0, 900_000))])
        p = oracle.make_params(d)
        n0, n1, n2 = (int(v) for v in rng.integers(0, 9, 3))
        P = (n0 + n1 + n2) * 16 + int(rng.integers(1, 40))
        D, K = int(rng.integers(0, 200)), int(rng.integers(0, 500_000))
        budget = int(rng.choice([-5, 0, int(rng.integers(0, 3_000_000)), int(rng.integers(0, 40_000_000))]))
        rem = max(0, budget)
        T = lambda k, x: 0 if x == 0 else d["delta_ns"][k] + x * d["blk_ns"][k]
        feas = []
        for x1 in range(n1 + 1):
            if T(1, x1) > rem:
                break
            feas.append((x1, 0))
            if x1 == n1:
                for x2 in range(1, n2 + 1):
                    if T(2, x2) > rem - T(1, n1):
                        break
                    feas.append((x1, x2))
        best = min(feas, key=lambda c: (py_cost_q20(d, D, K, P, n0, *c), -(c[0] + c[1])))
        reqs = dict(prompt=[P], n0=[n0], n1=[n1], n2=[n2], flags=[0])
        out = oracle.tier_plan(p, reqs, np.array([budget], np.int64), np.array([0], np.uint32),
                               np.array([P], np.int32), D, K, oracle.Pools(None, None, None, 1 << 30, None, 1 << 30))
        got = (int(out["x1"][0]), int(out["x2"][0]))
        assert got == best, (trial, got, best, feas)
        assert oracle.plan_cost_q20(p, D, K, P, n0, *got) == py_cost_q20(d, D, K, P, n0, *got)
        checked_partial += 0 < got[0] < n1
        checked_deep += got[1] > 0
        checked_none += got == (0, 0) and n1 > 0
    assert checked_partial > 20 and checked_deep > 20 and checked_none > 20


def test_tokens_run_and_need():
    d = wl.default_params()
    p = oracle.make_params(d)
    pools = lambda: oracle.Pools(None, None, None, 1 << 30, None, 1 << 30)
    # 3 HBM blocks cached, 2 host blocks restored, 100-token grant: runs tokens [80, 180) -> blocks 5..11 are new
    reqs = dict(prompt=[1000], n0=[3], n1=[2], n2=[0], flags=[0])
    out = oracle.tier_plan(p, reqs, np.array([10**9], np.int64), np.array([0], np.uint32),
                           np.array([100], np.int32), 0, 0, pools())
    assert (out["x1"][0], out["tokens_run"][0]) == (2, 100)
    assert out["counts"]["hbm_need"] == 2 + (12 - 5)
    # the grant is capped by what is left of the prompt
    reqs = dict(prompt=[90], n0=[3], n1=[2], n2=[0], flags=[0])
    out = oracle.tier_plan(p, reqs, np.array([10**9], np.int64), np.array([0], np.uint32),
                           np.array([100], np.int32), 0, 0, pools())
    assert out["tokens_run"][0] == 10 and out["counts"]["hbm_need"] == 2 + 1
    # a deep-tier fetch is staged: nothing runs, only the host part takes HBM now
    reqs = dict(prompt=[1000], n0=[1], n1=[2], n2=[30], flags=[0])
    out = oracle.tier_plan(p, reqs, np.array([10**11], np.int64), np.array([0], np.uint32),
                           np.array([100], np.int32), 0, 0, pools())
    assert (out["x1"][0], out["x2"][0], out["tokens_run"][0]) == (2, 30, 0)
    assert out["counts"]["hbm_need"] == 2


def literal_victims(order, grant, flags, n0, deficit):
    """Algorithm 1's preemption loop, literally: while HBM is short, take the eligible request that
    would be served last (largest remaining budget within its tier)."""
    victims, freed = [], 0
    taken = set()
    while freed < deficit:
        cand = [i for i in range(len(order)) if order[i] not in taken and grant[order[i]] <= 0
                and (flags[order[i]] & PRIV) and n0[order[i]] > 0]
        if not cand:
            break
        r = order[max(cand)]
        taken.add(r)
        victims.append(int(r))
        freed += int(n0[r])
    return victims


def check_iteration(w):
    res = oracle_iteration(w)
    plan, pools, grant = res["plan"], res["pools"], res["grant"]
    reqs, c = w.reqs, plan["counts"]
    n0, n1 = reqs["n0"], reqs["n1"]
    order = res["order"]
    adm = grant > 0
    # admitted after the plan is a subset of admitted by the scheduler, cut from the tail
    was = res["grant_sched"] > 0
    assert not np.any(adm & ~was)
    pos = np.empty(w.n, np.int64)
    pos[order] = np.arange(w.n)
    if np.any(was & ~adm):
        assert pos[was & ~adm].min() > pos[adm].max() if adm.any() else True
        assert res["status"] & oracle.ST_ENOSPC
    # per-request bounds
    assert np.all(plan["x1"] <= n1) and np.all(plan["x1"][~adm] == 0) and np.all(plan["tokens_run"][~adm] == 0)
    assert np.all(plan["tokens_run"] <= grant)
    # victims: never admitted, never shared; exactly the literal loop of Algorithm 1
    vict = np.isin(plan["action"], (oracle.ACT_EVICT, oracle.ACT_DROP))
    assert not np.any(vict & adm)
    assert np.all(reqs["flags"][vict] & PRIV)
    lit = literal_victims(order, grant, reqs["flags"], n0, c["deficit"])
    assert sorted(lit) == sorted(np.nonzero(vict)[0].tolist())
    freed = int(n0[vict].sum())
    assert freed >= c["deficit"]
    assert c["n_evict"] + c["n_drop_blocks"] == freed
    assert np.all(plan["action"][(~vict) & (n0 > 0)] == oracle.ACT_RETAIN)
    assert np.all(plan["action"][(~vict) & (n0 == 0)] == oracle.ACT_NONE)
    # spill only within the victim's own budget and the host pool's room
    p = oracle.make_params(w.params)
    for r in np.nonzero(plan["action"] == oracle.ACT_EVICT)[0]:
        assert oracle.restore_time(p, 1, int(n0[r])) <= res["budget"][r]
    assert c["n_evict"] <= w.host_free_count
    # ids: conservation and uniqueness
    assert c["hbm_free_after"] == w.hbm_free_count + freed - c["hbm_need"] >= 0
    assert c["host_free_after"] == w.host_free_count - c["n_evict"]
    assert c["n_restore"] == int(plan["x1"].sum())
    held = pools.hbm_tbl[pools.hbm_tbl >= 0]
    free = pools.hbm_free[: pools.hbm_free_count]
    before = np.concatenate([w.hbm_tbl[w.hbm_tbl >= 0], w.hbm_free[: w.hbm_free_count]])
    assert len(np.unique(before)) == len(before)
    both = np.concatenate([held, free])
    assert len(np.unique(both)) == len(both)
    assert set(both.tolist()) == set(before.tolist())
    hheld = pools.host_tbl[pools.host_tbl >= 0]
    hfree = pools.host_free[: pools.host_free_count]
    hboth = np.concatenate([hheld, hfree])
    assert len(np.unique(hboth)) == len(hboth)
    assert len(np.unique(plan["restore_dst"])) == len(plan["restore_dst"])
    assert len(np.unique(plan["evict_dst"])) == len(plan["evict_dst"])
    # every restored block is now in its request's table at the right position, source = its host block
    k = 0
    for r in order:
        for j in range(n0[r], n0[r] + plan["x1"][r]):
            assert plan["restore_src"][k] == w.host_tbl[r, j] == pools.host_tbl[r, j]
            assert plan["restore_dst"][k] == pools.hbm_tbl[r, j]
            k += 1
    assert k == c["n_restore"]
    # evicted victims: table moved to host ids, HBM row cleared
    for r in np.nonzero(vict)[0]:
        assert np.all(pools.hbm_tbl[r, : n0[r]] == -1)
        if plan["action"][r] == oracle.ACT_EVICT:
            assert np.all(pools.host_tbl[r, : n0[r]] >= 0)
    return res


def test_tiny_iteration_invariants_and_pressure():
    seen_evict = seen_drop = seen_nospc = 0
    for seed in range(12):
        w = wl.config_tiny(seed)
        res = check_iteration(w)
        c = res["plan"]["counts"]
        seen_evict += c["n_evict"] > 0
        seen_drop += c["n_drop_blocks"] > 0
        seen_nospc += c["n_unadmitted"] > 0
    assert seen_evict and seen_drop


def test_capacity_shrinks_admitted_set_from_the_tail():
    w = wl.config_tiny(0)
    w.hbm_free_count = 3
    w.reqs["flags"][:] = 0          # nothing evictable
    res = check_iteration(w)
    assert res["plan"]["counts"]["n_unadmitted"] > 0
    assert res["status"] & oracle.ST_ENOSPC
    assert res["plan"]["counts"]["hbm_need"] <= 3


def test_host_pool_full_forces_drop():
    w = wl.config_tiny(0)
    w.host_free_count = 0
    res = check_iteration(w)
    assert res["plan"]["counts"]["n_evict"] == 0
    assert res["plan"]["counts"]["n_victims"] > 0 and res["plan"]["counts"]["n_drop_blocks"] > 0


def test_plan_only_mode_matches_decisions_with_tables():
    w = wl.config_tiny(5)
    a = oracle_iteration(w, with_tables=True)
    b = oracle_iteration(w, with_tables=False)
    for k in ("x1", "x2", "tokens_run", "action"):
        assert np.array_equal(a["plan"][k], b["plan"][k])
    assert a["plan"]["counts"] == b["plan"]["counts"]


def test_transfer_beyond_budget_falls_back_to_recompute():
    """A hit whose transfer cannot fit the remaining budget is recomputed (Eq. 7 gives M = 0)."""
    p = oracle.make_params(wl.default_params())
    reqs = dict(prompt=[4100], n0=[64], n1=[128], n2=[0], flags=[0])
    out = oracle.tier_plan(p, reqs, np.array([30_000], np.int64), np.array([0], np.uint32),
                           np.array([512], np.int32), 0, 0, oracle.Pools(None, None, None, 1 << 30, None, 1 << 30))
    assert out["x1"][0] == 0 and out["tokens_run"][0] == 512


def _plan_only():
    return oracle.Pools(None, None, None, 1 << 30, None, 1 << 30)


def test_equal_cost_restores():
    """Transfer time exactly equal to the compute it saves: the tie goes to the restore."""
    d = wl.default_params(c_attn_q20=0, c_dseq_q20=0, c_dkv_q20=0, c_tok_q20=30_000 * wl.Q20,
                          c_iter_q20=512 * 1000 * wl.Q20, delta_ns=[0, 0, 0], blk_ns=[0, 16 * 31_000, 10**6])
    p = oracle.make_params(d)
    reqs = dict(prompt=[1000], n0=[2], n1=[7], n2=[0], flags=[0])
    assert oracle.plan_cost_q20(p, 0, 0, 1000, 2, 7, 0) == oracle.plan_cost_q20(p, 0, 0, 1000, 2, 0, 0)
    out = oracle.tier_plan(p, reqs, np.array([10**9], np.int64), np.array([0], np.uint32), np.array([64], np.int32),
                           0, 0, _plan_only())
    assert out["x1"][0] == 7
    d["blk_ns"][1] += 1                        # one nanosecond dearer per block: recompute
    out = oracle.tier_plan(oracle.make_params(d), reqs, np.array([10**9], np.int64), np.array([0], np.uint32),
                           np.array([64], np.int32), 0, 0, _plan_only())
    assert out["x1"][0] == 0


def three_requests(hbm_free, host_free, victim_n0=10, victim_n1=0, victim_budget=10**9):
    """Slot 0 is admitted and needs 2 restored + 4 new blocks; slot 1 holds `victim_n0` private HBM blocks
    and sits at the end of the order; slot 2 is queued without HBM blocks."""
    maxb = 32
    reqs = dict(prompt=[160, 400, 100], n0=[0, victim_n0, 0], n1=[2, victim_n1, 3], n2=[0, 0, 0],
                flags=[0, PRIV, 0])
    hbm_tbl = np.full((3, maxb), -1, np.int32)
    host_tbl = np.full((3, maxb), -1, np.int32)
    hbm_tbl[1, :victim_n0] = 100 + np.arange(victim_n0)
    host_tbl[0, :2] = [50, 51]
    host_tbl[1, victim_n0:victim_n0 + victim_n1] = 60 + np.arange(victim_n1)
    host_tbl[2, :3] = [70, 71, 72]
    hf = np.full(256, -1, np.int32)
    hf[:hbm_free] = 200 + np.arange(hbm_free)
    of = np.full(256, -1, np.int32)
    of[:host_free] = 300 + np.arange(host_free)
    pools = oracle.Pools(hbm_tbl, host_tbl, hf, hbm_free, of, host_free, 256, 256)
    budget = np.array([10**9, victim_budget, 5 * 10**8], np.int64)
    order = np.array([0, 2, 1], np.uint32)
    grant = np.array([64, 0, 0], np.int32)
    return reqs, budget, order, grant, pools


def test_capacity_and_host_room_exactly_met():
    p = oracle.make_params(wl.default_params())
    # need = 2 restored + 4 computed = 6; free 1 + preemptable 5 = 6: still admitted, the victim is taken
    reqs, budget, order, grant, pools = three_requests(hbm_free=1, host_free=5, victim_n0=5)
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert out["counts"]["n_unadmitted"] == 0 and out["counts"]["hbm_need"] == 6 and grant[0] == 64
    # the victim's 5 blocks fit the 5 free host records exactly: spilled, not dropped
    assert out["action"][1] == oracle.ACT_EVICT and out["counts"]["n_evict"] == 5
    # spilled blocks: sources are the victim's HBM ids in table order, destinations come off the top of the host stack
    assert out["evict_src"].tolist() == [100, 101, 102, 103, 104]
    assert out["evict_dst"].tolist() == [304, 303, 302, 301, 300]
    assert pools.host_tbl[1, :5].tolist() == [304, 303, 302, 301, 300] and np.all(pools.hbm_tbl[1, :5] == -1)
    # freed ids are pushed, then popped from the top for the restored and the computed blocks
    assert out["restore_src"].tolist() == [50, 51] and out["restore_dst"].tolist() == [104, 103]
    assert pools.hbm_tbl[0, :6].tolist() == [104, 103, 102, 101, 100, 200]
    assert pools.hbm_free_count == 0 and pools.host_free_count == 0
    # one block less of room on either side flips the decisions
    reqs, budget, order, grant, pools = three_requests(hbm_free=0, host_free=5, victim_n0=5)
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert out["counts"]["n_unadmitted"] == 1 and grant[0] == 0
    reqs, budget, order, grant, pools = three_requests(hbm_free=1, host_free=4, victim_n0=5)
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert out["action"][1] == oracle.ACT_DROP and out["counts"]["n_evict"] == 0


def test_iteration_invariants_with_restores():
    """Looser class targets leave the admitted set budget to restore with: the restore list is exercised."""
    restored = 0
    for seed in range(6):
        w = wl.config_tiny(seed, hbm_free_target=120)
        w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
        restored += check_iteration(w)["plan"]["counts"]["n_restore"]
    assert restored > 20
