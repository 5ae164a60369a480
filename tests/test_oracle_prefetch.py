"""Pins for the budget-bounded prefetch of queued requests (Eq. 6, Eq. 7 applied ahead of admission)."""
import numpy as np

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl
from test_oracle_plan import py_cost_q20


def python_prefetch(w, res, link_budget, reserve, hbm_free_count):
    """The same policy restated in Python integers: one pass over the order, a running link-time and HBM
    allowance (an independent statement; the per-request bound is Eq. 7 solved by search, not by division)."""
    d, r = w.params, w.reqs
    plan = res["plan"]
    T = lambda x: 0 if x == 0 else d["delta_ns"][1] + x * d["blk_ns"][1]
    link = link_budget - sum(T(int(x)) for x, g in zip(plan["x1"], res["grant"]) if g > 0)
    avail = hbm_free_count - reserve
    pf = np.zeros(w.n, np.int64)
    for s in res["order"]:
        n0, n1 = int(r["n0"][s]), int(r["n1"][s])
        if res["grant"][s] > 0 or n1 == 0 or plan["action"][s] in (oracle.ACT_EVICT, oracle.ACT_DROP):
            continue
        rem = max(0, int(res["budget"][s]))
        m = 0
        while m < n1 and T(m + 1) <= rem:          # largest m with T(m) <= rem
            m += 1
        P = int(r["prompt"][s])
        if m and py_cost_q20(d, w.D_act, w.K_act, P, n0, m, 0) > py_cost_q20(d, w.D_act, w.K_act, P, n0, 0, 0):
            m = 0
        b = 0
        while b < m and b < avail and T(b + 1) <= link:
            b += 1
        if b:
            pf[s] = b
            link -= T(b)
            avail -= b
    return pf


def run(w, link_budget, reserve):
    res = oracle_iteration(w)
    plan, pools = res["plan"], res["pools"]
    p = oracle.make_params(w.params)
    hbm_before = pools.hbm_free_count
    tbl_before = pools.hbm_tbl.copy()
    out = oracle.prefetch_plan(p, w.reqs, res["budget"], res["order"], res["grant"], plan["action"], plan["x1"],
                               w.D_act, w.K_act, link_budget, reserve, pools, plan["restore_src"],
                               plan["restore_dst"])
    return res, out, hbm_before, tbl_before


def test_prefetch_matches_the_python_restatement_and_respects_every_bound():
    seen = 0
    for seed in range(10):
        w = wl.config_tiny(seed, hbm_free_target=32 + 60 * (seed % 3))
        w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]    # leave the queue some budget to spend
        for link_budget, reserve in ((0, 0), (15_000, 0), (400_000, 4), (10**9, 0), (10**9, 10)):
            res, out, hbm_before, tbl_before = run(w, link_budget, reserve)
            pf = out["pf"]
            assert np.array_equal(pf, python_prefetch(w, res, link_budget, reserve, hbm_before)), (seed, link_budget, reserve)
            plan, pools = res["plan"], res["pools"]
            r = w.reqs
            # only queued, un-preempted holders of host blocks; never more than they hold or than Eq. 7 allows
            got = pf > 0
            assert not np.any(got & (res["grant"] > 0))
            assert not np.any(got & np.isin(plan["action"], (oracle.ACT_EVICT, oracle.ACT_DROP)))
            assert np.all(pf <= r["n1"])
            p = oracle.make_params(w.params)
            for s in np.nonzero(got)[0]:
                assert oracle.restore_time(p, 1, int(pf[s])) <= max(0, res["budget"][s])
            # link time and HBM
            spent = sum(oracle.restore_time(p, 1, int(x)) for x in pf if x)
            assert spent <= max(0, out["counts"]["link_ns_left"])
            assert pools.hbm_free_count == hbm_before - pf.sum() >= min(reserve, hbm_before)
            # ids: popped from the top of the stack in order, written behind the HBM prefix, appended to the list
            assert out["counts"]["n_prefetch"] == pf.sum() == len(out["restore_src"]) - len(plan["restore_src"])
            k = len(plan["restore_src"])
            top = hbm_before
            for s in res["order"]:
                for j in range(int(pf[s])):
                    top -= 1
                    t = r["n0"][s] + j
                    assert out["restore_dst"][k] == pools.hbm_free[top] == pools.hbm_tbl[s, t]
                    assert out["restore_src"][k] == pools.host_tbl[s, t] >= 0 and tbl_before[s, t] == -1
                    k += 1
            seen += int(pf.sum() > 0)
    assert seen > 10


def test_prefetch_serves_the_tightest_budget_first_and_stops_at_the_link_budget():
    w = wl.config_tiny(5, hbm_free_target=400)
    w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    res_full, out_full, _, _ = run(w, 10**9, 0)
    want = out_full["pf"]
    assert want.sum() > 8
    # a link budget that covers about half of it: a prefix of the order is served, then one partial, then nothing
    p = oracle.make_params(w.params)
    half = sum(oracle.restore_time(p, 1, int(x)) for x in want if x) // 2
    res, out, _, _ = run(w, half + sum(oracle.restore_time(p, 1, int(x)) for x, g in
                                        zip(res_full["plan"]["x1"], res_full["grant"]) if g > 0), 0)
    pf = out["pf"]
    served = [int(pf[s]) for s in res["order"] if want[s] > 0]
    full = [int(want[s]) for s in res["order"] if want[s] > 0]
    i = 0
    while i < len(served) and served[i] == full[i]:
        i += 1
    assert 0 < i < len(served)
    assert all(v == 0 for v in served[i + 1:])


def test_preempted_requests_are_not_prefetched():
    """A request spilled by this iteration's plan keeps host blocks but must not get them back at once."""
    from test_oracle_plan import three_requests
    p = oracle.make_params(wl.default_params())
    reqs, budget, order, grant, pools = three_requests(hbm_free=1, host_free=20, victim_n0=10, victim_n1=5)
    plan = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert plan["action"][1] == oracle.ACT_EVICT and pools.hbm_free_count == 5
    r = dict(reqs, arrival_ns=[0, 0, 0], pred_out=[1, 1, 1], id=[0, 1, 2], cls=[0, 0, 0])
    out = oracle.prefetch_plan(p, r, budget, order, grant, plan["action"], plan["x1"], 0, 0, 10**9, 0, pools,
                               plan["restore_src"], plan["restore_dst"])
    assert out["pf"].tolist() == [0, 0, 3]          # only the queued request that was left alone
    assert out["counts"]["n_prefetch"] == 3 and pools.hbm_free_count == 2
