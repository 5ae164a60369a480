"""Pins for the comparison orderings (FCFS, EDF, SJF) and the estimator's four regimes."""
import numpy as np

import oracle
from paper_2608_06557_b200 import workload as wl

S = wl.S


def test_comparison_policies_order_by_their_own_criterion():
    w = wl.config_llama8b(3, n=600, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    r = w.reqs
    ids = r["id"].astype(np.int64)
    ttft = np.asarray(w.params["ttft_ns"], np.int64)[r["cls"]]
    want = r["prompt"].astype(np.int64) - (r["n0"].astype(np.int64) + r["n1"] + r["n2"]) * w.params["bt"]
    expect = {oracle.POLICY_FCFS: np.lexsort((ids, r["arrival_ns"])),
              oracle.POLICY_EDF: np.lexsort((ids, r["arrival_ns"] + ttft)),
              oracle.POLICY_SJF: np.lexsort((ids, want))}
    base_budget, base_key, _ = oracle.budget(oracle.make_params(w.params), r, w.now_ns, w.D_act, w.K_act)
    for pol, exp in expect.items():
        p = oracle.make_params(dict(w.params, policy=pol))
        b, k, st = oracle.budget(p, r, w.now_ns, w.D_act, w.K_act)
        assert st == 0
        assert np.array_equal(b, base_budget)                 # the budget itself does not depend on the ordering
        assert not np.any(k >> np.uint64(63))                 # one queue
        order, grant, counts, _ = oracle.schedule(p, r, k, w.D_act)
        assert np.array_equal(order, exp), pol
        assert counts["n_tier1"] == w.n
    # the method's own order differs from all three on this queue
    order0 = np.argsort(base_key, kind="stable")
    assert all(not np.array_equal(order0, e) for e in expect.values())


def test_regimes_against_the_worked_example_and_each_other():
    d = wl.default_params(gamma_q16=65536, ttft_ns=[1 * S], tpot_ns=[0])
    p = oracle.make_params(d)
    one = lambda P, n: dict(prompt=[P], n0=[n[0]], n1=[n[1]], n2=[n[2]])
    lat, st = oracle.latency_regimes(p, one(1000, (0, 0, 0)), 0, 0)
    assert st == 0
    # idle, no hits: regimes 0, 1, 2 coincide with the hand-worked 1000-token prefill, regime 3 with its max-load value
    assert lat[0].tolist() == [54_406_250, 54_406_250, 54_406_250, 67_046_718]
    # the loaded host-hit example: regime 2 = 70 780 393 ns, regime 3 = 77 226 434 ns
    lat, _ = oracle.latency_regimes(p, one(4100, (64, 128, 0)), 64, 131072)
    assert lat[0, 2] == 70_780_393 and lat[0, 3] == 77_226_434
    assert lat[0, 0] < lat[0, 1] and lat[0, 2] < lat[0, 1] and lat[0, 2] <= lat[0, 3]


def test_budget_is_eq3_to_eq5_over_regimes_two_and_three():
    w = wl.config_tiny(7)
    d = dict(w.params, tpot_ns=[0, 0])
    p = oracle.make_params(d)
    lat, _ = oracle.latency_regimes(p, w.reqs, w.D_act, w.K_act)
    b, _, _ = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
    L = ((lat[:, 2] + lat[:, 3]) * d["gamma_q16"]) >> 17
    ttft = np.asarray(d["ttft_ns"], np.int64)[w.reqs["cls"]]
    assert np.array_equal(b, ttft - L - (w.now_ns - w.reqs["arrival_ns"]))
