"""Pins for the oracle's ordering and admission step (Algorithm 1, phase 2)."""
import json
import os

import numpy as np

import oracle
from paper_2608_06557_b200 import workload as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))


def reqs_with_want(want):
    n = len(want)
    z = np.zeros(n, np.int32)
    return dict(prompt=np.asarray(want, np.int32), n0=z, n1=z.copy(), n2=z.copy())


def test_worked_admission():
    g = GOLD["schedule"]
    p = oracle.make_params(wl.default_params(token_budget=g["token_budget"], tier2_reserve=g["tier2_reserve"],
                                             max_batch=g["max_batch"]))
    key = np.array([int(r["key"], 16) for r in g["requests"]], np.uint64)
    order, grant, counts, st = oracle.schedule(p, reqs_with_want([r["want"] for r in g["requests"]]), key,
                                               g["D_act"])
    assert [g["requests"][i]["id"] for i in order] == g["order_ids"]
    assert grant.tolist() == [r["grant"] for r in g["requests"]]
    assert counts["tokens_granted"] == g["tokens_granted"]
    assert counts["n_tier1"] == 5 and counts["n_admitted"] == 4


def scan_form(key, want, TB, reserve, seq_cap):
    """The same admission written as clamped prefix sums (numpy), the data-parallel statement."""
    order = np.argsort(key, kind="stable")
    w = want[order].astype(np.int64)
    t2 = (key[order] >> np.uint64(63)).astype(bool)
    n1 = int((~t2).sum())
    W1, W2 = int(w[:n1].sum()), int(w[n1:].sum())
    R2 = min(reserve, W2, TB)
    e = np.cumsum(w) - w
    g = np.zeros(len(w), np.int64)
    g[:n1] = np.clip((TB - R2) - e[:n1], 0, w[:n1])
    U1 = int(g[:n1].sum())
    g[n1:] = np.clip((TB - U1) - (e[n1:] - W1), 0, w[n1:])
    rank = np.cumsum(g > 0) - (g > 0)
    g[rank >= seq_cap] = 0
    out = np.zeros(len(w), np.int64)
    out[order] = g
    return order, out


def test_sequential_pops_equal_clamped_scans():
    rng = np.random.default_rng(11)
    for trial in range(200):
        n = int(rng.integers(1, 40))
        want = rng.integers(1, 600, n).astype(np.int32)
        tier2 = rng.integers(0, 2, n).astype(np.uint64)
        if trial % 7 == 0:
            tier2[:] = trial % 2
        key = (tier2 << np.uint64(63)) | (rng.integers(0, 50, n).astype(np.uint64) << np.uint64(23)) \
            | np.arange(n, dtype=np.uint64)
        tb, res, mb, D = int(rng.integers(0, 3000)), int(rng.integers(0, 500)), int(rng.integers(1, 12)), \
            int(rng.integers(0, 6))
        p = oracle.make_params(wl.default_params(token_budget=tb, tier2_reserve=res, max_batch=mb))
        order, grant, counts, st = oracle.schedule(p, reqs_with_want(want), key, D)
        TB = max(0, tb - D)
        o2, g2 = scan_form(key, want, TB, res, max(0, mb - D))
        assert np.array_equal(order, o2)
        assert np.array_equal(grant, g2)
        # invariants: token budget, batch size, order, prefix admission with at most one partial grant per tier
        assert grant.sum() <= TB and counts["tokens_granted"] == grant.sum()
        assert counts["n_admitted"] == (grant > 0).sum() <= max(0, mb - D)
        assert np.all(np.diff(key[order].astype(object)) > 0)
        for seg in (order[: counts["n_tier1"]], order[counts["n_tier1"]:]):
            adm = grant[seg] > 0
            assert not np.any(adm[1:] & ~adm[:-1])          # admitted requests form a prefix of the tier
            assert (adm & (grant[seg] < want[seg])).sum() <= 1


def test_reserve_only_reaches_tier2_when_it_wants_it():
    p = oracle.make_params(wl.default_params(token_budget=1000, tier2_reserve=300, max_batch=64))
    # no Tier-2 request: Tier-1 may use the whole budget
    key = np.arange(3, dtype=np.uint64)
    _, grant, _, _ = oracle.schedule(p, reqs_with_want([600, 600, 600]), key, 0)
    assert grant.tolist() == [600, 400, 0]
    # one small Tier-2 request: it gets what it wants out of the reserve, the rest returns to Tier-1
    key = np.array([0, 1, (1 << 63) | 2], np.uint64)
    _, grant, _, _ = oracle.schedule(p, reqs_with_want([600, 600, 100]), key, 0)
    assert grant.tolist() == [600, 300, 100]
    # decode sequences take one token each off the budget first
    _, grant, _, _ = oracle.schedule(p, reqs_with_want([600, 600, 100]), key, 40)
    assert grant.tolist() == [600, 260, 100]


def test_order_is_stable_for_equal_keys_and_matches_library_sort():
    w = wl.config_llama8b(9, n=700, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    p = oracle.make_params(w.params)
    b, k, _ = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
    k[100:110] = k[5]   # duplicated keys keep slot order
    order, grant, counts, _ = oracle.schedule(p, w.reqs, k, w.D_act)
    assert np.array_equal(order, np.argsort(k, kind="stable"))
    assert sorted(order.tolist()) == list(range(w.n))
