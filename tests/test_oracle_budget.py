"""Pins for the oracle's budget step (Eq. 3, Eq. 4, Eq. 5 and the priority key)."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2608_06557_b200 import workload as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))
S, MS = wl.S, wl.MS


def one_request(prompt, pred_out, n, elapsed, now=10 * S, cls=0, rid=0, flags=0):
    return dict(arrival_ns=np.array([now - elapsed], np.int64), prompt=np.array([prompt], np.int32),
                pred_out=np.array([pred_out], np.int32), n0=np.array([n[0]], np.int32),
                n1=np.array([n[1]], np.int32), n2=np.array([n[2]], np.int32), id=np.array([rid], np.uint32),
                cls=np.array([cls], np.uint8), flags=np.array([flags], np.uint8))


def pack_key(tier, budget, rid):
    """(Tier-2 bit, budget clamped to 40 bits and biased, low 23 id bits); checked against the
    stored hexadecimal keys in test_key_packing_matches_stored_keys."""
    u = min(max(budget, -(1 << 39)), (1 << 39) - 1) + (1 << 39)
    return ((1 if tier == 2 else 0) << 63) | (u << 23) | (rid & 0x7FFFFF)


def test_key_packing_matches_stored_keys():
    for r in GOLD["schedule"]["requests"]:
        assert pack_key(r["tier"], r["budget"], r["id"]) == int(r["key"], 16)


@pytest.mark.parametrize("ex", GOLD["budget"], ids=lambda e: e["name"])
def test_worked_budgets(ex):
    p = oracle.make_params(wl.default_params(gamma_q16=ex["gamma_q16"], ttft_ns=[ex["ttft_ns"]],
                                             tpot_ns=[ex["tpot_ns"]]))
    now = 10 * S
    req = one_request(ex["prompt"], ex["pred_out"], ex["n"], ex["elapsed_ns"], now=now, rid=7)
    b, k, st = oracle.budget(p, req, now, ex["D_act"], ex["K_act"])
    assert st == 0
    assert int(b[0]) == ex["budget"]
    assert int(k[0]) == pack_key(ex["tier"], ex["budget"], 7)


def test_closed_form_linear_model():
    """gamma = 1, no load dependence, no attention term, no hits: L = P * (c_tok + c_iter / chunk),
    so the budget is TTFT - L - elapsed exactly (Eq. 3-5 collapse to one line)."""
    d = wl.default_params(gamma_q16=65536, c_attn_q20=0, c_dseq_q20=0, c_dkv_q20=0,
                          c_tok_q20=30_000 * wl.Q20, c_iter_q20=512 * 1000 * wl.Q20, ttft_ns=[2 * S], tpot_ns=[0])
    p = oracle.make_params(d)
    for P in (1, 17, 1000, 131072):
        for elapsed in (0, 123_456_789):
            b, k, st = oracle.budget(p, one_request(P, 10, (0, 0, 0), elapsed), 10 * S, 5, 999)
            assert st == 0
            assert int(b[0]) == 2 * S - P * (30_000 + 1000) - elapsed


def real_budget(d, P, O, n, elapsed, ttft, tpot, D, K):
    """Eq. 3-5 in exact rational arithmetic, no flooring (independent of the integer shifts)."""
    f = lambda q: Fraction(q, 1 << 20)
    chunk = 1 << d["chunk_shift"]
    gamma = Fraction(d["gamma_q16"], 1 << 16)

    def iter_ns(D_, K_):
        return f(d["c_iter_q20"]) + D_ * f(d["c_dseq_q20"]) + K_ * f(d["c_dkv_q20"])

    def T(k, x):
        return 0 if x == 0 else d["delta_ns"][k] + x * d["blk_ns"][k]

    s = sum(n) * d["bt"]
    loads = [(D, K), (max(D, d["max_batch"] - 1), max(K, (d["max_batch"] - 1) * d["max_ctx_avg"]))]
    Ls, tds = [], []
    for D_, K_ in loads:
        A = f(d["c_tok_q20"]) + iter_ns(D_, K_) / chunk
        Ls.append(T(1, n[1]) + T(2, n[2]) + A * (P - s) + f(d["c_attn_q20"]) * (P * P - s * s))
        tds.append(iter_ns(D_ + 1, K_ + P) + f(d["c_tok_q20"]) * chunk)
    L = (Ls[0] + Ls[1]) / 2 * gamma
    B = ttft - L
    tdec = (tds[0] + tds[1]) / 2 * gamma
    pen = 0 if tpot == 0 else O * max(0, tdec - tpot)
    return B, B - elapsed - pen, Ls


def test_integer_model_tracks_real_arithmetic():
    """The integer model floors a handful of times; it must stay within a few ns of the exact
    rational value (times pred_out for the penalty term), also at the extreme input bounds."""
    rng = np.random.default_rng(5)
    d = wl.default_params(ttft_ns=[1 * S, 30 * S], tpot_ns=[50 * MS, 20 * MS])
    p = oracle.make_params(d)
    cases = [(131072, 1 << 20, (4000, 4000, 191), 1 << 50, 1, 1 << 16, 1 << 32)]
    for _ in range(300):
        P = int(rng.integers(1, 131073))
        hit = int(rng.integers(0, (P - 1) // 16 + 1))
        n0 = int(rng.integers(0, hit + 1))
        n1 = int(rng.integers(0, hit - n0 + 1))
        cases.append((P, int(rng.integers(0, 1 << 17)), (n0, n1, hit - n0 - n1), int(rng.integers(0, 60 * S)),
                      int(rng.integers(0, 2)), int(rng.integers(0, 600)), int(rng.integers(0, 1 << 22))))
    for P, O, n, elapsed, cls, D, K in cases:
        b, k, st = oracle.budget(p, one_request(P, O, n, elapsed, cls=cls, now=1 << 51), 1 << 51, D, K)
        assert st == 0
        B, want, _ = real_budget(d, P, O, n, elapsed, d["ttft_ns"][cls], d["tpot_ns"][cls], D, K)
        assert abs(int(b[0]) - want) <= 3 + 2 * O
        tier2 = int(k[0]) >> 63
        if abs(B) > 3:
            assert tier2 == (1 if B <= 0 else 0)


def test_remaining_budget_decays_one_for_one():
    """Eq. 5: a request waiting dt longer has exactly dt less budget; its tier bit does not move."""
    w = wl.config_tiny(3)
    p = oracle.make_params(w.params)
    b0, k0, _ = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
    for dt in (1, 999, 25 * MS, 7 * S):
        b1, k1, _ = oracle.budget(p, w.reqs, w.now_ns + dt, w.D_act, w.K_act)
        assert np.array_equal(b1, b0 - dt)
        assert np.array_equal(k1 >> np.uint64(63), k0 >> np.uint64(63))


def test_tpot_zero_gives_paper_literal_budget():
    """With the decode term disabled the budget is Eq. 5 alone: it no longer depends on pred_out."""
    w = wl.config_tiny(1)
    d = dict(w.params, tpot_ns=[0, 0])
    p = oracle.make_params(d)
    b0, _, _ = oracle.budget(p, w.reqs, w.now_ns, 300, 2_000_000)
    r2 = dict(w.reqs, pred_out=np.full(w.n, 1 << 20, np.int32))
    b1, _, _ = oracle.budget(p, r2, w.now_ns, 300, 2_000_000)
    assert np.array_equal(b0, b1)
    # and with the term enabled under heavy load it can only lower the budget
    b2, _, _ = oracle.budget(oracle.make_params(w.params), w.reqs, w.now_ns, 300, 2_000_000)
    assert np.all(b2 <= b0) and np.any(b2 < b0)


def test_faster_tier_never_lowers_budget():
    """Moving one matched block host -> HBM (or deep -> host) removes transfer time and nothing else."""
    p = oracle.make_params(wl.default_params())
    for n in ((3, 5, 4), (0, 1, 1), (10, 100, 50)):
        P = (sum(n) + 2) * 16
        base, _, _ = oracle.budget(p, one_request(P, 50, n, 0), 10 * S, 10, 10_000)
        up1, _, _ = oracle.budget(p, one_request(P, 50, (n[0] + 1, n[1] - 1, n[2]), 0), 10 * S, 10, 10_000)
        up2, _, _ = oracle.budget(p, one_request(P, 50, (n[0], n[1] + 1, n[2] - 1), 0), 10 * S, 10, 10_000)
        assert up1[0] >= base[0] and up2[0] >= base[0]
        # a single block moved out of the host tier saves exactly blk_ns[1] (plus delta when it was the last one)
        gain = 40_000 + (10_000 if n[1] == 1 else 0)
        assert int(up1[0] - base[0]) in (int(gain * 1.25) - 1, int(gain * 1.25), int(gain * 1.25) + 1)


def test_load_only_lowers_budget_and_max_regime_dominates():
    w = wl.config_tiny(2)
    p = oracle.make_params(w.params)
    idle, _, _ = oracle.budget(p, w.reqs, w.now_ns, 0, 0)
    busy, _, _ = oracle.budget(p, w.reqs, w.now_ns, 100, 300_000)
    full, _, _ = oracle.budget(p, w.reqs, w.now_ns, 127, 300_000)
    over, _, _ = oracle.budget(p, w.reqs, w.now_ns, 300, 2_000_000)
    assert np.all(busy <= idle) and np.all(full <= busy) and np.all(over <= full)


def test_keys_sort_like_the_tuple():
    """Sorting by key == sorting by (tier, clamped budget, id); saturated budgets tie-break by id."""
    w = wl.config_llama8b(4, n=512, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    p = oracle.make_params(w.params)
    b, k, st = oracle.budget(p, w.reqs, w.now_ns, 400, 3_000_000)
    assert st == 0
    tier2 = (k >> np.uint64(63)).astype(np.int64)
    clamped = np.clip(b, -(1 << 39), (1 << 39) - 1)
    ids = w.reqs["id"].astype(np.int64)
    assert np.array_equal(np.argsort(k, kind="stable"), np.lexsort((ids, clamped, tier2)))
    for i in range(w.n):
        assert int(k[i]) == pack_key(2 if tier2[i] else 1, int(b[i]), int(ids[i]))
    assert np.any(b < -(1 << 39))  # the clamp is exercised


def test_precondition_flag():
    p = oracle.make_params(wl.default_params())
    ok = one_request(100, 5, (1, 1, 1), 0)
    assert oracle.budget(p, ok, 10 * S, 0, 0)[2] == 0
    for bad in (one_request(48, 5, (1, 1, 1), 0),          # whole prompt cached
                one_request(0, 5, (0, 0, 0), 0),
                one_request((1 << 17) + 1, 5, (0, 0, 0), 0),
                one_request(100, -1, (0, 0, 0), 0),
                one_request(100, 5, (-1, 0, 0), 0),
                one_request(100, 5, (0, 0, 0), 0, cls=3)):
        b, k, st = oracle.budget(p, bad, 10 * S, 0, 0)
        assert st == oracle.ST_EPRECOND
        assert int(k[0]) >> 63 == 1


def test_zero_budget_goes_to_tier_two():
    """Eq. 4 with B exactly 0: only a strictly positive budget enters the Tier-1 queue."""
    d = wl.default_params(gamma_q16=65536, c_attn_q20=0, c_dseq_q20=0, c_dkv_q20=0, c_tok_q20=30_000 * wl.Q20,
                          c_iter_q20=512 * 1000 * wl.Q20, ttft_ns=[1000 * 31_000, 1000 * 31_000 + 1], tpot_ns=[0, 0])
    p = oracle.make_params(d)
    b, k, _ = oracle.budget(p, one_request(1000, 1, (0, 0, 0), 0, cls=0), 10 * S, 0, 0)
    assert int(b[0]) == 0 and int(k[0]) >> 63 == 1
    b, k, _ = oracle.budget(p, one_request(1000, 1, (0, 0, 0), 0, cls=1), 10 * S, 0, 0)
    assert int(b[0]) == 1 and int(k[0]) >> 63 == 0
