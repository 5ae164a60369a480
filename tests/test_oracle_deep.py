"""Pins for the deep-tier stage (first hop of the two-hop path of Eq. 6), for the one-copy-per-source
pass over a copy list, and for the record-to-record copy."""
import numpy as np

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl
from test_oracle_plan import py_cost_q20


# ---------------------------------------------------------------------------------------------------------
# stage plan
# ---------------------------------------------------------------------------------------------------------
def python_choice(d, D, K, P, n0, n1, n2, budget):
    """The request's own restore choice in Python integers: Eq. 7 by search (largest x with T_k(x) <= what is
    left), the deep tier only behind a fully restored host segment, then the cheapest of the three
    candidates, a tie restoring more."""
    T = lambda k, x: 0 if x == 0 else d["delta_ns"][k] + x * d["blk_ns"][k]
    rem = max(0, budget)
    x1 = 0
    while x1 < n1 and T(1, x1 + 1) <= rem:
        x1 += 1
    x2 = 0
    if x1 == n1 and n2 > 0:
        rem2 = rem - T(1, n1)
        while x2 < n2 and T(2, x2 + 1) <= rem2:
            x2 += 1
    best, bx = py_cost_q20(d, D, K, P, n0, 0, 0), (0, 0)
    for cand in ([(x1, 0)] if x1 else []) + ([(n1, x2)] if x2 else []):
        F = py_cost_q20(d, D, K, P, n0, *cand)
        if F <= best:
            best, bx = F, cand
    return bx


def python_stage(w, res, link_budget, reserve, host_count):
    d, r = w.params, w.reqs
    hop_d = max(0, d["delta_ns"][2] - d["delta_ns"][1])
    hop_b = max(1, d["blk_ns"][2] - d["blk_ns"][1])
    H = lambda x: 0 if x == 0 else hop_d + x * hop_b
    link, room = link_budget, host_count - reserve
    staged = np.zeros(w.n, np.int64)
    for s in res["order"]:
        if r["n2"][s] == 0 or res["plan"]["action"][s] in (oracle.ACT_EVICT, oracle.ACT_DROP):
            continue
        _, x2 = python_choice(d, w.D_act, w.K_act, int(r["prompt"][s]), int(r["n0"][s]), int(r["n1"][s]),
                              int(r["n2"][s]), int(res["budget"][s]))
        b = 0
        while b < x2 and b < room and H(b + 1) <= link:
            b += 1
        if b:
            staged[s] = b
            link -= H(b)
            room -= b
    return staged


def run_stage(w, link_budget, reserve, stage_cap=1 << 14):
    res = oracle_iteration(w)
    pools = res["pools"]
    p = oracle.make_params(w.params)
    before = dict(host_count=pools.host_free_count, host_tbl=pools.host_tbl.copy(), hbm_tbl=pools.hbm_tbl.copy(),
                  hbm_count=pools.hbm_free_count)
    out = oracle.stage_plan(p, w.reqs, res["budget"], res["order"], res["plan"]["action"], w.D_act, w.K_act,
                            link_budget, reserve, pools, w.deep_tbl, stage_cap)
    return res, out, before


def test_stage_matches_the_python_restatement_and_respects_every_bound():
    some_cut = some_full = 0
    for seed in range(6):
        for plan_first in (0, 1):
            w = wl.config_deep_shared(seed, n=96, host_free_target=(1 << 30) if seed % 2 else 300)
            w.params["plan_first"] = plan_first
            for link_budget, reserve in ((0, 0), (150_000, 0), (3_000_000, 0), (10**9, 0), (10**9, 250)):
                res, out, before = run_stage(w, link_budget, reserve)
                want = python_stage(w, res, link_budget, reserve, before["host_count"])
                assert np.array_equal(out["staged"], want), (seed, plan_first, link_budget, reserve)
                c = out["counts"]
                assert c["n_stage"] == want.sum() and c["n_requests"] == (want > 0).sum()
                assert c["host_free_after"] == before["host_count"] - want.sum()
                assert c["host_free_after"] >= min(reserve, before["host_count"])
                assert c["link_ns_left"] >= 0
                some_cut += c["n_short"] > 0
                some_full += c["n_short"] == 0 and c["n_stage"] > 0
                # the first hop never touches HBM
                assert np.array_equal(res["pools"].hbm_tbl, before["hbm_tbl"])
                assert res["pools"].hbm_free_count == before["hbm_count"]
    assert some_cut and some_full


def test_stage_ids_tables_and_list_pairing():
    w = wl.config_deep_shared(3, n=128)
    res, out, before = run_stage(w, 10**9, 0)
    pools, r = res["pools"], w.reqs
    ns = out["counts"]["n_stage"]
    assert ns > 0 and out["status"] == 0
    # popped from the top of the stack, in list order
    top = before["host_count"]
    assert np.array_equal(out["stage_dst"], pools.host_free[top - ns:top][::-1])
    assert pools.host_free_count == top - ns
    # list order = schedule order, request by request, block by block; the table cells agree with the list
    k = 0
    for s in res["order"]:
        b = int(out["staged"][s])
        lo = int(r["n0"][s] + r["n1"][s])
        assert np.array_equal(out["stage_src"][k:k + b], w.deep_tbl[s, lo:lo + b])
        assert np.array_equal(pools.host_tbl[s, lo:lo + b], out["stage_dst"][k:k + b])
        k += b
    assert k == ns
    # nothing else in the host table moved
    changed = pools.host_tbl != before["host_tbl"]
    assert changed.sum() == ns


def test_stage_hand_worked_three_requests():
    """bt 16, hop = (110000-10000) + x*(340000-40000) ns.  Slot 0: deep fetch of 3 blocks; slot 1 holds no deep
    block; slot 2: deep fetch of 2.  Order 2,0,1.  Link budget 1,050,000 ns: slot 2 takes 2 blocks
    (100000+600000 = 700000, leaving 350000), slot 0 gets floor((350000-100000)/300000) = 0 blocks."""
    d = wl.default_params(ttft_ns=[100 * wl.S])
    p = oracle.make_params(d)
    reqs = dict(prompt=[200, 100, 150], n0=[1, 0, 0], n1=[1, 2, 1], n2=[3, 0, 2])
    budget = np.array([50 * wl.S] * 3, np.int64)
    order = np.array([2, 0, 1], np.uint32)
    action = np.zeros(3, np.uint8)
    maxb = 16
    host_tbl = np.full((3, maxb), -1, np.int32)
    deep_tbl = np.full((3, maxb), -1, np.int32)
    deep_tbl[0, 2:5] = [70, 71, 72]
    deep_tbl[2, 1:3] = [80, 81]
    host_free = np.array([5, 6, 7, 8, 9, -1, -1, -1], np.int32)
    pools = oracle.Pools(None, host_tbl, None, 0, host_free, 5)
    out = oracle.stage_plan(p, reqs, budget, order, action, 0, 0, 1_050_000, 0, pools, deep_tbl, 8)
    assert out["staged"].tolist() == [0, 0, 2]
    assert out["stage_src"].tolist() == [80, 81] and out["stage_dst"].tolist() == [9, 8]
    assert host_tbl[2, 1:3].tolist() == [9, 8] and pools.host_free_count == 3
    assert out["counts"] == dict(n_stage=2, n_requests=1, n_short=1, host_free_after=3, link_ns_left=350_000)
    # a looser link: both are served, slot 0 after slot 2
    host_tbl[:] = -1
    pools = oracle.Pools(None, host_tbl, None, 0, host_free, 5)
    out = oracle.stage_plan(p, reqs, budget, order, action, 0, 0, 10**9, 0, pools, deep_tbl, 8)
    assert out["staged"].tolist() == [3, 0, 2]
    assert out["stage_src"].tolist() == [80, 81, 70, 71, 72] and out["stage_dst"].tolist() == [9, 8, 7, 6, 5]
    assert host_tbl[0, 2:5].tolist() == [7, 6, 5]
    # the host pool keeps two records back: slot 2 gets its two, slot 0 only one
    host_tbl[:] = -1
    pools = oracle.Pools(None, host_tbl, None, 0, host_free, 5)
    out = oracle.stage_plan(p, reqs, budget, order, action, 0, 0, 10**9, 2, pools, deep_tbl, 8)
    assert out["staged"].tolist() == [1, 0, 2] and out["counts"]["n_short"] == 1
    # a preempted request stages nothing; a budget too tight for the host segment never reaches the deep tier
    host_tbl[:] = -1
    pools = oracle.Pools(None, host_tbl, None, 0, host_free, 5)
    act2 = np.array([oracle.ACT_DROP, 0, 0], np.uint8)
    b2 = np.array([50 * wl.S, 50 * wl.S, 40_000], np.int64)     # T_1(1) = 50000 > 40000
    out = oracle.stage_plan(p, reqs, b2, order, act2, 0, 0, 10**9, 0, pools, deep_tbl, 8)
    assert out["staged"].tolist() == [0, 0, 0] and pools.host_free_count == 5


def test_stage_list_capacity_and_counts_only_mode():
    w = wl.config_deep_shared(1, n=96)
    res, full, _ = run_stage(w, 10**9, 0)
    res2, cut, _ = run_stage(w, 10**9, 0, stage_cap=10)
    assert cut["status"] & oracle.ST_ELISTCAP and len(cut["stage_src"]) == 10
    assert np.array_equal(cut["stage_src"], full["stage_src"][:10])
    assert np.array_equal(cut["staged"], full["staged"])
    assert np.array_equal(res2["pools"].host_tbl, res["pools"].host_tbl)
    # counts only: no table, no list
    p = oracle.make_params(w.params)
    res3 = oracle_iteration(w)
    pools = oracle.Pools(None, None, None, 0, None, res3["pools"].host_free_count)
    out = oracle.stage_plan(p, w.reqs, res3["budget"], res3["order"], res3["plan"]["action"], w.D_act, w.K_act,
                            10**9, 0, pools, None, 0)
    assert np.array_equal(out["staged"], full["staged"]) and out["counts"]["n_stage"] == full["counts"]["n_stage"]


def test_staged_blocks_reach_hbm_at_the_last_hop():
    """Two iterations: the first stages deep blocks into host records, the caller folds them into the hit
    profile (n1 += staged, n2 -= staged), the second restores them.  The bytes that land in the HBM block of
    table cell (r, j) must be the deep record that cell named at the start."""
    w = wl.config_deep_shared(5, n=64, n_chunks=2, chunk_bytes=128)
    w.params["plan_first"] = 1
    bb = w.block_bytes
    rng = np.random.default_rng(0)
    hbm = rng.integers(0, 256, w.layout["n_blocks"] * bb, dtype=np.uint8)
    host = rng.integers(0, 256, w.host_blocks * bb, dtype=np.uint8)
    deep = rng.integers(0, 256, w.deep_blocks * bb, dtype=np.uint8)
    res, out, _ = run_stage(w, 10**9, 0)
    assert out["counts"]["n_stage"] > 0
    assert oracle.kv_stage(deep, w.deep_blocks, host, w.host_blocks, bb, out["stage_src"], out["stage_dst"]) == 0
    pools = res["pools"]
    assert oracle.kv_evict(hbm, w.layout, host, w.host_blocks, res["plan"]["evict_src"], res["plan"]["evict_dst"]) == 0
    assert oracle.kv_restore(hbm, w.layout, host, w.host_blocks, res["plan"]["restore_src"], res["plan"]["restore_dst"]) == 0
    # fold and run a second iteration a little later with loose targets so that the staged blocks are restored
    staged, x1 = out["staged"], np.where(res["grant"] > 0, res["plan"]["x1"], 0)
    keep = (staged > 0) & (res["plan"]["action"] <= oracle.ACT_RETAIN)
    w2 = wl.Workload("second", dict(w.params, ttft_ns=[500 * wl.S, 500 * wl.S]), {k: v.copy() for k, v in w.reqs.items()},
                     w.now_ns + 10 * wl.MS, w.D_act, w.K_act, w.layout, w.host_blocks, w.maxb, pools.hbm_tbl,
                     pools.host_tbl, pools.hbm_free, pools.hbm_free_count, pools.host_free, pools.host_free_count)
    w2.reqs["n0"] = (w.reqs["n0"] + x1).astype(np.int32)
    w2.reqs["n1"] = (w.reqs["n1"] - x1 + staged).astype(np.int32)
    w2.reqs["n2"] = (w.reqs["n2"] - staged).astype(np.int32)
    w2.params["token_budget"] = 1 << 20
    w2.params["max_batch"] = 4096
    res2 = oracle_iteration(w2)
    plan2 = res2["plan"]
    assert oracle.kv_evict(hbm, w.layout, host, w.host_blocks, plan2["evict_src"], plan2["evict_dst"]) == 0
    assert oracle.kv_restore(hbm, w.layout, host, w.host_blocks, plan2["restore_src"], plan2["restore_dst"]) == 0
    checked = 0
    lay = w.layout
    for s in np.nonzero(keep)[0]:
        if res2["grant"][s] <= 0:
            continue
        lo = int(w.reqs["n0"][s] + w.reqs["n1"][s])
        upto = int(w2.reqs["n0"][s] + plan2["x1"][s])
        for j in range(lo, min(lo + int(staged[s]), upto)):
            g, dr = int(res2["pools"].hbm_tbl[s, j]), int(w.deep_tbl[s, j])
            for c in range(lay["n_chunks"]):
                a = c * lay["chunk_stride"] + g * lay["block_stride"]
                b = dr * bb + c * lay["chunk_bytes"]
                assert np.array_equal(hbm[a:a + lay["chunk_bytes"]], deep[b:b + lay["chunk_bytes"]]), (s, j, c)
            checked += 1
    assert checked > 20


# ---------------------------------------------------------------------------------------------------------
# one copy per distinct source block
# ---------------------------------------------------------------------------------------------------------
def test_dedup_hand_worked_list():
    """Sources 5,7,5,9,7,5 -> kept entries at positions 0,1,3; destinations 12,14,15 go back on the stack in
    that order; 5 is shared by three entries, 7 by two."""
    src = [5, 7, 5, 9, 7, 5]
    dst = [10, 11, 12, 13, 14, 15]
    # three slots: slot 0 holds 5,7 at cells 0,1; slot 1 holds 5,9 at cells 2,3; slot 2 holds 7,5 at cells 0,1
    src_tbl = np.full((3, 4), -1, np.int32)
    dst_tbl = np.full((3, 4), -1, np.int32)
    src_tbl[0, :2], dst_tbl[0, :2] = [5, 7], [10, 11]
    src_tbl[1, 2:], dst_tbl[1, 2:] = [5, 9], [12, 13]
    src_tbl[2, :2], dst_tbl[2, :2] = [7, 5], [14, 15]
    free = np.array([40, 41, -1, -1, -1, -1], np.int32)
    ref = np.zeros(32, np.int32)
    out = oracle.dedup([0, 2, 0], None, [2, 2, 2], None, src_tbl, dst_tbl, src, dst, 6, 16, 32, free, 2, ref)
    assert out["out_src"].tolist() == [5, 7, 9] and out["out_dst"].tolist() == [10, 11, 13]
    assert free.tolist() == [40, 41, 12, 14, 15, -1] and out["free_count"] == 5
    assert dst_tbl[0, :2].tolist() == [10, 11] and dst_tbl[1, 2:].tolist() == [10, 13] and dst_tbl[2, :2].tolist() == [11, 10]
    assert ref[10] == 3 and ref[11] == 2 and ref[13] == 1 and ref.sum() == 6
    assert out["shared"].tolist() == [1, 1, 1]
    assert out["counts"] == dict(n_in=6, n_unique=3, n_surplus=3, n_shared_requests=3, max_share=3, free_after=5)
    assert out["status"] == 0


def test_dedup_leaves_a_list_without_repeats_alone():
    rng = np.random.default_rng(2)
    src = rng.permutation(500)[:200].astype(np.int32)
    dst = rng.permutation(900)[:200].astype(np.int32)
    src_tbl = src.reshape(20, 10).copy()
    dst_tbl = dst.reshape(20, 10).copy()
    free = np.full(64, -1, np.int32)
    ref = np.zeros(900, np.int32)
    out = oracle.dedup(np.zeros(20), None, np.full(20, 10), None, src_tbl, dst_tbl, src, dst, 200, 500, 900, free, 0, ref)
    assert np.array_equal(out["out_src"], src) and np.array_equal(out["out_dst"], dst)
    assert np.array_equal(dst_tbl, dst.reshape(20, 10)) and (free == -1).all() and out["free_count"] == 0
    assert (ref[dst] == 1).all() and ref.sum() == 200 and not out["shared"].any()
    assert out["counts"]["max_share"] == 1 and out["counts"]["n_surplus"] == 0


def _random_shared_case(rng, n=40, maxb=24, n_src=300, n_dst=400):
    """Slots whose cell ranges draw their source ids from a small pool (so repeats are common), the list
    built slot by slot, cell by cell, with distinct destinations."""
    lo = rng.integers(0, 6, n).astype(np.int32)
    ln = rng.integers(0, maxb - 6, n).astype(np.int32)
    src_tbl = np.full((n, maxb), -1, np.int32)
    dst_tbl = np.full((n, maxb), -1, np.int32)
    dst_ids = rng.permutation(n_dst).astype(np.int32)
    ls, ld, k = [], [], 0
    hot = rng.permutation(n_src)[:60]
    for r in rng.permutation(n):
        for j in range(lo[r], lo[r] + ln[r]):
            if k >= len(dst_ids) - 50:
                ln[r] = j - lo[r]
                break
            s = int(rng.choice(hot)) if rng.uniform() < 0.5 else int(rng.integers(0, n_src))
            if s in src_tbl[r]:
                s = int(rng.integers(0, n_src))      # a slot does not hold one block twice (a second draw may)
            src_tbl[r, j], dst_tbl[r, j] = s, dst_ids[k]
            ls.append(s)
            ld.append(dst_ids[k])
            k += 1
    free = np.full(n_dst, -1, np.int32)
    nf = len(dst_ids) - k
    free[:nf] = dst_ids[k:]
    return lo, ln, src_tbl, dst_tbl, np.array(ls, np.int32), np.array(ld, np.int32), free, nf


def test_dedup_against_numpy_unique_and_conservation():
    rng = np.random.default_rng(11)
    for _ in range(30):
        lo, ln, src_tbl, dst_tbl, ls, ld, free, nf = _random_shared_case(rng)
        free0, tbl0 = free.copy(), dst_tbl.copy()
        ref = np.zeros(400, np.int32)
        out = oracle.dedup(lo, None, ln, None, src_tbl, dst_tbl, ls, ld, len(ls), 300, 400, free, nf, ref)
        uniq, first, counts = np.unique(ls, return_index=True, return_counts=True)
        keep = np.sort(first)
        assert np.array_equal(out["out_src"], ls[keep]) and np.array_equal(out["out_dst"], ld[keep])
        surplus = np.delete(ld, keep)
        assert np.array_equal(free[nf:nf + len(surplus)], surplus) and out["free_count"] == nf + len(surplus)
        assert np.array_equal(free[:nf], free0[:nf])
        # every destination id is either still in use by the list or back on the stack, never both
        assert sorted(np.concatenate([out["out_dst"], surplus]).tolist()) == sorted(ld.tolist())
        canon = dict(zip(ls[keep].tolist(), ld[keep].tolist()))
        share = dict(zip(uniq.tolist(), counts.tolist()))
        for r in range(len(lo)):
            cells = range(lo[r], lo[r] + ln[r])
            assert [dst_tbl[r, j] for j in cells] == [canon[int(src_tbl[r, j])] for j in cells]
            assert out["shared"][r] == int(any(share[int(src_tbl[r, j])] > 1 for j in cells))
        outside = np.ones_like(dst_tbl, bool)
        for r in range(len(lo)):
            outside[r, lo[r]:lo[r] + ln[r]] = False
        assert np.array_equal(dst_tbl[outside], tbl0[outside])
        for s, d in canon.items():
            assert ref[d] == share[s]
        assert ref.sum() == len(ls)
        assert out["counts"]["max_share"] == counts.max() and out["counts"]["n_shared_requests"] == out["shared"].sum()


def test_dedup_gives_every_cell_the_bytes_the_full_list_would_have():
    """Copy with the full list and with the merged list: cell (r, j) must see the same bytes either way."""
    rng = np.random.default_rng(5)
    lo, ln, src_tbl, dst_tbl, ls, ld, free, nf = _random_shared_case(rng)
    lay = wl.kv_layout(400, 2, 32)
    bb = 64
    host = rng.integers(0, 256, 300 * bb, dtype=np.uint8)
    hbm_full = np.zeros(400 * bb, np.uint8)
    hbm_merged = np.zeros(400 * bb, np.uint8)
    tbl_full = dst_tbl.copy()
    oracle.kv_restore(hbm_full, lay, host, 300, ls, ld)
    out = oracle.dedup(lo, None, ln, None, src_tbl, dst_tbl, ls, ld, len(ls), 300, 400, free, nf, np.zeros(400, np.int32))
    assert out["counts"]["n_surplus"] > 0
    oracle.kv_restore(hbm_merged, lay, host, 300, out["out_src"], out["out_dst"])

    def block(pool, g):
        return np.concatenate([pool[c * lay["chunk_stride"] + g * lay["block_stride"]:][:32] for c in range(2)])

    for r in range(len(lo)):
        for j in range(lo[r], lo[r] + ln[r]):
            assert np.array_equal(block(hbm_full, tbl_full[r, j]), block(hbm_merged, dst_tbl[r, j]))
    # surplus blocks were never written
    for g in free[nf:out["free_count"]]:
        assert not block(hbm_merged, g).any()


def test_dedup_degenerate_lists():
    # empty list
    free = np.full(4, -1, np.int32)
    out = oracle.dedup([0], None, [0], None, np.full((1, 4), -1, np.int32), np.full((1, 4), -1, np.int32),
                       np.zeros(1, np.int32), np.zeros(1, np.int32), 0, 8, 8, free, 0, np.zeros(8, np.int32))
    assert len(out["out_src"]) == 0 and out["counts"]["n_in"] == 0 and out["free_count"] == 0
    # one source everywhere
    m = 50
    src_tbl = np.full((m, 2), 3, np.int32)
    dst_tbl = np.arange(2 * m, dtype=np.int32).reshape(m, 2)
    dst_tbl[:, 1] = -1
    src_tbl[:, 1] = -1
    free = np.full(64, -1, np.int32)
    ref = np.zeros(128, np.int32)
    out = oracle.dedup(np.zeros(m), None, np.ones(m), None, src_tbl, dst_tbl, np.full(m, 3), dst_tbl[:, 0].copy(), m, 8,
                       128, free, 0, ref)
    assert out["out_src"].tolist() == [3] and out["out_dst"].tolist() == [0]
    assert (dst_tbl[:, 0] == 0).all() and ref[0] == m and out["counts"]["max_share"] == m
    assert free[:m - 1].tolist() == list(range(2, 2 * m, 2)) and out["shared"].all()
    # ids outside their pools are passed through untouched and flagged
    src = np.array([2, 99, 2, -1, 2], np.int32)
    dst = np.array([5, 6, 7, 8, 500], np.int32)
    free = np.full(8, -1, np.int32)
    ref = np.zeros(16, np.int32)
    out = oracle.dedup([0], None, [0], None, np.full((1, 4), -1, np.int32), np.full((1, 4), -1, np.int32), src, dst, 5,
                       16, 16, free, 0, ref)
    assert out["status"] & oracle.ST_EBOUNDS
    assert out["out_src"].tolist() == [2, 99, -1, 2] and out["out_dst"].tolist() == [5, 6, 8, 500]
    assert free[:1].tolist() == [7] and ref[5] == 2


def test_dedup_on_the_plan_of_the_shared_prefix_workload():
    """The restore list and the stage list of the shared-prefix workload both hold repeats; after the pass
    the lists hold each source once and the HBM / host blocks of the repeats are free again."""
    w = wl.config_deep_shared(2, n=192)
    w.params["plan_first"] = 1
    res, st, before = run_stage(w, 10**9, 0)
    plan, pools, r = res["plan"], res["pools"], w.reqs
    assert len(np.unique(plan["restore_src"])) < len(plan["restore_src"])
    assert len(np.unique(st["stage_src"])) < len(st["stage_src"])
    ref = np.zeros(w.layout["n_blocks"], np.int32)
    x1 = np.where(res["grant"] > 0, plan["x1"], 0)
    hbm_count = pools.hbm_free_count
    out = oracle.dedup(r["n0"], None, x1, None, pools.host_tbl, pools.hbm_tbl, plan["restore_src"], plan["restore_dst"],
                       len(plan["restore_src"]), w.host_blocks, w.layout["n_blocks"], pools.hbm_free, hbm_count, ref)
    assert len(np.unique(out["out_src"])) == len(out["out_src"]) == len(np.unique(plan["restore_src"]))
    assert out["free_count"] == hbm_count + out["counts"]["n_surplus"]
    # stage list: sources are deep records, destinations host records
    # (run after the restore pass: the host table cells of the staged range are what the pass rewrites)
    ref2 = np.zeros(w.host_blocks, np.int32)
    host_count = pools.host_free_count
    out2 = oracle.dedup(r["n0"], r["n1"], st["staged"], None, w.deep_tbl, pools.host_tbl, st["stage_src"], st["stage_dst"],
                        len(st["stage_src"]), w.deep_blocks, w.host_blocks, pools.host_free, host_count, ref2)
    assert len(np.unique(out2["out_src"])) == len(out2["out_src"]) == len(np.unique(st["stage_src"]))
    assert out2["free_count"] == host_count + out2["counts"]["n_surplus"]
    assert out2["counts"]["n_shared_requests"] > 0


# ---------------------------------------------------------------------------------------------------------
# record-to-record copy
# ---------------------------------------------------------------------------------------------------------
def test_kv_stage_is_a_gather_of_records():
    rng = np.random.default_rng(9)
    bb = 96
    deep = rng.integers(0, 256, 40 * bb, dtype=np.uint8)
    host = rng.integers(0, 256, 30 * bb, dtype=np.uint8)
    src = rng.permutation(40)[:12].astype(np.int32)
    dst = rng.permutation(30)[:12].astype(np.int32)
    want = host.reshape(30, bb).copy()
    want[dst] = deep.reshape(40, bb)[src]
    assert oracle.kv_stage(deep, 40, host, 30, bb, src, dst) == 0
    assert np.array_equal(host.reshape(30, bb), want)
    # ids outside either pool are skipped and flagged
    before = host.copy()
    st = oracle.kv_stage(deep, 40, host, 30, bb, np.array([40, -1, 3], np.int32), np.array([0, 1, 30], np.int32))
    assert st & oracle.ST_EBOUNDS and np.array_equal(host, before)
