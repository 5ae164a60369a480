"""Pins added after a second round of planted slips survived: input-bound edges, the key's clamp, the default
offer with a deep-tier match, an exactly covered HBM need, and two prefetch decisions (hand-worked values)."""
import numpy as np

import oracle
from paper_2608_06557_b200 import workload as wl
from test_oracle_plan import three_requests

S, MS = wl.S, wl.MS


def one_request(**over):
    r = dict(arrival_ns=[0], prompt=[100], pred_out=[10], n0=[0], n1=[0], n2=[0], id=[5], cls=[0], flags=[0])
    r.update({k: [v] for k, v in over.items()})
    return r


def test_input_bounds_are_inclusive_where_stated():
    d = wl.default_params(ttft_ns=[S, S], tpot_ns=[0, 0])
    p = oracle.make_params(d)
    parked = (1 << 63) | 5
    # class index n_classes is outside, n_classes - 1 inside
    _, key, st = oracle.budget(p, one_request(cls=2), 0, 0, 0)
    assert st & oracle.ST_EPRECOND and int(key[0]) == parked
    _, key, st = oracle.budget(p, one_request(cls=1), 0, 0, 0)
    assert st == 0 and int(key[0]) != parked
    # predicted output length: 2^20 inside, 2^20 + 1 outside
    _, key, st = oracle.budget(p, one_request(pred_out=1 << 20), 0, 0, 0)
    assert st == 0
    b, key, st = oracle.budget(p, one_request(pred_out=(1 << 20) + 1), 0, 0, 0)
    assert st & oracle.ST_EPRECOND and int(key[0]) == parked and int(b[0]) == -(1 << 62)


def test_key_saturates_inside_its_forty_bits():
    """A budget beyond +2^39 ns saturates at 2^39 - 1: the field reads 2^40 - 1 and the queue bit stays clear."""
    d = wl.default_params(ttft_ns=[1 << 40], tpot_ns=[0], c_tok_q20=0, c_attn_q20=0, c_iter_q20=0, c_dseq_q20=0,
                          c_dkv_q20=0)
    p = oracle.make_params(d)
    b, key, st = oracle.budget(p, one_request(), 0, 0, 0)
    assert st == 0 and int(b[0]) == 1 << 40
    k = int(key[0])
    assert k >> 63 == 0 and (k >> 23) & ((1 << 40) - 1) == (1 << 40) - 1 and k & 0x7FFFFF == 5
    # and at the other end: far below -2^39 the field reads 0 (Tier-2 queue)
    d2 = dict(d, ttft_ns=[0])
    b, key, _ = oracle.budget(oracle.make_params(d2), one_request(arrival_ns=-(1 << 45)), 0, 0, 0)
    k = int(key[0])
    assert int(b[0]) == -(1 << 45) and k >> 63 == 1 and (k >> 23) & ((1 << 40) - 1) == 0


def test_default_offer_counts_every_matched_tier():
    """bt 16, prompt 400, 3 + 4 + 5 matched blocks: offered 400 - 12 * 16 = 208 tokens, not more."""
    d = wl.default_params(token_budget=4096, tier2_reserve=0)
    p = oracle.make_params(d)
    reqs = dict(prompt=[400], n0=[3], n1=[4], n2=[5])
    order, grant, counts, _ = oracle.schedule(p, reqs, np.array([7], np.uint64), 0)
    assert grant.tolist() == [208] and counts["tokens_granted"] == 208


def test_need_exactly_covered_by_the_free_list_takes_no_victim():
    p = oracle.make_params(wl.default_params())
    # slot 0 needs 2 restored + 4 computed blocks; exactly 6 are free: nobody is preempted
    reqs, budget, order, grant, pools = three_requests(hbm_free=6, host_free=20, victim_n0=5)
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    c = out["counts"]
    assert c["hbm_need"] == 6 and c["deficit"] == 0 and c["n_victims"] == 0 and c["hbm_free_after"] == 0
    assert out["action"][1] == oracle.ACT_RETAIN
    # one block short: one victim
    reqs, budget, order, grant, pools = three_requests(hbm_free=5, host_free=20, victim_n0=5)
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert out["counts"]["deficit"] == 1 and out["counts"]["n_victims"] == 1


def _queued_request(d, n1, budget_ns, link_budget, hbm_free=64):
    """One queued request holding n1 host blocks, nothing admitted."""
    p = oracle.make_params(d)
    maxb = 64
    reqs = dict(arrival_ns=[0], prompt=[16 * 40], pred_out=[1], n0=[0], n1=[n1], n2=[0], id=[0], cls=[0], flags=[0])
    hbm_tbl = np.full((1, maxb), -1, np.int32)
    host_tbl = np.full((1, maxb), -1, np.int32)
    host_tbl[0, :n1] = 100 + np.arange(n1)
    hf = np.full(128, -1, np.int32)
    hf[:hbm_free] = np.arange(hbm_free)
    pools = oracle.Pools(hbm_tbl, host_tbl, hf, hbm_free, np.full(4, -1, np.int32), 0, 128, 4)
    out = oracle.prefetch_plan(p, reqs, np.array([budget_ns], np.int64), np.array([0], np.uint32),
                               np.array([0], np.int32), np.array([0], np.uint8), np.array([0], np.int32), 0, 0,
                               link_budget, 0, pools, np.zeros(0, np.int32), np.zeros(0, np.int32))
    return out


def test_prefetch_link_allowance_pays_the_per_transfer_overhead_once():
    """delta 100 us, 40 us per block.  Link budget 220 us: 100 + 3 * 40 fits, a fourth block does not."""
    d = wl.default_params(delta_ns=[0, 100_000, 110_000], blk_ns=[0, 40_000, 340_000])
    out = _queued_request(d, n1=10, budget_ns=10 * S, link_budget=220_000)
    assert out["pf"].tolist() == [3] and out["counts"]["link_ns_left"] == 220_000
    out = _queued_request(d, n1=10, budget_ns=10 * S, link_budget=219_999)
    assert out["pf"].tolist() == [2]
    out = _queued_request(d, n1=10, budget_ns=10 * S, link_budget=100_000)
    assert out["pf"].tolist() == [0]


def test_prefetch_leaves_blocks_that_are_cheaper_to_recompute():
    """16 tokens per block at 50 us per token = 0.8 ms of compute per block (plus attention).  A host link that
    needs 2 ms per block loses against recomputing, one that needs 40 us wins."""
    slow = wl.default_params(blk_ns=[0, 2_000_000, 340_000])
    out = _queued_request(slow, n1=10, budget_ns=10 * S, link_budget=10 * S)
    assert out["pf"].tolist() == [0]
    fast = wl.default_params(blk_ns=[0, 40_000, 340_000])
    out = _queued_request(fast, n1=10, budget_ns=10 * S, link_budget=10 * S)
    assert out["pf"].tolist() == [10]


def test_a_dropped_victim_takes_no_host_room_from_the_next_one():
    """Two victims are needed.  The first one walked (last in the order) cannot be brought back within its own
    budget and is dropped; the second fits and finds the host pool's 4 free records all its own."""
    PRIV = oracle.FLAG_HBM_PRIVATE
    p = oracle.make_params(wl.default_params())
    maxb = 32
    reqs = dict(prompt=[16 * 10, 400, 400], n0=[0, 4, 3], n1=[0, 0, 0], n2=[0, 0, 0], flags=[0, PRIV, PRIV])
    hbm_tbl = np.full((3, maxb), -1, np.int32)
    host_tbl = np.full((3, maxb), -1, np.int32)
    hbm_tbl[1, :4] = [10, 11, 12, 13]
    hbm_tbl[2, :3] = [20, 21, 22]
    hf = np.full(64, -1, np.int32)
    hf[:4] = [1, 2, 3, 4]
    of = np.full(8, -1, np.int32)
    of[:4] = [30, 31, 32, 33]
    pools = oracle.Pools(hbm_tbl, host_tbl, hf, 4, of, 4, 64, 8)
    budget = np.array([10**9, 10**9, 1000], np.int64)        # slot 2: T_1(3) = 10 us + 3 * 40 us > 1 us
    order = np.array([0, 1, 2], np.uint32)
    grant = np.array([160, 0, 0], np.int32)                  # slot 0 computes 10 blocks: 4 free, 6 short
    out = oracle.tier_plan(p, reqs, budget, order, grant, 0, 0, pools)
    assert out["counts"]["deficit"] == 6 and out["counts"]["n_victims"] == 2
    assert out["action"].tolist() == [oracle.ACT_NONE, oracle.ACT_EVICT, oracle.ACT_DROP]
    assert out["evict_src"].tolist() == [10, 11, 12, 13] and out["evict_dst"].tolist() == [33, 32, 31, 30]
    assert out["counts"]["n_drop_blocks"] == 3 and pools.host_free_count == 0
