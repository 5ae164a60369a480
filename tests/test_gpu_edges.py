"""GPU parity on the edges: empty queues, maximum sizes, degenerate policies and pools."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl
from test_gpu_schedule import compare_iteration

pytestmark = pytest.mark.gpu
S = wl.S


def test_empty_queue_through_every_call():
    import torch
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_tiny(0)
    inst = Instance(w)
    inst.n = 0
    inst.plan_counts.fill_(7)
    inst.sched_counts.fill_(7)
    hbm_before = inst.hbm_free_count.item()
    inst.run_iteration()
    inst.run_prefetch(10**6, 0)
    got = inst.fetch()
    assert got["sched_counts"] == dict(n_tier1=0, n_admitted=0, tokens_granted=0)
    assert all(v == 0 for k, v in got["plan_counts"].items() if k not in ("hbm_free_after", "host_free_after"))
    assert got["plan_counts"]["hbm_free_after"] == hbm_before == got["hbm_free_count"]
    assert got["status"] == 0
    assert inst.fetch_prefetch()["counts"]["n_prefetch"] == 0


def big_queue(n, maxb, seed):
    """n short requests with tables of width maxb (hit blocks within the row), plenty of both tiers."""
    rng = np.random.default_rng(seed)
    params = wl.default_params(ttft_ns=[2 * S, 20 * S], tpot_ns=[50 * wl.MS] * 2, token_budget=40_000,
                               tier2_reserve=2_000, max_batch=4096)
    reqs = wl.draw_requests(rng, n, [0.5, 0.5], params["ttft_ns"], 300, (16, maxb * 16), [64, 64], (1, 512),
                            50 * S, 1.0, lambda g, m: g.uniform(0, 1, m), 0.5, 16)
    n_hbm = n_host = 600_000
    tbl = wl.place_blocks(rng, reqs, n_hbm, n_host, maxb, 1.0, 2_000, 0.5)
    return wl.Workload("big", params, reqs, 50 * S, 100, 100 * 300, wl.kv_layout(n_hbm, 1, 16), n_host, maxb, *tbl)


def test_maximum_queue_with_tables():
    w = big_queue(65536, 64, 1)
    got, ref = compare_iteration(w, "max-n")
    c = got["plan_counts"]
    assert c["n_admitted"] > 100 and c["n_victims"] > 0 and c["n_evict"] > 0


def test_largest_request_and_load():
    """One request at every input bound: 2^17-token prompt, 2^13 - 1 hit blocks, the largest load terms."""
    params = wl.default_params(ttft_ns=[1 << 40], tpot_ns=[1 << 40], token_budget=1 << 30, tier2_reserve=1 << 20,
                               max_batch=65536, max_ctx_avg=1 << 16, c_attn_q20=1 << 20, gamma_q16=1 << 17,
                               delta_ns=[0, 1 << 30, 1 << 30], blk_ns=[0, 1 << 27, 1 << 27])
    maxb = 8192
    n = 3
    reqs = dict(arrival_ns=np.array([0, 1 << 49, (1 << 50) - 5], np.int64),
                prompt=np.array([1 << 17, 1 << 17, 17], np.int32), pred_out=np.array([1 << 20, 0, 1], np.int32),
                n0=np.array([4000, 0, 0], np.int32), n1=np.array([4191, 8191, 1], np.int32),
                n2=np.array([0, 0, 0], np.int32), id=np.array([0x7FFFFF, 0xFFFFFFFF, 5], np.uint32),
                cls=np.zeros(n, np.uint8), flags=np.array([1, 0, 0], np.uint8))
    hbm_tbl = np.full((n, maxb), -1, np.int32)
    host_tbl = np.full((n, maxb), -1, np.int32)
    hbm_tbl[0, :4000] = np.arange(4000)
    host_tbl[0, 4000:8191] = np.arange(4191)
    host_tbl[1, :8191] = 5000 + np.arange(8191)
    host_tbl[2, 0] = 14000
    hbm_free = np.full(40000, -1, np.int32)
    hbm_free[:30000] = 4000 + np.arange(30000)
    host_free = np.full(20000, -1, np.int32)
    host_free[:5000] = 15000 + np.arange(5000)
    w = wl.Workload("bounds", params, reqs, 1 << 50, 1 << 16, 1 << 32, wl.kv_layout(40000, 1, 16), 20000, maxb,
                    hbm_tbl, host_tbl, hbm_free, 30000, host_free, 5000)
    got, ref = compare_iteration(w, "bounds")
    assert got["status"] == 0


@pytest.mark.parametrize("case", ["no_tokens", "batch_full", "reserve_exceeds_budget", "all_tier2", "no_hbm", "one"])
def test_degenerate_policies_and_pools(case):
    w = wl.config_tiny(4)
    if case == "no_tokens":
        w.params["token_budget"] = w.D_act            # decodes take everything
    elif case == "batch_full":
        w.params["max_batch"] = w.D_act               # no sequence slot left
    elif case == "reserve_exceeds_budget":
        w.params["tier2_reserve"] = 10**6
    elif case == "all_tier2":
        w.params["ttft_ns"] = [1, 1]
    elif case == "no_hbm":
        w.hbm_free_count = 0
        w.reqs["flags"][:] = 0
    elif case == "one":
        keep = slice(0, 1)
        w.reqs = {k: v[keep].copy() for k, v in w.reqs.items()}
        w.hbm_tbl, w.host_tbl = w.hbm_tbl[keep].copy(), w.host_tbl[keep].copy()
    got, ref = compare_iteration(w, case)
    if case in ("no_tokens", "batch_full"):
        assert got["sched_counts"]["n_admitted"] == 0
    if case == "all_tier2":
        assert got["sched_counts"]["n_tier1"] == 0 and got["sched_counts"]["n_admitted"] > 0
    if case == "no_hbm":
        assert got["plan_counts"]["n_admitted"] == 0 and got["status"] & 2


def test_empty_queue_and_empty_lists_through_the_added_calls():
    """n = 0 and zero-length lists for the stage plan, the merge pass, the stage copy and the queue update."""
    import torch
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_deep_shared(0, n=64, n_hbm=512, n_host=512, n_deep=512, n_chunks=2, chunk_bytes=64)
    inst = Instance(w)
    inst.enable_deep(w)
    pools = [inst.hbm_pool.fill_(1).clone(), inst.host_pool.fill_(2).clone(), inst.deep_pool.fill_(3).clone()]
    inst.n = 0
    host_before, hbm_before = inst.host_free_count.item(), inst.hbm_free_count.item()
    tbl_before = (inst.hbm_tbl.clone(), inst.host_tbl.clone())
    inst.stage_counts.fill_(7)
    inst.dedup_counts_restore.fill_(7)
    inst.dedup_counts_stage.fill_(7)
    inst.run_iteration_deep(10**9, 0)
    inst.stage_slot_update(w.reqs, np.zeros(0, np.int64))
    inst.run_slot_update()
    got, deep = inst.fetch(), inst.fetch_deep()
    assert got["status"] == 0
    assert deep["stage_counts"] == dict(n_stage=0, n_requests=0, n_short=0, host_free_after=host_before,
                                        link_ns_left=10**9)
    for k in ("dedup_restore", "dedup_stage"):
        c = deep[k]
        assert (c["n_in"], c["n_unique"], c["n_surplus"], c["n_shared_requests"], c["max_share"]) == (0, 0, 0, 0, 0)
    assert deep["dedup_restore"]["free_after"] == hbm_before and deep["dedup_stage"]["free_after"] == host_before
    assert got["hbm_free_count"] == hbm_before and got["host_free_count"] == host_before
    assert torch.equal(inst.hbm_tbl, tbl_before[0]) and torch.equal(inst.host_tbl, tbl_before[1])
    assert torch.equal(inst.hbm_pool, pools[0]) and torch.equal(inst.host_pool, pools[1]) and torch.equal(inst.deep_pool, pools[2])


def test_parameters_replaced_between_iterations():
    """cascade_set_params takes effect for the calls made afterwards; a rejected block leaves the old one in place."""
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_tiny(2)
    inst = Instance(w, alloc_pools=False)
    inst.run_schedule()
    first = inst.fetch()
    ref = oracle_iteration(w)
    assert np.array_equal(first["budget"], ref["budget"]) and np.array_equal(first["grant"], ref["grant"])
    w2 = wl.config_tiny(2)
    w2.params = dict(w2.params, ttft_ns=[4 * S, 9 * S], gamma_q16=70000, token_budget=999, plan_first=1, c_tok_q20=30_000 << 20)
    inst2 = Instance(w2, alloc_pools=False, ctx=inst.ctx)          # same context, new parameters
    inst2.run_schedule()
    second = inst2.fetch()
    ref2 = oracle_iteration(w2)
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(second[k], ref2[k]), k
    assert second["plan_counts"] == ref2["plan"]["counts"] and not np.array_equal(second["budget"], first["budget"])
    with pytest.raises(cs.CascadeError):
        inst.ctx.set_params(dict(w2.params, bt=0))
    inst3 = Instance(w2, alloc_pools=False, ctx=None)               # reference run with a fresh context
    inst3.run_schedule()
    third = inst3.fetch()
    inst2.hbm_free_count.fill_(w2.hbm_free_count)
    inst2.host_free_count.fill_(w2.host_free_count)
    inst2.hbm_tbl.copy_(inst3.hbm_tbl.new_tensor(w2.hbm_tbl))
    inst2.host_tbl.copy_(inst3.host_tbl.new_tensor(w2.host_tbl))
    inst2.hbm_free.copy_(inst3.hbm_free.new_tensor(w2.hbm_free))
    inst2.host_free.copy_(inst3.host_free.new_tensor(w2.host_free))
    inst2.run_schedule()                                            # the rejected call changed nothing
    again = inst2.fetch()
    for k in ("budget", "key", "order", "grant", "x1", "action"):
        assert np.array_equal(again[k], third[k]), k


def test_a_context_of_another_device_is_rejected_before_any_launch():
    """The hot calls launch on the current device and dereference the context's own allocations: a context
    created for another GPU is refused on the host.  Needs two GPUs; skipped otherwise."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    w = wl.config_tiny(0)
    inst = Instance(w, device="cuda:1", alloc_pools=False)      # context and buffers on GPU 1
    torch.cuda.set_device(0)
    try:
        with pytest.raises(cs.CascadeError, match="CASCADE_EINVAL"):
            inst.ctx.budget(inst.reqs_struct, inst.n, w.now_ns, w.D_act, w.K_act, inst.budget, inst.key, 0)
        with pytest.raises(cs.CascadeError, match="CASCADE_EINVAL"):
            inst.ctx.schedule(inst.reqs_struct, inst.key, inst.n, w.D_act, inst.order, inst.grant, inst.sched_counts, 0)
    finally:
        torch.cuda.set_device(0)
