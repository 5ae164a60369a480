"""GPU parity: budget-bounded prefetch for queued requests, and the copies it adds to the restore list."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def both(w, link_budget, reserve, copies=False):
    import torch
    from paper_2608_06557_b200.runner import Instance
    ref = oracle_iteration(w)
    plan, pools = ref["plan"], ref["pools"]
    out = oracle.prefetch_plan(oracle.make_params(w.params), w.reqs, ref["budget"], ref["order"], ref["grant"],
                               plan["action"], plan["x1"], w.D_act, w.K_act, link_budget, reserve, pools,
                               plan["restore_src"], plan["restore_dst"], n_restore=plan["counts"]["n_restore"])
    inst = Instance(w, alloc_pools=copies)
    if copies:
        bb = w.block_bytes
        hbm_np = wl.pool_bytes(5, w.layout["n_blocks"] * bb).copy()
        host_np = wl.pool_bytes(6, w.host_blocks * bb).copy()
        inst.hbm_pool.copy_(torch.from_numpy(hbm_np))
        inst.host_pool.copy_(torch.from_numpy(host_np))
    inst.run_schedule()
    inst.run_prefetch(link_budget, reserve)
    if copies:
        inst.run_copies()
    got = inst.fetch()
    pf = inst.fetch_prefetch()
    assert np.array_equal(pf["pf"], out["pf"])
    assert pf["counts"] == out["counts"], (pf["counts"], out["counts"])
    assert got["status"] == (ref["status"] | out["status"])
    if w.hbm_tbl is not None:
        assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl)
        assert got["hbm_free_count"] == pools.hbm_free_count
        assert np.array_equal(got["restore_src"], out["restore_src"])
        assert np.array_equal(got["restore_dst"], out["restore_dst"])
        assert got["plan_counts"]["n_restore"] == out["counts"]["n_restore_total"]
    if copies:
        assert oracle.kv_evict(hbm_np, w.layout, host_np, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
        assert oracle.kv_restore(hbm_np, w.layout, host_np, w.host_blocks, out["restore_src"], out["restore_dst"]) == 0
        assert np.array_equal(inst.hbm_pool.cpu().numpy(), hbm_np)
        assert np.array_equal(inst.host_pool.cpu().numpy(), host_np)
    return out


@pytest.mark.parametrize("seed", range(6))
def test_tiny_prefetch(seed):
    total = 0
    for link_budget, reserve in ((0, 0), (15_000, 0), (400_000, 4), (10**9, 0), (10**9, 10)):
        w = wl.config_tiny(seed, hbm_free_target=32 + 60 * (seed % 3))
        w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
        total += both(w, link_budget, reserve)["counts"]["n_prefetch"]
    assert total > 0 or seed % 3 == 0


def test_prefetched_blocks_are_copied_with_the_restore_list():
    w = wl.config_tiny(5, hbm_free_target=400)
    w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    out = both(w, 10**9, 0, copies=True)
    assert out["counts"]["n_prefetch"] > 20


@pytest.mark.parametrize("n", [700, 5000, 20000])
def test_llama8b_shaped_prefetch(n):
    w = wl.config_llama8b(seed=n, n=n, hbm_bytes=4 * 10**9, host_bytes=3 * 10**9, hbm_free_target=600,
                          elapsed_scale=0.3)
    if n > 4096:
        w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
        w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    out = both(w, 20_000_000, 16)
    assert out["counts"]["n_prefetch"] > 0
    both(w, 3_000_000, 0)
