"""Random parameters, queues and pools through the whole plan chain on the GPU, compared with the oracle
field by field (fixed seeds; the generator covers the validated parameter space, extremes included)."""
import numpy as np
import pytest

from chain import oracle_chain
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def _compare(w, link, hbm_reserve, stage_link, host_reserve, one_call=False):
    from paper_2608_06557_b200.runner import Instance
    out = oracle_chain(w, link, hbm_reserve, stage_link, host_reserve)
    res, pf, dr, st, ds = out["res"], out["pf"], out["dr"], out["st"], out["ds"]
    pools, plan = res["pools"], res["plan"]
    inst = Instance(w, alloc_pools=False)
    inst.enable_deep(w, alloc_pool=False)
    if one_call:
        inst.run_step(inst.step_args())     # one cascade_step call
    else:
        inst.run_schedule()                 # the three calls
    inst.run_prefetch(link, hbm_reserve)
    inst.run_dedup_restore()
    inst.run_stage_plan(stage_link, host_reserve)
    inst.run_dedup_stage()
    got, gp, gd = inst.fetch(), inst.fetch_prefetch(), inst.fetch_deep()
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(got[k], res[k]), k
    for k in ("x1", "x2", "tokens_run", "action", "evict_src", "evict_dst"):
        assert np.array_equal(got[k], plan[k]), k
    assert got["sched_counts"] == res["sched_counts"]
    assert got["plan_counts"] == dict(plan["counts"], n_restore=pf["counts"]["n_restore_total"])
    assert np.array_equal(gp["pf"], pf["pf"]) and gp["counts"] == pf["counts"]
    assert gd["dedup_restore"] == dr["counts"] and gd["dedup_stage"] == ds["counts"]
    assert np.array_equal(gd["restore_src_m"], dr["out_src"]) and np.array_equal(gd["restore_dst_m"], dr["out_dst"])
    assert np.array_equal(gd["staged"], st["staged"]) and gd["stage_counts"] == st["counts"]
    assert np.array_equal(gd["stage_src_m"], ds["out_src"]) and np.array_equal(gd["stage_dst_m"], ds["out_dst"])
    assert np.array_equal(gd["hbm_ref"], out["hbm_ref"]) and np.array_equal(gd["host_ref"], out["host_ref"])
    assert np.array_equal(gd["shared_restore"], dr["shared"]) and np.array_equal(gd["shared_stage"], ds["shared"])
    assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl) and np.array_equal(got["host_tbl"], pools.host_tbl)
    assert got["hbm_free_count"] == pools.hbm_free_count and got["host_free_count"] == pools.host_free_count
    nh, no = min(pools.hbm_free_count, len(pools.hbm_free)), min(pools.host_free_count, len(pools.host_free))
    assert np.array_equal(got["hbm_free"][:nh], pools.hbm_free[:nh])
    assert np.array_equal(got["host_free"][:no], pools.host_free[:no])
    assert got["status"] == (res["status"] | pf["status"] | dr["status"] | st["status"] | ds["status"])


@pytest.mark.parametrize("first", range(0, 160, 20))
def test_random_inputs_through_the_whole_plan_chain(first):
    for seed in range(first, first + 20):
        g = np.random.default_rng(1000 + seed)
        d = wl.fuzz_params(g)
        w = wl.fuzz_workload(g, d)
        args = (int(g.choice([0, 10**6, 10**9, 1 << 50])), int(g.choice([0, 2, 100])),
                int(g.choice([0, 10**6, 10**9, 1 << 50])), int(g.choice([0, 2, 100])))
        try:
            _compare(w, *args, one_call=seed % 2 == 1)
        except AssertionError as e:
            raise AssertionError(f"seed {1000 + seed}: {e}") from e


@pytest.mark.parametrize("first", range(0, 48, 8))
def test_random_inputs_with_queues_beyond_one_key_per_thread(first):
    """The same chain on queues of 4097 to 20000 requests: two and four keys per thread, the radix passes with the
    two-stage order, the tier plan with its per-request phase as a grid of its own (from 8192 requests up)."""
    for seed in range(first, first + 8):
        g = np.random.default_rng(7000 + seed)
        d = wl.fuzz_params(g)
        w = wl.fuzz_workload(g, d, sizes=(4097, 5000, 8191, 8192, 9000, 16384, 20000))
        args = (int(g.choice([0, 10**6, 10**9, 1 << 50])), int(g.choice([0, 2, 100])),
                int(g.choice([0, 10**6, 10**9, 1 << 50])), int(g.choice([0, 2, 100])))
        try:
            _compare(w, *args, one_call=seed % 2 == 1)
        except AssertionError as e:
            raise AssertionError(f"seed {7000 + seed}: {e}") from e


def test_request_parked_for_a_bad_class_is_still_offered_tokens_in_both_admission_modes():
    """A request whose class index is out of range is parked at the very end of the order with the lowest
    budget; it is still a request with a usable shape, so whatever tokens are left reach it, in the default
    and in the plan-first admission alike."""
    for plan_first in (0, 1):
        w = wl.config_tiny(1)
        w.params["plan_first"] = plan_first
        w.params["token_budget"] = 1 << 20
        w.params["tier2_reserve"] = 0
        w.reqs["cls"][3] = 6
        w.deep_tbl, w.deep_blocks = np.full_like(w.host_tbl, -1), 8
        _compare(w, 0, 0, 0, 0)
        from helpers import oracle_iteration
        res = oracle_iteration(w)
        assert res["status"] & 8 and res["grant_sched"][3] > 0 and res["order"][-1] == 3
