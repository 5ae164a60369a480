"""The allocation-free tier plan gives the same results as the context-based one.

Some users of the library cannot allocate device memory when they call it (all HBM already belongs to
their KV pool, or a host framework owns the allocator), so cascade_tier_plan_noalloc runs the same
kernels on a scratch area built into the library.  This file is collected last on purpose: it runs the
new entry point twice in a row, on different inputs, against cascade_tier_plan, through the C ABI."""
import numpy as np
import pytest

from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def _plan_both_ways(w):
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance

    ref = Instance(w, alloc_pools=False)
    ref.run_schedule()
    want = ref.fetch()

    got_inst = Instance(w, alloc_pools=False)
    c = got_inst.ctx
    c.budget(got_inst.reqs_struct, got_inst.n, w.now_ns, w.D_act, w.K_act, got_inst.budget, got_inst.key)
    c.schedule(got_inst.reqs_struct, got_inst.key, got_inst.n, w.D_act, got_inst.order, got_inst.grant,
               got_inst.sched_counts)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cs.tier_plan_noalloc(c.params, got_inst.reqs_struct, got_inst.budget, got_inst.order, got_inst.grant,
                         got_inst.n, w.D_act, w.K_act, got_inst.pools_struct, got_inst.plan_struct, status)
    got = got_inst.fetch()
    got["status"] |= int(status.item())
    return want, got


def _same(want, got):
    for k in want:
        if isinstance(want[k], np.ndarray):
            assert np.array_equal(want[k], got[k]), k
        else:
            assert want[k] == got[k], k


def test_no_alloc_plan_matches_on_two_calls_in_a_row():
    seen_victims = 0
    for w in (wl.config_tiny(0), wl.config_tiny(3),
              wl.config_llama8b(seed=9, n=3000, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9, hbm_free_target=64)):
        want, got = _plan_both_ways(w)
        _same(want, got)
        seen_victims += want["plan_counts"]["n_victims"]
    assert seen_victims > 0


def test_no_alloc_plan_rejects_oversized_queues_and_plan_only_mode_works():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance

    sw = wl.SchedulerSweep(4096, seed=2)
    w = sw.workload()
    want, got = _plan_both_ways(w)
    _same(want, got)
    _same_as_oracle(w, got)
    inst = Instance(w, alloc_pools=False)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(cs.CascadeError, match="CASCADE_ETOOBIG"):
        cs.tier_plan_noalloc(inst.ctx.params, inst.reqs_struct, inst.budget, inst.order, inst.grant,
                             cs.NOALLOC_MAX_REQUESTS + 1, w.D_act, w.K_act, inst.pools_struct, inst.plan_struct,
                             status)


def _same_as_oracle(w, got):
    ref = oracle_iteration(w, with_tables=w.hbm_tbl is not None)
    plan = ref["plan"]
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(got[k], ref[k]), k
    for k in ("x1", "x2", "tokens_run", "action"):
        assert np.array_equal(got[k], plan[k]), k
    assert got["plan_counts"] == plan["counts"] and got["status"] == ref["status"]
    if w.hbm_tbl is not None:
        pools = ref["pools"]
        assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl) and np.array_equal(got["host_tbl"], pools.host_tbl)
        assert got["hbm_free_count"] == pools.hbm_free_count and got["host_free_count"] == pools.host_free_count
        assert np.array_equal(got["hbm_free"][: pools.hbm_free_count], pools.hbm_free[: pools.hbm_free_count])
        assert np.array_equal(got["host_free"][: pools.host_free_count], pools.host_free[: pools.host_free_count])
        for k in ("restore_src", "restore_dst", "evict_src", "evict_dst"):
            assert np.array_equal(got[k], plan[k]), k


@pytest.mark.parametrize("n", [64, 3000, 4097, 8192])
def test_no_alloc_plan_against_the_oracle(n):
    """The entry point's own results against the CPU oracle, up to the largest queue it takes (the sizes
    above 4096 use two requests per thread, a geometry the smaller cases never reach)."""
    if n == 64:
        w = wl.config_tiny(1)
    elif n == 3000:
        w = wl.config_llama8b(seed=11, n=n, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9, hbm_free_target=64)
    else:
        w = wl.SchedulerSweep(n, seed=3).workload()
    _, got = _plan_both_ways(w)
    _same_as_oracle(w, got)


def test_no_alloc_plan_falls_back_to_a_smaller_cluster(monkeypatch):
    """A device that co-schedules fewer CTAs than the preferred cluster gets the same fallback geometry as
    cascade_tier_plan; exercised in a fresh process, where the per-device set-up still lies ahead."""
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests')\n"
        "import test_zz_no_alloc as t\n"
        "from paper_2608_06557_b200 import workload as wl\n"
        "w = wl.SchedulerSweep(8192, seed=4).workload()\n"
        "want, got = t._plan_both_ways(w)\n"
        "t._same(want, got); t._same_as_oracle(w, got)\n"
        "print('fallback ok')\n")
    import os
    env = dict(os.environ, CASCADE_MAX_CLUSTER="4")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "fallback ok" in out.stdout, out.stdout + out.stderr
