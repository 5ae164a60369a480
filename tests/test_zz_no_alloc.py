"""The allocation-free tier plan gives the same results as the context-based one.

Some users of the library cannot allocate device memory when they call it (all HBM already belongs to
their KV pool, or a host framework owns the allocator), so cascade_tier_plan_noalloc runs the same
kernels on a scratch area built into the library.  This file is collected last on purpose: it runs the
new entry point twice in a row, on different inputs, against cascade_tier_plan, through the C ABI."""
import numpy as np
import pytest

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
    inst = Instance(w, alloc_pools=False)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(cs.CascadeError, match="CASCADE_ETOOBIG"):
        cs.tier_plan_noalloc(inst.ctx.params, inst.reqs_struct, inst.budget, inst.order, inst.grant,
                             cs.NOALLOC_MAX_REQUESTS + 1, w.D_act, w.K_act, inst.pools_struct, inst.plan_struct,
                             status)
