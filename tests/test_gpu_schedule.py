"""GPU parity: budget, ordering/admission and tier plan against the CPU oracle, bit for bit."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def _gpu():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance
    assert torch.cuda.is_available()
    return torch, cs, Instance


def compare_iteration(w, tag=""):
    torch, cs, Instance = _gpu()
    ref = oracle_iteration(w)
    inst = Instance(w, alloc_pools=False)
    inst.run_schedule()
    got = inst.fetch()
    for k in ("budget", "key", "order"):
        assert np.array_equal(got[k], ref[k]), (tag, k)
    assert np.array_equal(got["grant"], ref["grant"]), (tag, "grant")
    plan = ref["plan"]
    for k in ("x1", "x2", "tokens_run", "action"):
        assert np.array_equal(got[k], plan[k]), (tag, k)
    assert got["plan_counts"] == plan["counts"], (tag, got["plan_counts"], plan["counts"])
    assert got["status"] == ref["status"], (tag, got["status"], ref["status"])
    if w.hbm_tbl is not None:
        pools = ref["pools"]
        assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl), (tag, "hbm_tbl")
        assert np.array_equal(got["host_tbl"], pools.host_tbl), (tag, "host_tbl")
        assert got["hbm_free_count"] == pools.hbm_free_count and got["host_free_count"] == pools.host_free_count
        assert np.array_equal(got["hbm_free"][: pools.hbm_free_count], pools.hbm_free[: pools.hbm_free_count])
        assert np.array_equal(got["host_free"][: pools.host_free_count], pools.host_free[: pools.host_free_count])
        for k in ("restore_src", "restore_dst", "evict_src", "evict_dst"):
            assert np.array_equal(got[k], plan[k]), (tag, k)
    return got, ref


@pytest.mark.parametrize("seed", range(6))
def test_tiny_config(seed):
    got, ref = compare_iteration(wl.config_tiny(seed), f"tiny{seed}")
    assert got["plan_counts"]["n_victims"] > 0 or seed > 0


def test_tiny_schedule_counts_match():
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(0)
    ref = oracle_iteration(w)
    inst = Instance(w, alloc_pools=False)
    inst.ctx.budget(inst.reqs_struct, inst.n, w.now_ns, w.D_act, w.K_act, inst.budget, inst.key)
    inst.ctx.schedule(inst.reqs_struct, inst.key, inst.n, w.D_act, inst.order, inst.grant, inst.sched_counts)
    torch.cuda.synchronize()
    assert np.array_equal(inst.grant[: w.n].cpu().numpy(), ref["grant_sched"])
    sc = inst.sched_counts.cpu().numpy()
    assert int(sc[0] & 0xFFFFFFFF) == ref["sched_counts"]["n_tier1"]
    assert int(sc[0] >> 32) == ref["sched_counts"]["n_admitted"]
    assert int(sc[1]) == ref["sched_counts"]["tokens_granted"]


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 64, 65, 500, 513, 1023, 1024, 1025, 2047, 2048, 2049, 3000, 8192, 8193, 16384,
                               40000, 65536])
def test_llama8b_shaped_queue_sizes(n):
    """Spans every cluster / keys-per-thread configuration of the ordering kernel and ragged tails."""
    w = wl.config_llama8b(seed=n, n=n, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9, hbm_free_target=64)
    if n > 4096:      # tables of 65536 x 2048 are not needed to exercise the ordering: plan-only above 4096
        w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
        w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    compare_iteration(w, f"n{n}")


def test_heavy_load_tier2_and_saturated_budgets():
    w = wl.config_llama8b(seed=77, n=5000, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    w.D_act, w.K_act = 120, 4_000_000
    got, ref = compare_iteration(w, "heavy")
    assert 0 < ref["sched_counts"]["n_tier1"] < w.n
    assert np.any(ref["budget"] < -(1 << 39))


def test_duplicate_and_constant_keys_keep_slot_order():
    torch, cs, Instance = _gpu()
    w = wl.config_llama8b(seed=5, n=2500, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    p = oracle.make_params(w.params)
    inst = Instance(w, alloc_pools=False)
    rng = np.random.default_rng(0)
    for case in range(4):
        if case == 0:
            key = np.full(w.n, 12345 << 23, np.uint64)                        # every key equal: no pass runs
        elif case == 1:
            key = (rng.integers(0, 4, w.n).astype(np.uint64) << np.uint64(40))  # four distinct keys
        elif case == 2:
            key = rng.integers(0, 1 << 63, w.n).astype(np.uint64) * np.uint64(2) + np.uint64(1)
            key[::7] = np.uint64(0xFFFFFFFFFFFFFFFF)                           # equals the padding value
        else:
            key = np.arange(w.n, dtype=np.uint64)[::-1].copy()
        order, grant, counts, _ = oracle.schedule(p, w.reqs, key, w.D_act)
        inst.key.view(torch.int64)[: w.n].copy_(torch.from_numpy(key.view(np.int64)))
        inst.ctx.schedule(inst.reqs_struct, inst.key, inst.n, w.D_act, inst.order, inst.grant, inst.sched_counts)
        torch.cuda.synchronize()
        assert np.array_equal(inst.order[: w.n].cpu().numpy(), order), case
        assert np.array_equal(inst.grant[: w.n].cpu().numpy(), grant), case


@pytest.mark.parametrize("n", [2500, 5000, 16384, 40000, 65536])
def test_runs_of_equal_budgets_are_ordered_by_id_then_slot(n):
    """The radix path orders by bits 32..63 first and repairs runs of equal values afterwards: short runs inside a
    CTA locally, runs across a CTA boundary through the neighbour's shared memory, long runs by ordering again with every pass.  Keys are built so
    that the sorted position of every element is known, then runs are planted at chosen sorted positions: pairs and
    triples whose low bits are in descending slot order, runs of exactly 128 and of 129 (the local repair's limit),
    runs astride every multiple of 256 (every possible CTA boundary), full-key duplicates that must keep slot order,
    and a dense variant in which every 16 neighbours form a run."""
    torch, cs, Instance = _gpu()
    w = wl.config_llama8b(seed=n, n=n, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    p = oracle.make_params(w.params)
    inst = Instance(w, alloc_pools=False)
    rng = np.random.default_rng(n)

    def check(key, tag):
        order, grant, counts, _ = oracle.schedule(p, w.reqs, key, w.D_act)
        inst.key.view(torch.int64)[:n].copy_(torch.from_numpy(key.view(np.int64)))
        inst.ctx.schedule(inst.reqs_struct, inst.key, inst.n, w.D_act, inst.order, inst.grant, inst.sched_counts)
        torch.cuda.synchronize()
        assert np.array_equal(inst.order[:n].cpu().numpy(), order), tag
        assert np.array_equal(inst.grant[:n].cpu().numpy(), grant), tag
        assert inst.ctx.status()[0] == 0

    def keys_with_runs(runs, shift=32):
        """runs: list of (first sorted position, length).  Element at sorted position q has bits shift.. = q, except
        inside a run, where all share the run's first position and differ (or not) in the low 16 bits."""
        rank = np.arange(n, dtype=np.uint64)
        top = rank.copy()
        low = rng.integers(0, 1 << 16, n).astype(np.uint64)
        for q, length in runs:
            if q + length > n:
                continue
            top[q:q + length] = q
            low[q:q + length] = np.arange(length, 0, -1)          # descending: the repair has to reverse the run
            if length >= 3:
                low[q + 1] = low[q]                                # one full-key duplicate: slot order decides
        key_sorted = (top << np.uint64(shift)) | low
        slot_of = rng.permutation(n)                               # sorted position -> slot
        key = np.empty(n, np.uint64)
        key[slot_of] = key_sorted
        return key

    check(keys_with_runs([]), "no runs")
    check(keys_with_runs([(q, 2) for q in range(10, n - 2, 97)]), "pairs")
    check(keys_with_runs([(q, 3) for q in range(5, n - 3, 61)]), "triples")
    check(keys_with_runs([(100, 128), (900, 128), (n - 130, 128)]), "runs of 128")
    check(keys_with_runs([(100, 2), (2000, 129)]), "a run of 129")
    check(keys_with_runs([(3, 2), (700, 5)], shift=28), "every 16 neighbours equal above bit 32")
    check(keys_with_runs([(3, 2)], shift=26), "every 64 neighbours equal above bit 32: runs astride every boundary")
    check(keys_with_runs([(b - 1, 2) for b in range(256, n - 1, 256)]), "pairs astride every boundary")
    check(keys_with_runs([(b - 7, 14) for b in range(1024, n - 7, 1024)] + [(3, 2)]), "runs of 14 astride boundaries")
    check(keys_with_runs([(0, 2), (n - 2, 2)]), "first and last")


@pytest.mark.parametrize("n,iters", [(1024, 1000), (4096, 1000), (16384, 1000), (65536, 1000)])
def test_scheduler_sweep_iterations_with_churn(n, iters):
    """The scheduler-scale sweep at its stated length: 1000 consecutive iterations (plan-only) for each queue
    size; the clock advances 25 ms and 5 % of the slots and of the decode contexts are replaced every iteration."""
    torch, cs, Instance = _gpu()
    sw = wl.SchedulerSweep(n, seed=1)
    inst = Instance(sw.workload(), alloc_pools=False)
    slots = None
    for it in range(iters):
        w = sw.workload()
        ref = oracle_iteration(w, with_tables=False)
        if slots is None:
            inst.upload_requests(w.reqs)
        else:                                   # only the replaced slots travel, scattered by the library
            inst.stage_slot_update(w.reqs, slots)
            inst.run_slot_update()
        inst.set_clock(w.now_ns, w.D_act, w.K_act)
        inst.run_schedule()
        got = inst.fetch()
        assert got["status"] == 0
        for k in ("budget", "key", "order", "grant"):
            assert np.array_equal(got[k], ref[k]), (it, k)
        for k in ("x1", "x2", "tokens_run", "action"):
            assert np.array_equal(got[k], ref["plan"][k]), (it, k)
        assert got["plan_counts"] == ref["plan"]["counts"]
        if it + 1 < iters:
            slots = sw.step()
    for k, v in w.reqs.items():                 # the device queue is the host queue of the last iteration
        assert np.array_equal(inst.reqs[k][:n].cpu().numpy().view(v.dtype), v), k


def test_slot_update_edges():
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(0)
    inst = Instance(w, alloc_pools=False)
    before = {k: inst.reqs[k].clone() for k in inst.reqs}
    inst.stage_slot_update(w.reqs, np.zeros(0, np.int64))
    inst.run_slot_update()                      # m = 0: nothing happens
    new = {k: (v.copy() if k != "prompt" else v + 1) for k, v in w.reqs.items()}
    inst.stage_slot_update(new, np.array([5, 9], np.int64))
    inst.upd_slots[1] = w.n + 100               # outside the queue: skipped and flagged
    inst.run_slot_update()
    torch.cuda.synchronize()
    assert inst.ctx.status()[0] == cs.ST_EBOUNDS
    got = inst.reqs["prompt"].cpu().numpy()
    want = before["prompt"].cpu().numpy().copy()
    want[5] += 1
    assert np.array_equal(got, want)
    for k in inst.reqs:
        if k != "prompt":
            assert torch.equal(inst.reqs[k], before[k]), k


def test_precondition_flag_and_parking():
    w = wl.config_tiny(2)
    w.reqs["prompt"][3] = 0
    w.reqs["n0"][5] = -4
    w.reqs["cls"][7] = 6
    got, ref = compare_iteration(w, "precond")
    assert got["status"] & 8


def test_capacity_and_host_pressure_variants():
    w = wl.config_tiny(0)
    w.hbm_free_count = 3
    w.reqs["flags"][:] = 0
    got, ref = compare_iteration(w, "nospace")
    assert got["status"] & 2 and got["plan_counts"]["n_unadmitted"] > 0
    w = wl.config_tiny(0)
    w.host_free_count = 0
    got, ref = compare_iteration(w, "hostfull")
    assert got["plan_counts"]["n_evict"] == 0 and got["plan_counts"]["n_drop_blocks"] > 0
    w = wl.config_tiny(4)
    w.host_free_count = 7
    compare_iteration(w, "hosttight")


def test_host_side_validation_needs_no_launch():
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(0)
    inst = Instance(w, alloc_pools=False)
    lib = cs.raw()
    import ctypes as C
    h = inst.ctx._h
    assert lib.cascade_budget(h, C.byref(inst.reqs_struct), -1, 0, 0, 0, None, None, None) == cs.EINVAL
    assert lib.cascade_budget(h, C.byref(inst.reqs_struct), w.n + 1, 0, 0, 0, cs._p(inst.budget), cs._p(inst.key),
                              None) == cs.EINVAL
    assert lib.cascade_budget(h, C.byref(inst.reqs_struct), w.n, 0, -1, 0, cs._p(inst.budget), cs._p(inst.key),
                              None) == cs.ERANGE
    assert lib.cascade_budget(h, C.byref(inst.reqs_struct), w.n, 0, 0, 0, None, cs._p(inst.key), None) == cs.EINVAL
    bad = dict(w.params, blk_ns=[0, 0, 5])
    with pytest.raises(cs.CascadeError):
        cs.Context(bad, 16, 0)
    with pytest.raises(cs.CascadeError):
        cs.Context(w.params, cs.MAX_REQUESTS + 1, 0)


@pytest.mark.parametrize("policy", [1, 2, 3])
def test_comparison_policies(policy):
    w = wl.config_tiny(1)
    w.params = dict(w.params, policy=policy)
    compare_iteration(w, f"policy{policy}")
    w = wl.config_llama8b(seed=21, n=6000, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    w.params = dict(w.params, policy=policy)
    compare_iteration(w, f"policy{policy}-6000")


def test_latency_regimes_match():
    torch, cs, Instance = _gpu()
    for w in (wl.config_tiny(5), wl.config_llama8b(seed=8, n=3000, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)):
        w.reqs["prompt"][2] = 0                       # one request outside the input bounds
        inst = Instance(w, alloc_pools=False)
        lat = torch.empty((w.n, 4), dtype=torch.int64, device="cuda")
        inst.ctx.latency_regimes(inst.reqs_struct, w.n, w.D_act, w.K_act, lat)
        ref, st = oracle.latency_regimes(oracle.make_params(w.params), w.reqs, w.D_act, w.K_act)
        assert np.array_equal(lat.cpu().numpy(), ref)
        assert inst.ctx.status()[0] == st == 8


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_plan_first_admission(seed):
    w = wl.config_tiny(seed, hbm_free_target=200)
    w.params = dict(w.params, plan_first=1)
    if seed % 2:
        w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    compare_iteration(w, f"plan-first{seed}")
    w = wl.config_llama8b(seed=30 + seed, n=7000, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9, elapsed_scale=0.3)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    w.reqs["n2"][::5] = 3                                  # some deep-tier hits (the prompt bound still holds)
    w.reqs["prompt"][::5] += 48
    w.params = dict(w.params, plan_first=1, token_budget=200_000, max_batch=2048)
    got, ref = compare_iteration(w, f"plan-first-7000-{seed}")
    assert got["sched_counts"]["n_admitted"] > 50


@pytest.mark.parametrize("seed", [0, 3])
def test_one_call_iteration_equals_the_single_calls(seed):
    """cascade_step issues slot update, budget, schedule, tier plan and the fused move from C: same outputs as
    the oracle, same bytes moved."""
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(seed, hbm_free_target=60)
    w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    ref = oracle_iteration(w)
    plan = ref["plan"]
    bb = w.block_bytes
    hbm_np = wl.pool_bytes(3, w.layout["n_blocks"] * bb).copy()
    host_np = wl.pool_bytes(4, w.host_blocks * bb).copy()
    inst = Instance(w)
    inst.hbm_pool.copy_(torch.from_numpy(hbm_np))
    inst.host_pool.copy_(torch.from_numpy(host_np))
    # start from a queue whose first slots are wrong, and let the step's own slot update repair them
    slots = np.arange(0, w.n, 3, dtype=np.int64)
    for k in ("prompt", "n0", "n1"):
        inst.reqs[k][: w.n][torch.from_numpy(slots).cuda()] = 1
    inst.stage_slot_update(w.reqs, slots)
    args = inst.step_args(with_update=True, with_move=True)
    inst.run_step(args)
    got = inst.fetch()
    assert oracle.kv_evict(hbm_np, w.layout, host_np, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
    assert oracle.kv_restore(hbm_np, w.layout, host_np, w.host_blocks, plan["restore_src"], plan["restore_dst"]) == 0
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(got[k], ref[k]), k
    for k in ("x1", "x2", "tokens_run", "action", "restore_src", "restore_dst", "evict_src", "evict_dst"):
        assert np.array_equal(got[k], plan[k]), k
    assert got["plan_counts"] == plan["counts"] and got["status"] == ref["status"]
    assert np.array_equal(inst.hbm_pool.cpu().numpy(), hbm_np) and np.array_equal(inst.host_pool.cpu().numpy(), host_np)
    assert plan["counts"]["n_restore"] > 0 and plan["counts"]["n_evict"] > 0
    # plan-only queue, no update, no copies
    sw = wl.SchedulerSweep(5000, seed=seed)
    w2 = sw.workload()
    inst2 = Instance(w2, alloc_pools=False)
    inst2.run_step(inst2.step_args())
    got2, ref2 = inst2.fetch(), oracle_iteration(w2, with_tables=False)
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(got2[k], ref2[k]), k
    assert got2["plan_counts"] == ref2["plan"]["counts"]
