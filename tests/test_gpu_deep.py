"""GPU parity for the deep-tier stage plan, the one-copy-per-source pass and the stage copy (bit exact)."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu

DD_NAMES = ("n_in", "n_unique", "n_surplus", "n_shared_requests", "max_share", "free_after")


def oracle_deep(w, link_budget, reserve, stage_cap=None):
    """Oracle side of run_iteration_deep's plan steps: plan, merged restore list, stage plan, merged stage list."""
    res = oracle_iteration(w)
    plan, pools, r = res["plan"], res["pools"], w.reqs
    p = oracle.make_params(w.params)
    hbm_ref = np.zeros(w.layout["n_blocks"], np.int32)
    host_ref = np.zeros(w.host_blocks, np.int32)
    x1 = np.where(res["grant"] > 0, plan["x1"], 0).astype(np.int32)
    dr = oracle.dedup(r["n0"], None, x1, None, pools.host_tbl, pools.hbm_tbl, plan["restore_src"], plan["restore_dst"],
                      len(plan["restore_src"]), w.host_blocks, w.layout["n_blocks"], pools.hbm_free,
                      pools.hbm_free_count, hbm_ref)
    pools.hbm_free_count = dr["free_count"]
    st = oracle.stage_plan(p, r, res["budget"], res["order"], plan["action"], w.D_act, w.K_act, link_budget, reserve,
                           pools, w.deep_tbl, len(w.host_free) if stage_cap is None else stage_cap)
    ds = oracle.dedup(r["n0"], r["n1"], st["staged"], None, w.deep_tbl, pools.host_tbl, st["stage_src"], st["stage_dst"],
                      len(st["stage_src"]), w.deep_blocks, w.host_blocks, pools.host_free, pools.host_free_count,
                      host_ref)
    pools.host_free_count = ds["free_count"]
    return res, dr, st, ds, hbm_ref, host_ref


def make_instance(w, pools=True):
    from paper_2608_06557_b200.runner import Instance
    inst = Instance(w, alloc_pools=pools)
    inst.enable_deep(w, alloc_pool=pools)
    return inst


@pytest.mark.parametrize("seed,plan_first,link_budget,reserve,host_free_target", [
    (0, 0, 10**9, 0, 1 << 30), (0, 1, 10**9, 0, 1 << 30), (1, 1, 3_000_000, 0, 1 << 30), (2, 1, 10**9, 250, 300),
    (3, 0, 0, 0, 1 << 30), (4, 1, 10**9, 0, 40), (5, 1, 150_000, 0, 1 << 30),
])
def test_plan_steps_match_the_oracle(seed, plan_first, link_budget, reserve, host_free_target):
    import torch
    w = wl.config_deep_shared(seed, n=256, host_free_target=host_free_target)
    w.params["plan_first"] = plan_first
    res, dr, st, ds, hbm_ref, host_ref = oracle_deep(w, link_budget, reserve)
    inst = make_instance(w, pools=False)
    inst.run_schedule()
    inst.run_dedup_restore()
    inst.run_stage_plan(link_budget, reserve)
    inst.run_dedup_stage()
    got, deep = inst.fetch(), inst.fetch_deep()
    pools = res["pools"]
    # the plan itself (already covered elsewhere) must agree before anything else can
    assert np.array_equal(got["order"], res["order"]) and np.array_equal(got["grant"], res["grant"])
    assert np.array_equal(got["restore_src"], res["plan"]["restore_src"])
    # stage plan
    assert np.array_equal(deep["staged"], st["staged"])
    assert deep["stage_counts"] == st["counts"]
    assert np.array_equal(deep["stage_src"], st["stage_src"]) and np.array_equal(deep["stage_dst"], st["stage_dst"])
    # merged lists, counts, share counts, flags
    assert deep["dedup_restore"] == dr["counts"] and deep["dedup_stage"] == ds["counts"]
    assert np.array_equal(deep["restore_src_m"], dr["out_src"]) and np.array_equal(deep["restore_dst_m"], dr["out_dst"])
    assert np.array_equal(deep["stage_src_m"], ds["out_src"]) and np.array_equal(deep["stage_dst_m"], ds["out_dst"])
    assert np.array_equal(deep["hbm_ref"], hbm_ref) and np.array_equal(deep["host_ref"], host_ref)
    assert np.array_equal(deep["shared_restore"], dr["shared"]) and np.array_equal(deep["shared_stage"], ds["shared"])
    # tables and free lists
    assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl) and np.array_equal(got["host_tbl"], pools.host_tbl)
    assert got["hbm_free_count"] == pools.hbm_free_count and got["host_free_count"] == pools.host_free_count
    assert np.array_equal(got["hbm_free"][: pools.hbm_free_count], pools.hbm_free[: pools.hbm_free_count])
    assert np.array_equal(got["host_free"][: pools.host_free_count], pools.host_free[: pools.host_free_count])
    assert got["status"] == (res["status"] | dr["status"] | st["status"] | ds["status"])
    if seed == 0:
        assert st["counts"]["n_stage"] > 0 and ds["counts"]["n_surplus"] > 0
    del inst
    torch.cuda.empty_cache()


def test_whole_deep_iteration_moves_the_right_bytes():
    """Plan, merge, stage and all three copies on the GPU; pools compared byte for byte with the oracle's."""
    import torch
    w = wl.config_deep_shared(7, n=256, hbm_free_target=300)
    w.params["plan_first"] = 1
    w.params["ttft_ns"] = [40 * wl.S, 80 * wl.S]
    bb = w.block_bytes
    rng = np.random.default_rng(1)
    hbm = rng.integers(0, 256, w.layout["n_blocks"] * bb, dtype=np.uint8)
    host = rng.integers(0, 256, w.host_blocks * bb, dtype=np.uint8)
    deep = rng.integers(0, 256, w.deep_blocks * bb, dtype=np.uint8)
    res, dr, st, ds, _, _ = oracle_deep(w, 10**9, 0)
    plan = res["plan"]
    assert dr["counts"]["n_unique"] > 0 and ds["counts"]["n_unique"] > 0
    ref_hbm, ref_host = hbm.copy(), host.copy()
    assert oracle.kv_evict(ref_hbm, w.layout, ref_host, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
    assert oracle.kv_restore(ref_hbm, w.layout, ref_host, w.host_blocks, dr["out_src"], dr["out_dst"]) == 0
    assert oracle.kv_stage(deep, w.deep_blocks, ref_host, w.host_blocks, bb, ds["out_src"], ds["out_dst"]) == 0
    inst = make_instance(w)
    inst.hbm_pool.copy_(torch.from_numpy(hbm))
    inst.host_pool.copy_(torch.from_numpy(host))
    inst.deep_pool.copy_(torch.from_numpy(deep))
    torch.cuda.synchronize()
    inst.run_iteration_deep(10**9, 0)
    got = inst.fetch()
    assert got["status"] == 0
    assert np.array_equal(inst.hbm_pool.cpu().numpy(), ref_hbm)
    assert np.array_equal(inst.host_pool.numpy(), ref_host)
    assert np.array_equal(inst.deep_pool.numpy(), deep)


@pytest.mark.parametrize("n_chunks,chunk_bytes,n", [(1, 16, 5), (4, 4096, 40), (64, 32768, 24), (3, 32768 + 48, 9)])
def test_stage_copy_matches_the_oracle(n_chunks, chunk_bytes, n):
    import torch
    from paper_2608_06557_b200 import cascade as cs
    rng = np.random.default_rng(n)
    bb = n_chunks * chunk_bytes
    n_deep, n_host = 3 * n + 5, 2 * n + 3
    deep = rng.integers(0, 256, n_deep * bb, dtype=np.uint8)
    host = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
    src = rng.permutation(n_deep)[:n].astype(np.int32)
    dst = rng.permutation(n_host)[:n].astype(np.int32)
    src[0], dst[1] = n_deep, -1                       # skipped and flagged on both sides
    ref = host.copy()
    st = oracle.kv_stage(deep, n_deep, ref, n_host, bb, src, dst)
    ctx = cs.Context(wl.default_params(), 16, 0)
    d_deep = torch.from_numpy(deep).pin_memory()
    d_host = torch.from_numpy(host).pin_memory()
    cnt = torch.tensor([n], dtype=torch.int32, device="cuda")
    ctx.kv_stage(d_deep, n_deep, d_host, n_host, bb, torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), cnt,
                 n + 7)
    torch.cuda.synchronize()
    assert np.array_equal(d_host.numpy(), ref)
    assert ctx.status()[0] == st == oracle.ST_EBOUNDS


def _gpu_dedup(ctx, lo, ln, src_tbl, dst_tbl, ls, ld, count, n_src, n_dst, free, nf, scratch=None, cap=None):
    import torch
    from paper_2608_06557_b200 import cascade as cs
    cap = len(ls) if cap is None else cap
    t = lambda a, dt=np.int32: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).cuda()
    n = len(lo)
    pad = lambda a: np.concatenate([np.asarray(a, np.int32), np.full(max(cap - len(a), 0) + 1, -7, np.int32)])
    T = dict(lo=t(lo), ln=t(ln), src_tbl=t(src_tbl), dst_tbl=t(dst_tbl), ls=t(pad(ls)), ld=t(pad(ld)),
             cnt=t([count]), os=t(np.full(cap + 1, -1)), od=t(np.full(cap + 1, -1)), free=t(free), fc=t([nf]),
             ref=t(np.zeros(n_dst)), shared=t(np.zeros(n + 1), np.uint8), counts=t(np.zeros(6)))
    if scratch is None:
        scratch = torch.randint(-5, 1 << 20, (cs.dedup_scratch_len(n_src, cap),), dtype=torch.int32, device="cuda")
    args = cs.make_dedup_args(lo_a=T["lo"], lo_b=None, len_a=T["ln"], len_b=None, src_tbl=T["src_tbl"],
                              dst_tbl=T["dst_tbl"], maxb=src_tbl.shape[1], list_src=T["ls"], list_dst=T["ld"],
                              list_count=T["cnt"], list_cap=cap, out_src=T["os"], out_dst=T["od"], n_src_ids=n_src,
                              n_dst_ids=n_dst, free_list=T["free"], free_count=T["fc"], free_cap=len(free),
                              ref=T["ref"], shared=T["shared"], scratch=scratch, scratch_len=scratch.numel(),
                              counts=T["counts"])
    ctx.dedup(args, n)
    torch.cuda.synchronize()
    counts = dict(zip(DD_NAMES, (int(v) for v in T["counts"].cpu().numpy())))
    nu = counts["n_unique"]
    return dict(out_src=T["os"].cpu().numpy()[:nu], out_dst=T["od"].cpu().numpy()[:nu], dst_tbl=T["dst_tbl"].cpu().numpy(),
                free=T["free"].cpu().numpy(), free_count=int(T["fc"].item()), ref=T["ref"].cpu().numpy(),
                shared=T["shared"].cpu().numpy()[:n], counts=counts, scratch=scratch,
                tail=(int(T["os"][cap].item()), int(T["od"][cap].item())))


def _random_case(rng, n, maxb, n_src, n_dst, hot_frac):
    lo = rng.integers(0, 6, n).astype(np.int32)
    ln = rng.integers(0, maxb - 6, n).astype(np.int32)
    src_tbl = np.full((n, maxb), -1, np.int32)
    dst_tbl = np.full((n, maxb), -1, np.int32)
    total = int(ln.sum())
    assert total + 10 < n_dst
    dst_ids = rng.permutation(n_dst).astype(np.int32)
    hot = rng.permutation(n_src)[: max(4, n_src // 50)]
    ls = np.where(rng.uniform(0, 1, total) < hot_frac, rng.choice(hot, total), rng.integers(0, n_src, total)).astype(np.int32)
    ld = dst_ids[:total].copy()
    k = 0
    for r in rng.permutation(n):
        src_tbl[r, lo[r]:lo[r] + ln[r]] = ls[k:k + ln[r]]
        dst_tbl[r, lo[r]:lo[r] + ln[r]] = ld[k:k + ln[r]]
        k += ln[r]
    # the list is the concatenation in that same slot order
    free = np.full(n_dst, -1, np.int32)
    nf = n_dst - total
    free[:nf] = dst_ids[total:]
    return lo, ln, src_tbl, dst_tbl, ls, ld, free, nf


@pytest.mark.parametrize("n,maxb,n_src,n_dst,hot_frac", [
    (40, 24, 300, 2000, 0.5), (700, 40, 20000, 40000, 0.3), (2000, 30, 5000, 70000, 0.7), (3, 5000, 100, 20000, 0.9),
])
def test_dedup_random_lists_match_the_oracle(n, maxb, n_src, n_dst, hot_frac):
    from paper_2608_06557_b200 import cascade as cs
    rng = np.random.default_rng(n)
    import torch
    ctx = cs.Context(wl.default_params(), 16, 0)
    # one scratch for all trials, reused as the previous trial left it: stale entries must not matter
    scratch = torch.randint(-5, 1 << 20, (cs.dedup_scratch_len(n_src, n * maxb),), dtype=torch.int32, device="cuda")
    for trial in range(3):
        lo, ln, src_tbl, dst_tbl, ls, ld, free, nf = _random_case(rng, n, maxb, n_src, n_dst, hot_frac)
        ref_tbl, ref_free, ref = dst_tbl.copy(), free.copy(), np.zeros(n_dst, np.int32)
        want = oracle.dedup(lo, None, ln, None, src_tbl, ref_tbl, ls, ld, len(ls), n_src, n_dst, ref_free, nf, ref)
        got = _gpu_dedup(ctx, lo, ln, src_tbl, dst_tbl, ls, ld, len(ls), n_src, n_dst, free, nf, scratch)
        assert got["counts"] == want["counts"]
        assert np.array_equal(got["out_src"], want["out_src"]) and np.array_equal(got["out_dst"], want["out_dst"])
        assert np.array_equal(got["dst_tbl"], ref_tbl) and np.array_equal(got["ref"], ref)
        assert got["free_count"] == want["free_count"]
        assert np.array_equal(got["free"][: got["free_count"]], ref_free[: got["free_count"]])
        assert np.array_equal(got["shared"], want["shared"])
        assert got["tail"] == (-1, -1)
        assert ctx.status()[0] == want["status"] == 0


def test_dedup_edges():
    """Empty list, a list of one source, ids outside their pools, a count above the capacity, a negative count,
    a slot whose range leaves its row, a free list that is too short, and cells naming ids that are not in
    the list while the scratch still holds an earlier list's entries for them."""
    from paper_2608_06557_b200 import cascade as cs
    ctx = cs.Context(wl.default_params(), 16, 0)
    tbl = lambda rows, maxb: (np.full((rows, maxb), -1, np.int32), np.full((rows, maxb), -1, np.int32))

    def both(lo, ln, s_tbl, d_tbl, ls, ld, count, n_src, n_dst, free, nf, scratch=None, cap=None):
        ref_tbl, ref_free, ref = d_tbl.copy(), free.copy(), np.zeros(n_dst, np.int32)
        cap_ = len(ls) if cap is None else cap
        want = oracle.dedup(lo, None, ln, None, s_tbl, ref_tbl, np.asarray(ls, np.int32)[:cap_] if cap_ else np.zeros(1, np.int32),
                            np.asarray(ld, np.int32)[:cap_] if cap_ else np.zeros(1, np.int32), count, n_src, n_dst,
                            ref_free, nf, ref) if cap_ else None
        got = _gpu_dedup(ctx, lo, ln, s_tbl, d_tbl, ls, ld, count, n_src, n_dst, free, nf, scratch, cap)
        st = ctx.status()[0]
        if want is not None:
            assert got["counts"] == want["counts"], (got["counts"], want["counts"])
            assert np.array_equal(got["out_src"], want["out_src"]) and np.array_equal(got["out_dst"], want["out_dst"])
            assert np.array_equal(got["dst_tbl"], ref_tbl) and np.array_equal(got["ref"], ref)
            assert got["free_count"] == want["free_count"]
            k = min(got["free_count"], len(free))
            assert np.array_equal(got["free"][:k], ref_free[:k])
            assert np.array_equal(got["shared"], want["shared"])
            assert st == want["status"], (st, want["status"])
        return got, st

    s_tbl, d_tbl = tbl(2, 8)
    free = np.full(16, -1, np.int32)
    # empty list (count 0 with room for four entries)
    got, st = both([0, 0], [0, 0], s_tbl, d_tbl, [0, 0, 0, 0], [0, 0, 0, 0], 0, 8, 8, free, 0)
    assert got["counts"]["n_in"] == 0 and got["counts"]["n_unique"] == 0 and st == 0
    # one source everywhere, spanning three tiles
    m = 2500
    s_tbl, d_tbl = tbl(m, 2)
    s_tbl[:, 0], d_tbl[:, 0] = 3, np.arange(m)
    free = np.full(m + 4, -1, np.int32)
    got, st = both(np.zeros(m), np.ones(m), s_tbl, d_tbl, np.full(m, 3), np.arange(m), m, 8, m, free, 0)
    assert got["counts"]["n_unique"] == 1 and got["counts"]["max_share"] == m and got["shared"].all() and st == 0
    # ids outside their pools are passed through and flagged
    s_tbl, d_tbl = tbl(1, 4)
    got, st = both([0], [0], s_tbl, d_tbl, [2, 99, 2, -1, 2], [5, 6, 7, 8, 500], 5, 16, 16, np.full(8, -1, np.int32), 0)
    assert st == cs.ST_EBOUNDS and got["out_dst"].tolist() == [5, 6, 8, 500]
    # a count above the capacity means the capacity; a negative count is an empty list and flagged
    s_tbl, d_tbl = tbl(1, 4)
    got, st = both([0], [0], s_tbl, d_tbl, [1, 1, 2, 2], [4, 5, 6, 7], 9, 16, 16, np.full(8, -1, np.int32), 0)
    assert got["counts"]["n_in"] == 4 and st == 0
    got, st = both([0], [0], s_tbl, d_tbl, [1, 1, 2, 2], [4, 5, 6, 7], -3, 16, 16, np.full(8, -1, np.int32), 0)
    assert got["counts"]["n_in"] == 0 and st == cs.ST_EBOUNDS
    # a range that leaves the row is skipped and flagged; the rest is done
    s_tbl, d_tbl = tbl(2, 4)
    s_tbl[0, :2], d_tbl[0, :2] = [1, 2], [4, 5]
    s_tbl[1, 2:], d_tbl[1, 2:] = [1, 2], [6, 7]
    got, st = both([0, 2], [2, 3], s_tbl, d_tbl, [1, 2, 1, 2], [4, 5, 6, 7], 4, 16, 16, np.full(8, -1, np.int32), 0)
    assert st == cs.ST_EPRECOND and got["dst_tbl"][1, 2:].tolist() == [6, 7] and got["shared"].tolist() == [1, 0]
    # the free list cannot take every surplus id: the rest is dropped and flagged, the count still advances
    s_tbl, d_tbl = tbl(1, 4)
    got, st = both([0], [0], s_tbl, d_tbl, [1, 1, 1, 1], [4, 5, 6, 7], 4, 16, 16, np.array([9, -1], np.int32), 1)
    assert st == cs.ST_EBOUNDS and got["free"].tolist() == [9, 5] and got["free_count"] == 4
    # stale scratch: the first list holds source 3 at position 1; the second list does not hold 3 at all but
    # a table cell still names it and position 1 of the second list is some other source
    s_tbl, d_tbl = tbl(1, 4)
    s_tbl[0, :3], d_tbl[0, :3] = [3, 5, 5], [10, 11, 12]
    first, _ = both([0], [0], s_tbl, d_tbl, [7, 3, 3], [1, 2, 3], 3, 16, 16, np.full(8, -1, np.int32), 0)
    got, st = both([0], [3], s_tbl, d_tbl, [5, 6, 5], [11, 13, 12], 3, 16, 16, np.full(8, -1, np.int32), 0,
                   scratch=first["scratch"])
    assert got["dst_tbl"][0, :3].tolist() == [10, 11, 11] and st == 0


def test_entry_points_reject_bad_arguments():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    ctx = cs.Context(wl.default_params(), 16, 0)
    z = torch.zeros(64, dtype=torch.int32, device="cuda")
    base = dict(lo_a=z, lo_b=None, len_a=z, len_b=None, src_tbl=z, dst_tbl=z, maxb=4, list_src=z, list_dst=z[8:],
                list_count=z, list_cap=4, out_src=z[16:], out_dst=z[24:], n_src_ids=4, n_dst_ids=4, free_list=z,
                free_count=z, free_cap=4, ref=z, shared=z, scratch=z, scratch_len=64, counts=z)
    for bad in (dict(scratch_len=8), dict(out_src=z), dict(list_count=None), dict(scratch=None), dict(list_cap=-1)):
        with pytest.raises(cs.CascadeError):
            ctx.dedup(cs.make_dedup_args(**dict(base, **bad)), 1)
    with pytest.raises(cs.CascadeError):
        ctx.kv_stage(z, 4, z, 4, 24, z, z, None, 2)       # record size not a multiple of 16
    pools = cs.Pools(None, None, 0, None, None, 0, None, cs._p(z), 0)
    stage = cs.Stage(None, None, None, 0, cs._p(z), cs._p(z))
    reqs = cs.make_reqs({k: z for k, _ in cs.Reqs._fields_})
    with pytest.raises(cs.CascadeError):
        ctx.stage_plan(reqs, z, z, z, 1, 0, 0, -1, 0, pools, stage)          # negative link budget
    with pytest.raises(cs.CascadeError):
        ctx.stage_plan(reqs, z, z, z, 17, 0, 0, 0, 0, pools, stage)          # more requests than the context holds
    assert ctx.status()[0] == 0


def test_two_iterations_staged_blocks_reach_hbm_through_the_ordinary_restore():
    """Iteration 1 stages deep blocks (plan-first admission keeps those requests queued); the caller folds
    `staged` into the hit profile; iteration 2, over the requests that stayed queued, restores them.  Both
    iterations run on the GPU and on the oracle; plans and pools must agree, and the HBM block of every
    staged cell that iteration 2 restored must hold the bytes of the deep record the cell named at the start."""
    import torch
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_deep_shared(11, n=256, hbm_free_target=1500)
    w.params["plan_first"] = 1
    bb = w.block_bytes
    rng = np.random.default_rng(4)
    hbm = rng.integers(0, 256, w.layout["n_blocks"] * bb, dtype=np.uint8)
    host = rng.integers(0, 256, w.host_blocks * bb, dtype=np.uint8)
    deep = rng.integers(0, 256, w.deep_blocks * bb, dtype=np.uint8)

    def oracle_side(w, ref_hbm, ref_host):
        res, dr, st, ds, _, _ = oracle_deep(w, 10**9, 0)
        plan = res["plan"]
        assert oracle.kv_evict(ref_hbm, w.layout, ref_host, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
        assert oracle.kv_restore(ref_hbm, w.layout, ref_host, w.host_blocks, dr["out_src"], dr["out_dst"]) == 0
        assert oracle.kv_stage(deep, w.deep_blocks, ref_host, w.host_blocks, bb, ds["out_src"], ds["out_dst"]) == 0
        return res, dr, st, ds

    def gpu_side(w, pools):
        inst = Instance(w, hbm_pool=pools[0], host_pool=pools[1])
        inst.enable_deep(w, deep_pool=pools[2])
        inst.run_iteration_deep(10**9, 0)
        return inst, inst.fetch(), inst.fetch_deep()

    ref_hbm, ref_host = hbm.copy(), host.copy()
    pools = (torch.from_numpy(hbm).cuda(), torch.from_numpy(host).pin_memory(), torch.from_numpy(deep).pin_memory())
    res1, dr1, st1, ds1 = oracle_side(w, ref_hbm, ref_host)
    inst1, got1, deep1 = gpu_side(w, pools)
    assert got1["status"] == 0 and np.array_equal(deep1["staged"], st1["staged"]) and st1["counts"]["n_stage"] > 50
    assert np.array_equal(pools[0].cpu().numpy(), ref_hbm) and np.array_equal(pools[1].numpy(), ref_host)

    # fold: the requests that stayed queued and were not preempted go on, with their staged blocks now on host
    p1 = res1["pools"]
    keep = np.nonzero((res1["grant"] <= 0) & (res1["plan"]["action"] <= oracle.ACT_RETAIN))[0]
    staged = st1["staged"][keep]
    reqs2 = {k: np.ascontiguousarray(v[keep]) for k, v in w.reqs.items()}
    reqs2["n1"] = (reqs2["n1"] + staged).astype(np.int32)
    reqs2["n2"] = (reqs2["n2"] - staged).astype(np.int32)
    shared = (dr1["shared"][keep] | ds1["shared"][keep]).astype(bool)
    reqs2["flags"] = np.where(shared, reqs2["flags"] & ~np.uint8(wl.FLAG_HBM_PRIVATE), reqs2["flags"]).astype(np.uint8)
    params2 = dict(w.params, ttft_ns=[500 * wl.S, 500 * wl.S], token_budget=1 << 20, max_batch=4096)
    w2 = wl.Workload("second", params2, reqs2, w.now_ns + 10 * wl.MS, w.D_act, w.K_act, w.layout, w.host_blocks, w.maxb,
                     p1.hbm_tbl[keep].copy(), p1.host_tbl[keep].copy(), p1.hbm_free.copy(), p1.hbm_free_count,
                     p1.host_free.copy(), p1.host_free_count)
    w2.deep_tbl, w2.deep_blocks = w.deep_tbl[keep].copy(), w.deep_blocks
    res2, dr2, st2, ds2 = oracle_side(w2, ref_hbm, ref_host)
    inst2, got2, deep2 = gpu_side(w2, pools)
    assert got2["status"] == res2["status"] | dr2["status"] | st2["status"] | ds2["status"]
    assert np.array_equal(got2["grant"], res2["grant"]) and np.array_equal(got2["x1"], res2["plan"]["x1"])
    assert np.array_equal(deep2["restore_src_m"], dr2["out_src"]) and np.array_equal(deep2["restore_dst_m"], dr2["out_dst"])
    assert np.array_equal(got2["hbm_tbl"], res2["pools"].hbm_tbl)
    assert np.array_equal(pools[0].cpu().numpy(), ref_hbm) and np.array_equal(pools[1].numpy(), ref_host)
    # content: staged cells that iteration 2 restored hold the deep record's bytes
    lay, out_hbm, checked = w.layout, pools[0].cpu().numpy(), 0
    for s in range(len(keep)):
        if res2["grant"][s] <= 0 or staged[s] == 0:
            continue
        lo = int(w.reqs["n0"][keep[s]] + w.reqs["n1"][keep[s]])
        upto = int(reqs2["n0"][s] + res2["plan"]["x1"][s])
        for j in range(lo, min(lo + int(staged[s]), upto)):
            g, dr = int(got2["hbm_tbl"][s, j]), int(w2.deep_tbl[s, j])
            for c in range(lay["n_chunks"]):
                a = c * lay["chunk_stride"] + g * lay["block_stride"]
                b = dr * bb + c * lay["chunk_bytes"]
                assert np.array_equal(out_hbm[a:a + lay["chunk_bytes"]], deep[b:b + lay["chunk_bytes"]]), (s, j, c)
            checked += 1
    assert checked > 50


@pytest.mark.parametrize("seed,plan_first", [(0, 1), (3, 0), (6, 1)])
def test_merge_after_the_prefetch_plan(seed, plan_first):
    """Restore list = the admitted set's blocks followed by the prefetched ones; the merge pass then covers the
    cells [n0, n0 + x1 + prefetched) of every slot (two length arrays)."""
    w = wl.config_deep_shared(seed, n=256)
    w.params["plan_first"] = plan_first
    res = oracle_iteration(w)
    plan, pools, r = res["plan"], res["pools"], w.reqs
    p = oracle.make_params(w.params)
    pf = oracle.prefetch_plan(p, r, res["budget"], res["order"], res["grant"], plan["action"], plan["x1"], w.D_act,
                              w.K_act, 10**9, 4, pools, plan["restore_src"], plan["restore_dst"])
    assert pf["counts"]["n_prefetch"] > 0
    ref = np.zeros(w.layout["n_blocks"], np.int32)
    x1 = np.where(res["grant"] > 0, plan["x1"], 0).astype(np.int32)
    dr = oracle.dedup(r["n0"], None, x1, pf["pf"], pools.host_tbl, pools.hbm_tbl, pf["restore_src"], pf["restore_dst"],
                      len(pf["restore_src"]), w.host_blocks, w.layout["n_blocks"], pools.hbm_free, pools.hbm_free_count,
                      ref)
    assert dr["counts"]["n_surplus"] > 0
    inst = make_instance(w, pools=False)
    inst.run_schedule()
    inst.run_prefetch(10**9, 4)
    inst.run_dedup_restore()
    got, gp, deep = inst.fetch(), inst.fetch_prefetch(), inst.fetch_deep()
    assert np.array_equal(gp["pf"], pf["pf"]) and gp["counts"] == pf["counts"]
    assert deep["dedup_restore"] == dr["counts"]
    assert np.array_equal(deep["restore_src_m"], dr["out_src"]) and np.array_equal(deep["restore_dst_m"], dr["out_dst"])
    assert np.array_equal(deep["hbm_ref"], ref) and np.array_equal(deep["shared_restore"], dr["shared"])
    assert np.array_equal(got["hbm_tbl"], pools.hbm_tbl)
    assert got["hbm_free_count"] == dr["free_count"]
    assert np.array_equal(got["hbm_free"][: dr["free_count"]], pools.hbm_free[: dr["free_count"]])
    assert got["status"] == res["status"] | pf["status"] | dr["status"]


@pytest.mark.parametrize("n", [3000, 20000])
def test_plan_steps_on_large_queues(n):
    """Several keys per thread and the full cluster: the same comparison as above on 3 000 and 20 000 requests."""
    import torch
    w = wl.config_deep_shared(1, n=n, n_hbm=16 * n, n_host=16 * n, n_deep=32 * n, hbm_free_target=8 * n)
    w.params["plan_first"] = 1
    res, dr, st, ds, hbm_ref, host_ref = oracle_deep(w, 10**9, 100)
    assert st["counts"]["n_stage"] > n and ds["counts"]["n_surplus"] > 0
    inst = make_instance(w, pools=False)
    inst.run_schedule()
    inst.run_dedup_restore()
    inst.run_stage_plan(10**9, 100)
    inst.run_dedup_stage()
    got, deep = inst.fetch(), inst.fetch_deep()
    pools = res["pools"]
    assert np.array_equal(deep["staged"], st["staged"]) and deep["stage_counts"] == st["counts"]
    assert np.array_equal(deep["stage_src"], st["stage_src"]) and np.array_equal(deep["stage_dst"], st["stage_dst"])
    assert deep["dedup_restore"] == dr["counts"] and deep["dedup_stage"] == ds["counts"]
    assert np.array_equal(deep["stage_src_m"], ds["out_src"]) and np.array_equal(deep["stage_dst_m"], ds["out_dst"])
    assert np.array_equal(deep["host_ref"], host_ref) and np.array_equal(deep["shared_stage"], ds["shared"])
    assert np.array_equal(got["host_tbl"], pools.host_tbl) and np.array_equal(got["hbm_tbl"], pools.hbm_tbl)
    assert got["host_free_count"] == pools.host_free_count
    assert np.array_equal(got["host_free"][: pools.host_free_count], pools.host_free[: pools.host_free_count])
    assert got["status"] == (res["status"] | dr["status"] | st["status"] | ds["status"])
    del inst
    torch.cuda.empty_cache()
