"""Many consecutive iterations with the deep-tier stage and the shared-block merge, state carried between
them (GPU and oracle side by side, bit exact at every step, pools compared at the end).

The bookkeeping between iterations is harness code, the same for both sides: requests join in waves, a
request that ran its last token leaves, an evicted one continues from the host tier, a dropped one starts
over, staged deep blocks become host blocks, restored ones HBM blocks.  Nothing is ever released, so the
pools only fill up: HBM pressure (preemption, capacity cuts) sets in after a few iterations."""
import numpy as np
import pytest

import oracle
from paper_2608_06557_b200 import workload as wl
from test_gpu_deep import oracle_deep

pytestmark = pytest.mark.gpu


class State:
    def __init__(self, w, wave):
        self.w, self.wave = w, wave
        r = w.reqs
        self.n = w.n
        self.n0, self.n1, self.n2 = r["n0"].copy(), r["n1"].copy(), r["n2"].copy()
        self.flags = r["flags"].copy()
        self.shared = np.zeros(self.n, bool)
        self.joined = np.zeros(self.n, bool)
        self.done = np.zeros(self.n, bool)
        self.hbm_tbl, self.host_tbl = w.hbm_tbl.copy(), w.host_tbl.copy()
        self.hbm_free, self.host_free = w.hbm_free.copy(), w.host_free.copy()
        self.hbm_free_count, self.host_free_count = w.hbm_free_count, w.host_free_count
        self.now = w.now_ns
        self.it = 0

    def workload(self):
        self.joined[self.it * self.wave:(self.it + 1) * self.wave] = True
        ids = np.nonzero(self.joined & ~self.done)[0]
        w, r = self.w, self.w.reqs
        flags = self.flags[ids].copy()
        own = (self.n0[ids] > 0) & ~self.shared[ids]
        flags[own] |= wl.FLAG_HBM_PRIVATE | wl.FLAG_RUNNING
        flags[~own] &= ~np.uint8(wl.FLAG_HBM_PRIVATE)
        reqs = dict(arrival_ns=r["arrival_ns"][ids].copy(), prompt=r["prompt"][ids].copy(),
                    pred_out=r["pred_out"][ids].copy(), n0=self.n0[ids].copy(), n1=self.n1[ids].copy(),
                    n2=self.n2[ids].copy(), id=r["id"][ids].copy(), cls=r["cls"][ids].copy(), flags=flags)
        w2 = wl.Workload(f"it{self.it}", w.params, reqs, self.now, w.D_act, w.K_act, w.layout, w.host_blocks, w.maxb,
                         self.hbm_tbl[ids].copy(), self.host_tbl[ids].copy(), self.hbm_free.copy(),
                         self.hbm_free_count, self.host_free.copy(), self.host_free_count)
        w2.deep_tbl, w2.deep_blocks = w.deep_tbl[ids].copy(), w.deep_blocks
        return w2, ids

    def fold(self, ids, res, dr, st, ds):
        pools, plan = res["pools"], res["plan"]
        bt = self.w.params["bt"]
        self.hbm_tbl[ids], self.host_tbl[ids] = pools.hbm_tbl, pools.host_tbl
        self.hbm_free[:], self.host_free[:] = pools.hbm_free, pools.host_free
        self.hbm_free_count, self.host_free_count = pools.hbm_free_count, pools.host_free_count
        self.shared[ids] |= (dr["shared"] | ds["shared"]).astype(bool)
        for s, r in enumerate(ids):
            act = int(plan["action"][s])
            staged = int(st["staged"][s])
            if act == oracle.ACT_EVICT:            # the HBM part now sits in front of the old host part
                self.n1[r] += self.n0[r]
                self.n0[r] = 0
            elif act == oracle.ACT_DROP:           # prefix lost: what was behind it cannot be used any more
                self.n0[r] = self.n1[r] = self.n2[r] = 0
            if res["grant"][s] > 0:
                x1, run = int(plan["x1"][s]), int(plan["tokens_run"][s])
                self.n0[r] += x1
                self.n1[r] -= x1
                if run > 0:
                    have = int(self.n0[r]) * bt + run
                    if have >= self.w.reqs["prompt"][r]:
                        self.done[r] = True
                    self.n0[r] = have // bt        # a partly filled block is recomputed next time
                    self.n1[r] = self.n2[r] = 0    # the rest of the match was recomputed
                    continue
            self.n1[r] += staged
            self.n2[r] -= staged
        self.now += 50 * wl.MS
        self.it += 1


@pytest.mark.parametrize("seed,plan_first,hbm_free_target", [(0, 1, 700), (1, 0, 500), (2, 1, 5000)])
def test_state_carried_over_many_deep_iterations(seed, plan_first, hbm_free_target):
    import torch
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_deep_shared(seed, n=640, n_hbm=8192, n_host=16384, n_deep=16384, hbm_free_target=hbm_free_target,
                              n_chunks=2, chunk_bytes=256)
    w.params["plan_first"] = plan_first
    w.params["ttft_ns"] = [4 * wl.S, 40 * wl.S]
    bb = w.block_bytes
    rng = np.random.default_rng(seed)
    hbm = rng.integers(0, 256, w.layout["n_blocks"] * bb, dtype=np.uint8)
    host = rng.integers(0, 256, w.host_blocks * bb, dtype=np.uint8)
    deep = rng.integers(0, 256, w.deep_blocks * bb, dtype=np.uint8)
    g_hbm, g_host, g_deep = torch.from_numpy(hbm.copy()).cuda(), torch.from_numpy(host.copy()).pin_memory(), \
        torch.from_numpy(deep).pin_memory()
    state = State(w, wave=64)
    seen = dict(evict=0, drop=0, unadmitted=0, staged=0, merged=0, restored=0, finished=0)
    ctx = None
    for it in range(24):
        w_it, ids = state.workload()
        if len(ids) == 0:
            break
        res, dr, st, ds, hbm_ref, host_ref = oracle_deep(w_it, 3_000_000, 8)
        plan = res["plan"]
        assert oracle.kv_evict(hbm, w.layout, host, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
        assert oracle.kv_restore(hbm, w.layout, host, w.host_blocks, dr["out_src"], dr["out_dst"]) == 0
        assert oracle.kv_stage(deep, w.deep_blocks, host, w.host_blocks, bb, ds["out_src"], ds["out_dst"]) == 0
        inst = Instance(w_it, hbm_pool=g_hbm, host_pool=g_host, ctx=ctx, max_requests=640)
        ctx = inst.ctx
        inst.enable_deep(w_it, deep_pool=g_deep)
        inst.run_iteration_deep(3_000_000, 8)
        got, gd = inst.fetch(), inst.fetch_deep()
        want_status = res["status"] | dr["status"] | st["status"] | ds["status"]
        assert got["status"] == want_status, (it, got["status"], want_status)
        for k in ("order", "grant"):
            assert np.array_equal(got[k], res[k]), (it, k)
        for k in ("x1", "x2", "tokens_run", "action"):
            assert np.array_equal(got[k], plan[k]), (it, k)
        assert got["plan_counts"] == plan["counts"], it
        assert np.array_equal(gd["staged"], st["staged"]) and gd["stage_counts"] == st["counts"], it
        assert gd["dedup_restore"] == dr["counts"] and gd["dedup_stage"] == ds["counts"], it
        assert np.array_equal(gd["restore_src_m"], dr["out_src"]) and np.array_equal(gd["restore_dst_m"], dr["out_dst"])
        assert np.array_equal(gd["stage_src_m"], ds["out_src"]) and np.array_equal(gd["stage_dst_m"], ds["out_dst"])
        assert np.array_equal(gd["shared_restore"], dr["shared"]) and np.array_equal(gd["shared_stage"], ds["shared"])
        p = res["pools"]
        assert np.array_equal(got["hbm_tbl"], p.hbm_tbl) and np.array_equal(got["host_tbl"], p.host_tbl), it
        assert got["hbm_free_count"] == p.hbm_free_count and got["host_free_count"] == p.host_free_count, it
        assert np.array_equal(got["hbm_free"][: p.hbm_free_count], p.hbm_free[: p.hbm_free_count]), it
        assert np.array_equal(got["host_free"][: p.host_free_count], p.host_free[: p.host_free_count]), it
        seen["evict"] += plan["counts"]["n_evict"]
        seen["drop"] += plan["counts"]["n_drop_blocks"]
        seen["unadmitted"] += plan["counts"]["n_unadmitted"]
        seen["staged"] += st["counts"]["n_stage"]
        seen["merged"] += dr["counts"]["n_surplus"] + ds["counts"]["n_surplus"]
        seen["restored"] += dr["counts"]["n_unique"]
        before = state.done.sum()
        state.fold(ids, res, dr, st, ds)
        seen["finished"] += int(state.done.sum() - before)
        del inst
    assert np.array_equal(g_hbm.cpu().numpy(), hbm)
    assert np.array_equal(g_host.numpy(), host)
    assert seen["staged"] > 500 and seen["merged"] > 20 and seen["restored"] > 100 and seen["finished"] > 40, seen
    if hbm_free_target <= 700:
        assert seen["evict"] + seen["drop"] > 0, seen
