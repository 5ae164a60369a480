"""Random inputs over the whole validated parameter space through the oracle's plan chain: properties that
must hold for any input (no id lost or handed out twice, every bound respected, status bits only where a
cause exists)."""
import numpy as np

import oracle
from chain import oracle_chain
from paper_2608_06557_b200 import workload as wl


def test_chain_invariants_on_random_inputs():
    seen_status = 0
    for seed in range(80):
        g = np.random.default_rng(seed)
        d = wl.fuzz_params(g)
        w = wl.fuzz_workload(g, d)
        hbm0 = set(w.hbm_free[: w.hbm_free_count].tolist())
        host0 = set(w.host_free[: w.host_free_count].tolist())
        held_hbm = w.hbm_tbl[w.hbm_tbl >= 0]
        out = oracle_chain(w, int(g.choice([0, 10**6, 1 << 50])), int(g.choice([0, 2])), int(g.choice([0, 10**9])),
                           int(g.choice([0, 2])))
        res, pools, plan = out["res"], out["res"]["pools"], out["res"]["plan"]
        status = res["status"] | out["pf"]["status"] | out["dr"]["status"] | out["st"]["status"] | out["ds"]["status"]
        seen_status |= status
        assert not status & (oracle.ST_EBOUNDS | oracle.ST_ELISTCAP), seed      # inputs are well-formed in that respect
        # order is a permutation; grants respect the token budget and the batch cap
        assert sorted(res["order"].tolist()) == list(range(w.n))
        grant = res["grant"]
        assert (grant >= 0).all() and grant.sum() <= max(0, d["token_budget"] - w.D_act)
        assert (grant > 0).sum() <= max(0, d["max_batch"] - w.D_act)
        assert (plan["tokens_run"] <= np.maximum(grant, 0)).all()
        # HBM ids: free stack + table cells hold every id at most once, nothing invented
        free_now = pools.hbm_free[: pools.hbm_free_count]
        assert len(set(free_now.tolist())) == len(free_now) and (free_now >= 0).all(), seed
        cells = np.unique(pools.hbm_tbl[pools.hbm_tbl >= 0])
        assert not set(free_now.tolist()) & set(cells.tolist()), seed
        assert set(free_now.tolist()) | set(cells.tolist()) <= hbm0 | set(held_hbm.tolist()), seed
        # host ids likewise (shared records may sit in several cells, never on the free stack as well)
        hfree = pools.host_free[: pools.host_free_count]
        assert len(set(hfree.tolist())) == len(hfree), seed
        assert not set(hfree.tolist()) & set(pools.host_tbl[pools.host_tbl >= 0].tolist()), seed
        assert set(hfree.tolist()) <= host0, seed
        # merged lists hold every source once; a kept destination is what its cells point at
        for key in ("dr", "ds"):
            o = out[key]
            assert len(np.unique(o["out_src"])) == len(o["out_src"]), (seed, key)
            assert o["counts"]["n_in"] == o["counts"]["n_unique"] + o["counts"]["n_surplus"]
        # evicted blocks left HBM, their requests hold no HBM cell any more
        ev = np.nonzero(plan["action"] == oracle.ACT_EVICT)[0]
        for r in ev:
            assert (pools.hbm_tbl[r, : w.reqs["n0"][r]] == -1).all() and (pools.host_tbl[r, : w.reqs["n0"][r]] >= 0).all()
    assert seen_status & oracle.ST_EPRECOND and seen_status & oracle.ST_ENOSPC
