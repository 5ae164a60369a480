"""Host-side bookkeeping of the closed-loop replay: fairness index and SLO report."""
import numpy as np

from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl
from paper_2608_06557_b200.replay import Replay, jain_index, slo_report


def test_jain_index_closed_forms():
    assert jain_index([5, 5, 5, 5]) == 1.0
    assert abs(jain_index([1, 0, 0, 0]) - 0.25) < 1e-12
    assert abs(jain_index([1, 1, 0, 0]) - 0.5) < 1e-12
    assert jain_index([]) == 1.0 and jain_index([0, 0]) == 1.0
    assert abs(jain_index([1, 2, 3]) - 36 / (3 * 14)) < 1e-12


def test_replay_conserves_block_ids_and_reports():
    tr = wl.config_llama70b_trace(1, n=512, hbm_bytes=12 * 10**9, host_bytes=8 * 10**9, hbm_occupancy=0.7,
                                  rate_per_s=60.0)
    rp = Replay(tr)
    for _ in range(120):
        w, ids = rp.workload()
        if len(ids) == 0:
            break
        res = oracle_iteration(w)
        plan, pools = res["plan"], res["pools"]
        rp.apply(ids, dict(grant=res["grant"], x1=plan["x1"], tokens_run=plan["tokens_run"], action=plan["action"],
                           hbm_tbl=pools.hbm_tbl, host_tbl=pools.host_tbl, hbm_free=pools.hbm_free,
                           host_free=pools.host_free, hbm_free_count=pools.hbm_free_count,
                           host_free_count=pools.host_free_count))
    held = np.unique(rp.hbm_tbl[rp.hbm_tbl >= 0])
    free = rp.hbm_free[: rp.hbm_free_count]
    assert len(np.intersect1d(held, free)) == 0 and len(held) + len(free) == tr.layout["n_blocks"]
    hheld = rp.host_tbl[rp.host_tbl >= 0]
    hfree = rp.host_free[: rp.host_free_count]
    assert len(np.unique(hheld)) == len(hheld) and len(np.intersect1d(hheld, hfree)) == 0
    rep = slo_report(rp)
    assert rep["finished"] == rp.stats["finished"] > 0
    assert 0.0 <= rep["violation_rate"] <= 1.0 and 0.0 < rep["jain_index"] <= 1.0
    assert 1 <= len(rep["violation_pct_by_length_bin"]) <= 6
