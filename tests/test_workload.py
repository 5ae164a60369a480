"""The synthetic generators are deterministic and respect the input bounds of the path."""
import numpy as np

from paper_2608_06557_b200 import workload as wl


def check_bounds(w):
    r = w.reqs
    bt = w.params["bt"]
    hit = r["n0"].astype(np.int64) + r["n1"] + r["n2"]
    assert np.all(hit * bt < r["prompt"])
    assert np.all(r["prompt"] >= 1) and np.all(r["prompt"] <= 1 << 17)
    assert np.all(r["cls"] < len(w.params["ttft_ns"]))
    assert len(np.unique(r["id"] & 0x7FFFFF)) == w.n


def test_tiny_is_deterministic_and_consistent():
    a, b = wl.config_tiny(0), wl.config_tiny(0)
    for k in a.reqs:
        assert np.array_equal(a.reqs[k], b.reqs[k])
    assert np.array_equal(a.hbm_tbl, b.hbm_tbl) and np.array_equal(a.host_free, b.host_free)
    check_bounds(a)
    assert a.n == 64 and a.block_bytes == 16384 and a.hbm_free_count == 32
    # table rows agree with the hit profile
    for r in range(a.n):
        n0, n1 = a.reqs["n0"][r], a.reqs["n1"][r]
        assert np.all(a.hbm_tbl[r, :n0] >= 0) and np.all(a.hbm_tbl[r, n0:] == -1)
        assert np.all(a.host_tbl[r, n0:n0 + n1] >= 0)
    used = a.hbm_tbl[a.hbm_tbl >= 0]
    free = a.hbm_free[: a.hbm_free_count]
    assert len(np.unique(np.concatenate([used, free]))) == len(used) + len(free)


def test_llama8b_shape():
    w = wl.config_llama8b(0, n=1024, hbm_bytes=6 * 10**9, host_bytes=4 * 10**9)
    check_bounds(w)
    assert w.block_bytes == 2 * 1024 * 1024 and w.layout["n_chunks"] == 64
    assert 700 < np.median(w.reqs["prompt"]) < 1500
    assert w.reqs["prompt"].max() > 8000
    assert set(np.unique(w.reqs["cls"]).tolist()) == {0, 1, 2}


def test_sweep_churn_keeps_ids_unique():
    sw = wl.SchedulerSweep(1024, seed=3)
    for _ in range(20):
        slots = sw.step()
        assert len(slots) == 51
        check_bounds(sw.workload())
    assert sw.D_act == 256 and sw.K_act > 0
