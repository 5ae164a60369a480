"""Toy closed-loop comparison of the ordering policies on synthetic traffic, run on the GPU library.

    python -m paper_2608_06557_b200.policy_demo [iterations] [requests/s]

Replays a seeded Llama-3-70B-shaped arrival trace through budget -> schedule -> tier plan (the KV
copies are skipped: no pools are allocated, only tables and free lists) under the method's own
ordering and under FCFS, EDF and SJF, and prints TTFT violation rates and the fairness index over
input-length bins.  The clock is the replay's simple service-time rule, the traffic is synthetic:
the numbers illustrate the policies and are NOT comparable with the paper's trace results.
"""
from __future__ import annotations

import json
import sys

from . import cascade as cs
from . import workload as wl
from .replay import Replay, slo_report
from .runner import Instance

NAMES = {cs.POLICY_BUDGET: "cascade", cs.POLICY_FCFS: "fcfs", cs.POLICY_EDF: "edf", cs.POLICY_SJF: "sjf"}


def run(policy: int, iterations: int, rate: float, seed: int = 2, n: int = 2048) -> dict:
    tr = wl.config_llama70b_trace(seed, n=n, hbm_bytes=24 * 10**9, host_bytes=16 * 10**9, hbm_occupancy=0.6,
                                  rate_per_s=rate)
    tr.params = dict(tr.params, policy=policy)
    rp = Replay(tr)
    ctx = cs.Context(tr.params, n, 0)
    for _ in range(iterations):
        w, ids = rp.workload()
        if len(ids) == 0:
            break
        inst = Instance(w, ctx=ctx, alloc_pools=False)
        inst.run_schedule()
        got = inst.fetch()
        rp.apply(ids, dict(grant=got["grant"], x1=got["x1"], tokens_run=got["tokens_run"], action=got["action"],
                           hbm_tbl=got["hbm_tbl"], host_tbl=got["host_tbl"], hbm_free=got["hbm_free"],
                           host_free=got["host_free"], hbm_free_count=got["hbm_free_count"],
                           host_free_count=got["host_free_count"]))
    rep = slo_report(rp)
    rep.update(policy=NAMES[policy], iterations=rp.iteration, virtual_seconds=round(rp.now / 1e9, 2), **rp.stats)
    return rep


def main(argv):
    iterations = int(argv[1]) if len(argv) > 1 else 300
    rate = float(argv[2]) if len(argv) > 2 else 15.0
    for policy in (cs.POLICY_BUDGET, cs.POLICY_FCFS, cs.POLICY_EDF, cs.POLICY_SJF):
        print(json.dumps(run(policy, iterations, rate)))


if __name__ == "__main__":
    main(sys.argv)
