"""Closed-loop replay of an arrival trace through the scheduling + KV-tier step (host bookkeeping only).

The step itself is a callable supplied by the user of this module (the CUDA library in production,
any other implementation in tests); this file only keeps the serving state between iterations: which
requests are queued, their hit profiles and table rows, the free lists, the decode load and a virtual
clock.  None of the method's arithmetic lives here: the clock advance uses its own, deliberately
simple service-time rule.
"""
from __future__ import annotations

import numpy as np

from .workload import FLAG_HBM_PRIVATE, FLAG_RUNNING, Workload

ACT_EVICT, ACT_DROP = 2, 3
FUTURE, QUEUED, DECODING, DONE = 0, 1, 2, 3


class Replay:
    """Serving state of one instance driven by a ``workload.Trace``."""

    def __init__(self, trace, max_active: int = 4096, decode_residency: int = 24):
        t = self.t = trace
        n = len(t.prompt)
        self.n = n
        self.now = int(t.arrival_ns[0])
        self.state = np.full(n, FUTURE, np.int8)
        self.n0 = t.n0.copy()
        self.n1 = t.n1.copy()
        self.hbm_tbl = t.hbm_tbl.copy()
        self.host_tbl = t.host_tbl.copy()
        self.hbm_free = t.hbm_free.copy()
        self.hbm_free_count = int(t.hbm_free_count)
        self.host_free = t.host_free.copy()
        self.host_free_count = int(t.host_free_count)
        self.decode_left = np.zeros(n, np.int64)
        self.generated = np.zeros(n, np.int64)
        self.iteration = 0
        self.max_active = max_active
        self.decode_residency = decode_residency   # iterations a finished prefill keeps its blocks (at most)
        self.stats = dict(restored=0, evicted=0, dropped=0, admitted=0, tokens=0, finished=0)
        self.finish_ns = np.full(n, -1, np.int64)   # virtual time at which the prefill completed

    # ---- queue view ---------------------------------------------------------------------------
    def active_ids(self) -> np.ndarray:
        self.state[(self.state == FUTURE) & (self.t.arrival_ns <= self.now)] = QUEUED
        ids = np.nonzero(self.state == QUEUED)[0]
        return ids[: self.max_active]

    def load(self):
        dec = self.state == DECODING
        return int(dec.sum()), int((self.t.prompt[dec].astype(np.int64) + self.generated[dec]).sum())

    def workload(self) -> tuple[Workload, np.ndarray]:
        """The compacted queue of this iteration as a one-iteration Workload (arrays are copies)."""
        ids = self.active_ids()
        while len(ids) == 0 and (self.state == FUTURE).any():      # idle: jump to the next arrival
            self.now = int(self.t.arrival_ns[self.state == FUTURE].min())
            ids = self.active_ids()
        t = self.t
        flags = np.zeros(len(ids), np.uint8)
        own = (self.n0[ids] > 0) & ~t.shared[ids]
        flags[own] = FLAG_HBM_PRIVATE | FLAG_RUNNING
        reqs = dict(arrival_ns=t.arrival_ns[ids].copy(), prompt=t.prompt[ids].copy(), pred_out=t.pred_out[ids].copy(),
                    n0=self.n0[ids].copy(), n1=self.n1[ids].copy(), n2=np.zeros(len(ids), np.int32),
                    id=ids.astype(np.uint32), cls=t.cls[ids].copy(), flags=flags)
        D, K = self.load()
        w = Workload(f"replay{self.iteration}", t.params, reqs, self.now, D, min(K, 1 << 32), t.layout, t.host_blocks,
                     t.maxb, self.hbm_tbl[ids].copy(), self.host_tbl[ids].copy(), self.hbm_free.copy(),
                     self.hbm_free_count, self.host_free.copy(), self.host_free_count)
        return w, ids

    # ---- state update ---------------------------------------------------------------------------
    def _release_hbm(self, ids):
        ids = ids[ids >= 0]
        self.hbm_free[self.hbm_free_count:self.hbm_free_count + len(ids)] = ids
        self.hbm_free_count += len(ids)

    def _release_host(self, ids):
        ids = ids[ids >= 0]
        self.host_free[self.host_free_count:self.host_free_count + len(ids)] = ids
        self.host_free_count += len(ids)

    def apply(self, ids, out):
        """Fold one iteration's results back into the serving state.  ``out`` holds grant, x1, tokens_run,
        action (per compacted slot), the updated table rows and the free lists with their counts."""
        t = self.t
        bt = t.params["bt"]
        self.hbm_tbl[ids] = out["hbm_tbl"]
        self.host_tbl[ids] = out["host_tbl"]
        self.hbm_free[:] = out["hbm_free"]
        self.host_free[:] = out["host_free"]
        self.hbm_free_count = int(out["hbm_free_count"])
        self.host_free_count = int(out["host_free_count"])
        tokens = 0
        x1_sum = 0
        self._just_finished = []
        for s, r in enumerate(ids):
            act = int(out["action"][s])
            if act == ACT_EVICT:                       # whole HBM part now lives on host, in front of the old host part
                self.n1[r] += self.n0[r]
                self.n0[r] = 0
                self.stats["evicted"] += 1
            elif act == ACT_DROP:                      # prefix lost: the host blocks behind it cannot be used any more
                self._release_host(self.host_tbl[r].copy())
                self.host_tbl[r] = -1
                self.n0[r] = self.n1[r] = 0
                self.stats["dropped"] += 1
            if out["grant"][s] <= 0:
                continue
            x1, run = int(out["x1"][s]), int(out["tokens_run"][s])
            have = (int(self.n0[r]) + x1) * bt + run
            tokens += run
            x1_sum += x1
            self.stats["admitted"] += 1
            self.stats["restored"] += x1
            # host copies of the matched prefix are no longer needed once the request runs
            self._release_host(self.host_tbl[r].copy())
            self.host_tbl[r] = -1
            self.n1[r] = 0
            if have >= t.prompt[r]:
                self.state[r] = DECODING
                self.decode_left[r] = min(int(t.pred_out[r]), self.decode_residency)
                self.n0[r] = -(-int(t.prompt[r]) // bt)
                self.stats["finished"] += 1
                self._just_finished.append(r)
            else:
                full = have // bt
                if have % bt:                          # a partly filled block is recomputed next time
                    self._release_hbm(self.hbm_tbl[r, full:full + 1].copy())
                    self.hbm_tbl[r, full] = -1
                self.n0[r] = full
        self.stats["tokens"] += tokens
        # decode sequences advance one token; finished ones give their own blocks back
        dec = np.nonzero(self.state == DECODING)[0]
        self.generated[dec] += 1
        self.decode_left[dec] -= 1
        for r in dec[self.decode_left[dec] <= 0]:
            row = self.hbm_tbl[r].copy()
            if t.shared[r]:
                row[: len(t.shared_ids)] = -1          # the shared prefix stays resident
            self._release_hbm(row)
            self.hbm_tbl[r] = -1
            self.state[r] = DONE
        # virtual clock: a fixed per-token service time plus the transfer time of the restored blocks
        p = t.params
        per_tok = p["c_tok_q20"] >> 20
        xfer = 0 if x1_sum == 0 else p["delta_ns"][1] + x1_sum * p["blk_ns"][1]
        self.now += max(1_000_000, tokens * per_tok + xfer)
        self.finish_ns[self._just_finished] = self.now       # first token leaves at the end of the iteration
        self.iteration += 1

    def done(self) -> bool:
        return not ((self.state == FUTURE) | (self.state == QUEUED)).any()


def jain_index(values) -> float:
    """Jain's fairness index of non-negative values: (sum v)^2 / (n * sum v^2); 1 when all are equal."""
    v = np.asarray(values, float)
    if len(v) == 0 or not np.any(v):
        return 1.0
    return float(v.sum() ** 2 / (len(v) * (v * v).sum()))


def slo_report(replay: "Replay", bins=(0, 25, 50, 75, 90, 99, 100)) -> dict:
    """TTFT outcome of the requests that have arrived: violation rate overall and per input-length
    percentile bin (a request still queued past its target counts as violated), and the fairness
    index over the bins' attainment A_i = max(0, 100 - V_i) in percent (the paper's Eq. 1)."""
    t = replay.t
    arrived = t.arrival_ns <= replay.now
    ttft = np.asarray(t.params["ttft_ns"], np.int64)[t.cls]
    done = replay.finish_ns >= 0
    lat = np.where(done, replay.finish_ns - t.arrival_ns, replay.now - t.arrival_ns)
    judged = arrived & (done | (lat > ttft))            # still waiting inside the target: not judged yet
    viol = judged & (lat > ttft)
    out = dict(arrived=int(arrived.sum()), judged=int(judged.sum()), finished=int((done & arrived).sum()),
               violation_rate=float(viol.sum() / max(judged.sum(), 1)))
    edges = np.percentile(t.prompt[judged], bins) if judged.any() else np.zeros(len(bins))
    per_bin = []
    for lo, hi in zip(edges[:-1], edges[1:]):
        m = judged & (t.prompt >= lo) & ((t.prompt < hi) | (hi == edges[-1]))
        if m.any():                                      # equal prompt lengths can leave a bin empty
            per_bin.append(100.0 * float(viol[m].sum()) / int(m.sum()))
    out["violation_pct_by_length_bin"] = [round(v, 1) for v in per_bin]
    out["jain_index"] = round(jain_index([max(0.0, 100.0 - v) for v in per_bin]), 4)
    lat_done = lat[done & arrived]
    out["ttft_p50_s"] = float(np.percentile(lat_done, 50) / 1e9) if len(lat_done) else None
    out["ttft_p95_s"] = float(np.percentile(lat_done, 95) / 1e9) if len(lat_done) else None
    return out
