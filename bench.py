#!/usr/bin/env python
"""Benchmark of the Cascade scheduling + KV-tier step on B200.

A step is one pass of the whole hot path (budget -> schedule -> tier plan -> KV evict -> KV restore)
over one batch of synthetic input in the Llama-3-8B-shaped configuration: 1024 queued requests,
2 MiB KV blocks, a 60 GB paged HBM pool and a 40 GB pinned host pool.  Every step works on a fresh
seeded batch (request arrays, block tables, free lists) that is already resident in HBM when the
timed region starts; the KV bytes a step moves cross the host link inside the copy kernels.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --case copy-hbm|copy-host|move|staged|schedule|deep [--case-n N]

Prints one JSON line.  `--case` runs one small, self-contained invocation of a single kernel family instead
(a few launches, a few GB on the device at most, more than the 126 MB L2 per launch where bandwidth is
measured): the commands behind the ncu summaries under profiles/.  With --gpus N > 1 (launched by torchrun) every rank runs an independent
replica on its own GPU: the path has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "restored KV GB/s vs host-link/HBM roofline; per-iteration schedule latency us"
# dram__bytes_read.sum + dram__bytes_write.sum per 2 MiB block of the two grids of the fused move, from the
# 128 + 128-block ncu capture summarised in profiles/cascade_kv_move_pinned_host_128+128_blocks.md; the traffic
# grows in proportion to the blocks moved, so a launch's traffic is this figure times its block count
# (the restore figure is low because part of the written lines is still in L2 when the kernel ends)
NCU_DRAM_BYTES_PER_BLOCK = {"evict": (268_466_688 + 4_401_664) / 128, "restore": (228_096 + 208_928_768) / 128}
GB = 1e9


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--hbm-gb", type=float, default=60.0, help="paged HBM pool size in 10^9 bytes")
    ap.add_argument("--host-gb", type=float, default=40.0, help="pinned host pool size in 10^9 bytes")
    ap.add_argument("--requests", type=int, default=1024)
    ap.add_argument("--no-sweeps", action="store_true", help="skip the copy-size and queue-size sweeps")
    ap.add_argument("--separate-copies", action="store_true",
                    help="run cascade_kv_evict then cascade_kv_restore instead of the fused cascade_kv_move")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU time bound of the oracle baseline leg")
    ap.add_argument("--host-sweep-gb", type=float, default=100.0,
                    help="pinned host pool asked for (10^9 bytes): the copy sweep uses all of it, the step its first --host-gb")
    ap.add_argument("--case", default=None, choices=["copy-hbm", "copy-host", "move", "staged", "schedule", "deep"],
                    help="run one small profiling case instead of the benchmark")
    ap.add_argument("--case-n", type=int, default=None, help="blocks / requests of the --case")
    return ap.parse_args()


def make_batch(args, seed):
    from paper_2608_06557_b200 import workload as wl
    return wl.config_llama8b(seed=seed, n=args.requests, hbm_bytes=int(args.hbm_gb * GB),
                             host_bytes=int(args.host_gb * GB), hbm_free_target=256, elapsed_scale=0.3)


# --------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle as it stands, on the host cores
# --------------------------------------------------------------------------------------------
class OracleScratch:
    """Host buffers the oracle arm reuses from step to step, touched once before anything is timed."""

    def __init__(self, w):
        self.hbm_tbl = np.empty_like(w.hbm_tbl)
        self.host_tbl = np.empty_like(w.host_tbl)
        self.hbm_free = np.empty_like(w.hbm_free)
        self.host_free = np.empty_like(w.host_free)
        self.mirror_blocks = 0
        self.hbm_m = self.host_m = None

    def mirrors(self, n_hbm, n_host, bb):
        need = max(n_hbm, n_host, 1)
        if need > self.mirror_blocks:
            self.mirror_blocks = need + need // 4
            self.hbm_m = np.ones(self.mirror_blocks * bb, np.uint8)
            self.host_m = np.ones(self.mirror_blocks * bb, np.uint8)
        return self.hbm_m[: max(n_hbm, 1) * bb], self.host_m[: max(n_host, 1) * bb]


def oracle_step(w, scratch):
    """One step on the CPU oracle.  The pools are compacted to the blocks the step touches (the
    full 100 GB of pools cannot be mirrored in host RAM); the byte volume copied is unchanged.
    Returns (seconds, bytes moved)."""
    import oracle
    p = oracle.make_params(w.params)
    for dst, src in ((scratch.hbm_tbl, w.hbm_tbl), (scratch.host_tbl, w.host_tbl), (scratch.hbm_free, w.hbm_free),
                     (scratch.host_free, w.host_free)):
        np.copyto(dst, src)
    pools = oracle.Pools(scratch.hbm_tbl, scratch.host_tbl, scratch.hbm_free, w.hbm_free_count,
                         scratch.host_free, w.host_free_count, len(w.hbm_free), len(w.host_free))
    t0 = time.perf_counter()
    budget, key, _ = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
    order, grant, _, _ = oracle.schedule(p, w.reqs, key, w.D_act)
    plan = oracle.tier_plan(p, w.reqs, budget, order, grant, w.D_act, w.K_act, pools)
    t_sched = time.perf_counter() - t0
    # compact pools: one slot per touched block
    hb = np.unique(np.concatenate([plan["evict_src"], plan["restore_dst"]]))
    ob = np.unique(np.concatenate([plan["evict_dst"], plan["restore_src"]]))
    bb = w.block_bytes
    nh, no = max(len(hb), 1), max(len(ob), 1)
    lay = dict(n_blocks=nh, n_chunks=w.layout["n_chunks"], chunk_bytes=w.layout["chunk_bytes"],
               chunk_stride=nh * w.layout["chunk_bytes"], block_stride=w.layout["chunk_bytes"])
    hbm_m, host_m = scratch.mirrors(nh, no, bb)
    remap = lambda ids, uni: np.searchsorted(uni, ids).astype(np.int32)
    es, ed = remap(plan["evict_src"], hb), remap(plan["evict_dst"], ob)
    rs, rd = remap(plan["restore_src"], ob), remap(plan["restore_dst"], hb)
    t1 = time.perf_counter()
    oracle.kv_evict(hbm_m, lay, host_m, no, es, ed)
    oracle.kv_restore(hbm_m, lay, host_m, no, rs, rd)
    t_copy = time.perf_counter() - t1
    moved = (len(es) + len(rs)) * bb
    return t_sched + t_copy, moved


def host_description(core):
    """What the oracle ran on: logical cores of the box, CPU model, the core the process was pinned to."""
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    return dict(nproc=os.cpu_count(), cpu_model=model, pinned_to_core=core)


def run_oracle_arm(args, seconds, first_seed=0, max_steps=None, warmup=1):
    core = None
    try:
        core = sorted(os.sched_getaffinity(0))[0]
        os.sched_setaffinity(0, {core})
    except (OSError, AttributeError):
        pass
    w = make_batch(args, first_seed)
    scratch = OracleScratch(w)
    for s in range(max(warmup, 1)):                 # untimed: touches every buffer the timed steps use
        oracle_step(make_batch(args, 5000 + s), scratch)
    total_t, total_b, steps = 0.0, 0, 0
    t_begin = time.perf_counter()
    while True:
        if steps:
            w = make_batch(args, first_seed + steps)
        t, b = oracle_step(w, scratch)
        total_t += t
        total_b += b
        steps += 1
        if (max_steps and steps >= max_steps) or time.perf_counter() - t_begin > seconds:
            break
    return dict(value=total_b / total_t / GB if total_t > 0 else 0.0, unit="GB/s", cores=1, kind="oracle",
                sample=f"{steps} step(s) of the same workload (seeds {first_seed}..{first_seed + steps - 1}): "
                       "budget+schedule+plan on the full queue, evict/restore as memcpy on host mirrors "
                       "compacted to the blocks each step touches",
                ms_per_step=total_t / steps * 1e3, steps=steps, host=host_description(core))


def oracle_schedule_latency():
    """The oracle's budget + schedule + plan on the scheduler-scale sweep (plan-only), one core: median
    microseconds over a few iterations with churn, per queue size."""
    import oracle
    from paper_2608_06557_b200 import workload as wl
    out = {}
    for n, iters in ((1024, 20), (4096, 10), (16384, 6), (65536, 4)):
        sw = wl.SchedulerSweep(n, seed=0)
        p = oracle.make_params(sw.params)
        ts = []
        for it in range(iters):
            w = sw.workload()
            pools = oracle.Pools(None, None, None, w.hbm_free_count, None, w.host_free_count, 0, 0)
            t0 = time.perf_counter()
            budget, key, _ = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
            order, grant, _, _ = oracle.schedule(p, w.reqs, key, w.D_act)
            oracle.tier_plan(p, w.reqs, budget, order, grant, w.D_act, w.K_act, pools)
            if it:                                   # the first iteration warms the caches
                ts.append((time.perf_counter() - t0) * 1e6)
            sw.step()
        out[str(n)] = round(statistics.median(ts), 1)
    return out


def reference_main(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    # warm-up steps are run and discarded, then exactly K bounded steps are timed
    res = run_oracle_arm(args, seconds=150.0, first_seed=args.warmup, max_steps=args.steps,
                         warmup=min(max(args.warmup, 1), 3))
    line = dict(impl="reference", metric=METRIC, value=res["value"], unit="GB/s", n_gpus=args.gpus,
                steps=res["steps"], warmup=args.warmup, ms_per_step=res["ms_per_step"], higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="u8", data="synthetic",
                config=workload_config(args),
                cpu_baseline=dict(value=res["value"], unit="GB/s", cores=1, kind="oracle", sample=res["sample"],
                                  host=res["host"]),
                e2e=dict(value=res["value"], unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def workload_config(args):
    """The workload and nothing else (both arms print the same dictionary; what a run measured goes to "run")."""
    return dict(workload="llama3-8b-shaped KV step: %d requests, 3 SLO classes, 2 MiB blocks (64 x 32 KiB), "
                         "HBM pool %.0f GB, pinned host pool %.0f GB, token budget 8192, one fresh seeded batch per step"
                         % (args.requests, args.hbm_gb, args.host_gb),
                l2="every step moves far more than the 126 MB L2 across the host link; inputs larger than L2",
                replicas=args.gpus)


def rank_seed(rank: int, step: int) -> int:
    """Every replica draws its own batches: disjoint seed ranges per rank."""
    return 10_000 * rank + step


def aggregate_over_ranks(dist, ms_total: float, moved: int, device):
    """Whole-job figures of N independent replicas: the slowest rank's time, the sum of the bytes moved."""
    import torch
    t = torch.tensor([ms_total], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    mv = torch.tensor([moved], dtype=torch.int64, device=device)
    dist.all_reduce(mv, op=dist.ReduceOp.SUM)
    return float(t.item()), int(mv.item())


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def event_pair(torch):
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def measure_link_peaks(torch, host_pool, hbm_pool):
    """Pinned cudaMemcpyAsync peaks of this machine (one contiguous 1 GiB buffer, best of 5) and the
    device copy peak, the denominators of the host-link and HBM rooflines."""
    n = min(1 << 30, host_pool.numel(), hbm_pool.numel() // 2)
    h, d, d2 = host_pool[:n], hbm_pool[:n], hbm_pool[n:2 * n]
    keep_h, keep_d = h.clone(), d.clone()
    out = {}
    for name, dst, src in (("h2d", d, h), ("d2h", h, d), ("d2d", d2, d)):
        best = 1e30
        for _ in range(6):
            a, b = event_pair(torch)
            a.record()
            dst.copy_(src, non_blocking=True)
            b.record()
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        out[name] = (2 if name == "d2d" else 1) * n / best / 1e6
    h.copy_(keep_h)
    d.copy_(keep_d)
    torch.cuda.synchronize()
    return out


def timed_calls(torch, fn, reps, warm=3):
    """CUDA-event time of single calls launched from Python (the host's launch work is inside): best, median in ms."""
    ts = []
    for it in range(warm + reps):
        a, b = event_pair(torch)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        if it >= warm:
            ts.append(a.elapsed_time(b))
    return min(ts), statistics.median(ts)


def graph_per_call_us(torch, fn_i, flush, reps=20):
    """Device time per call with the host out of the way: `reps` calls (call i works on its own blocks) captured in
    one CUDA graph; a buffer larger than L2 is rewritten before every replay.  Median microseconds per call."""
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        for i in range(reps):
            fn_i(i, st)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for i in range(reps):
            fn_i(i, st)
    ts = []
    for it in range(8):
        flush.fill_(it)
        torch.cuda.synchronize()
        a, b = event_pair(torch)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(a.elapsed_time(b) / reps * 1e3)
    return statistics.median(ts)


def copy_sweep(torch, cs, ctx, layout, lay, hbm_pool, host_pool, host_blocks, stage, peaks):
    """Evict / restore bandwidth for 1, 16, 256 and 4096 scattered blocks per call, through the pinned host pool
    (host link) and through a device staging buffer (HBM).  Every figure is given twice where the call is short:
    launched from Python and bracketed by events (3 warm-ups, 20 calls; 10 for 4096 blocks over the link), and
    as device time per call inside a CUDA graph of 20 calls on distinct blocks, next to cudaMemcpyAsync copies of
    the same size measured the same way."""
    from paper_2608_06557_b200 import workload as wl
    bb = lay["n_chunks"] * lay["chunk_bytes"]
    out, median = {}, {}
    stage_blocks = stage.numel() // bb
    for n in (1, 16, 256, 4096):
        for name, rec, nrec, isdev in (("host", host_pool, host_blocks, False), ("hbm", stage, stage_blocks, True)):
            m = min(n, nrec, lay["n_blocks"])
            src, dst = wl.copy_lists(100 + n, m, nrec, lay["n_blocks"])
            s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
            reps = 20 if n <= 256 or isdev else 10
            scale = (2 if isdev else 1) * m * bb / 1e6
            best, med = timed_calls(torch, lambda: ctx.kv_evict(layout, hbm_pool, rec, nrec, isdev, d, s, None, m), reps)
            out[f"evict_{name}_{n}"], median[f"evict_{name}_{n}"] = round(scale / best, 1), round(scale / med, 1)
            best, med = timed_calls(torch, lambda: ctx.kv_restore(layout, hbm_pool, rec, nrec, isdev, s, d, None, m), reps)
            out[f"restore_{name}_{n}"], median[f"restore_{name}_{n}"] = round(scale / best, 1), round(scale / med, 1)

    # short calls without the host's launch work, and copy-engine copies of the same size measured the same way
    small = {}
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    REPS = 20
    for n in (1, 16):
        rng = np.random.default_rng(n)
        hp = rng.permutation(lay["n_blocks"])[: REPS * n].astype(np.int32).reshape(REPS, n)
        op = rng.permutation(min(host_blocks, stage_blocks))[: REPS * n].astype(np.int32).reshape(REPS, n)
        H = [torch.from_numpy(hp[i]).cuda() for i in range(REPS)]
        O = [torch.from_numpy(op[i]).cuda() for i in range(REPS)]
        nbytes = n * bb
        for name, rec, nrec, isdev, mult in (("host", host_pool, host_blocks, False, 1), ("hbm", stage, stage_blocks, True, 2)):
            t = graph_per_call_us(torch, lambda i, st: ctx.kv_restore(layout, hbm_pool, rec, nrec, isdev, O[i], H[i], None, n, st), flush)
            small[f"restore_{name}_{n}"] = dict(us=round(t, 1), GBps=round(mult * nbytes / t / 1e3, 1))
            t = graph_per_call_us(torch, lambda i, st: ctx.kv_evict(layout, hbm_pool, rec, nrec, isdev, H[i], O[i], None, n, st), flush)
            small[f"evict_{name}_{n}"] = dict(us=round(t, 1), GBps=round(mult * nbytes / t / 1e3, 1))
        for name, dst, src, mult in (("h2d", hbm_pool, host_pool, 1), ("d2h", host_pool, hbm_pool, 1), ("d2d", stage, hbm_pool, 2)):
            t = graph_per_call_us(torch, lambda i, st: dst[i * nbytes:(i + 1) * nbytes].copy_(src[i * nbytes:(i + 1) * nbytes], non_blocking=True), flush)
            small[f"cudaMemcpyAsync_{name}_{n}x2MiB"] = dict(us=round(t, 1), GBps=round(mult * nbytes / t / 1e3, 1))
        small[f"restore_host_{n}_fraction_of_same_size_copy"] = round(
            small[f"restore_host_{n}"]["GBps"] / small[f"cudaMemcpyAsync_h2d_{n}x2MiB"]["GBps"], 3)
        small[f"evict_host_{n}_fraction_of_same_size_copy"] = round(
            small[f"evict_host_{n}"]["GBps"] / small[f"cudaMemcpyAsync_d2h_{n}x2MiB"]["GBps"], 3)
        small[f"restore_host_{n}_fraction_of_1GiB_peak"] = round(small[f"restore_host_{n}"]["GBps"] / peaks["h2d"], 3)
        small[f"evict_host_{n}_fraction_of_1GiB_peak"] = round(small[f"evict_host_{n}"]["GBps"] / peaks["d2h"], 3)
    del flush
    out["graph_timed_small_calls"] = small

    # other block sizes: the tiny configuration's 16 KiB blocks (4 chunks of 4 KiB) and the 70B-shaped 5 MiB blocks
    # (160 chunks of 32 KiB), 256 blocks per call, over the link and through the staging buffer
    other = {}
    for tag, n_chunks, cb in (("16KiB", 4, 4096), ("5MiB", 160, 32768)):
        bb2 = n_chunks * cb
        nb = min(4096, hbm_pool.numel() // bb2 // 2)
        lay2 = wl.kv_layout(nb, n_chunks, cb)
        layout2 = cs.make_layout(lay2)
        m = 256
        for name, rec, isdev in (("host", host_pool, False), ("hbm", stage, True)):
            nrec = min(rec.numel() // bb2, 4096)
            src, dst = wl.copy_lists(300, m, nrec, nb)
            s_, d_ = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
            scale = (2 if isdev else 1) * m * bb2 / 1e6
            best, med = timed_calls(torch, lambda: ctx.kv_evict(layout2, hbm_pool, rec, nrec, isdev, d_, s_, None, m), 10)
            other[f"evict_{name}_{tag}_256"] = round(scale / med, 1)
            best, med = timed_calls(torch, lambda: ctx.kv_restore(layout2, hbm_pool, rec, nrec, isdev, s_, d_, None, m), 10)
            other[f"restore_{name}_{tag}_256"] = round(scale / med, 1)
    out["other_block_sizes_median_GBps"] = other

    # both directions at once: n blocks evicted and n restored in one call, half of the restores into blocks the
    # same call evicts; the zero-copy kernels (cascade_kv_move) next to the copy engines (cascade_kv_move_staged)
    duplex = {}
    for tag, n_chunks, cb, pairs in (("2MiB", lay["n_chunks"], lay["chunk_bytes"], ((16, 16), (240, 20), (256, 256), (2048, 2048))),
                                     ("5MiB", 160, 32768, ((128, 128),))):
        bb2 = n_chunks * cb
        if tag == "2MiB":
            lay2, layout2, nb, nrec = lay, layout, lay["n_blocks"], host_blocks
        else:
            nb = min(4096, hbm_pool.numel() // bb2 // 2)
            lay2 = wl.kv_layout(nb, n_chunks, cb)
            layout2, nrec = cs.make_layout(lay2), min(host_pool.numel() // bb2, 8192)
        for ne, nr in pairs:
            if ne + nr > nrec or ne + nr > nb or (ne + nr) * bb2 > stage.numel():
                continue
            rng = np.random.default_rng(ne + nr)
            hp, op = rng.permutation(nb).astype(np.int32), rng.permutation(nrec).astype(np.int32)
            es, ed, rs = hp[:ne], op[:ne], op[ne:ne + nr]
            k = min(ne, nr) // 2
            rd = np.concatenate([es[::-1][:k], hp[ne:ne + nr - k]]).astype(np.int32)
            t = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in (es, ed, rs, rd)]
            scratch = torch.empty(cs.kv_move_scratch_len(ne, nr), dtype=torch.int32, device="cuda")
            mailbox = torch.empty(cs.kv_mailbox_len(ne, nr), dtype=torch.int32, pin_memory=True)
            reps = 4 if ne + nr > 1000 else 6
            _, med = timed_calls(torch, lambda: ctx.kv_move(layout2, hbm_pool, host_pool, nrec, t[0], t[1], None, ne, t[2], t[3],
                                                            None, nr, scratch), reps, warm=2)
            _, med2 = timed_calls(torch, lambda: ctx.kv_move_staged(layout2, hbm_pool, host_pool, nrec, t[0], t[1], None, ne, t[2],
                                                                    t[3], None, nr, stage, (ne + nr), mailbox), reps, warm=2)
            gb = (ne + nr) * bb2 / 1e6
            duplex[f"{tag}_{ne}+{nr}"] = dict(zero_copy_kernels_GBps=round(gb / med, 1), copy_engines_GBps=round(gb / med2, 1))
    # what the copy engines reach with ONE contiguous copy per direction, both at once
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    nbytes = 512 << 20

    def two_way():
        cur = torch.cuda.current_stream()
        s1.wait_stream(cur)
        s2.wait_stream(cur)
        with torch.cuda.stream(s1):
            hbm_pool[:nbytes].copy_(host_pool[:nbytes], non_blocking=True)
        with torch.cuda.stream(s2):
            host_pool[nbytes:2 * nbytes].copy_(hbm_pool[nbytes:2 * nbytes], non_blocking=True)
        cur.wait_stream(s1)
        cur.wait_stream(s2)
    _, med = timed_calls(torch, two_way, 5, warm=2)
    duplex["cudaMemcpyAsync_512MiB_each_way_GBps"] = round(2 * nbytes / med / 1e6, 1)
    out["both_directions"] = duplex

    # first hop of the deep-tier path: pinned "deep" records -> pinned host records (the bytes cross the host
    # link twice, once in each direction)
    m = min(256, host_blocks)
    deep = torch.empty(m * bb, dtype=torch.uint8, pin_memory=True)
    src, dst = wl.copy_lists(77, m, m, host_blocks)
    s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
    best, _ = timed_calls(torch, lambda: ctx.kv_stage(deep, m, host_pool, host_blocks, bb, s, d, None, m), 4, warm=2)
    out[f"stage_host_{m}"] = round(m * bb / best / 1e6, 1)
    del deep
    return out, median


def deep_sweep(torch, cs):
    """Latency of the deep-tier plan steps on the shared-prefix workload (tables on the device, no pools):
    the tier plan alone, then each added step, captured in CUDA graphs of 20 iterations (each iteration also
    restores the two free-list counts with 4-byte copies so that every replay sees the same state)."""
    from paper_2608_06557_b200 import workload as wl
    from paper_2608_06557_b200.runner import Instance
    out = {}
    for n in (1024, 8192):
        w = wl.config_deep_shared(0, n=n, n_hbm=16 * n, n_host=16 * n, n_deep=32 * n, hbm_free_target=8 * n)
        w.params["plan_first"] = 1
        inst = Instance(w, alloc_pools=False)
        inst.enable_deep(w, alloc_pool=False)
        st = torch.cuda.Stream()
        saved = (inst.hbm_free_count.clone(), inst.host_free_count.clone(), inst.plan_counts.clone())
        with torch.cuda.stream(st):
            inst.run_schedule(st)
            inst.run_dedup_restore(st)
            inst.run_stage_plan(10**9, 0, st)
            inst.run_dedup_stage(st)
        torch.cuda.synchronize()
        after_plan = inst.plan_counts.clone()
        info = inst.fetch_deep()

        def reset(full):
            inst.hbm_free_count.copy_(saved[0], non_blocking=True)
            inst.host_free_count.copy_(saved[1], non_blocking=True)

        steps = dict(
            budget_schedule_plan=lambda: inst.run_schedule(st),
            merge_restore_list=lambda: inst.run_dedup_restore(st),
            stage_plan=lambda: inst.run_stage_plan(10**9, 0, st),
            merge_stage_list=lambda: inst.run_dedup_stage(st),
        )
        res = {}
        for name, fn in steps.items():
            g = torch.cuda.CUDAGraph()
            reps = 20
            with torch.cuda.graph(g, stream=st):
                for _ in range(reps):
                    reset(True)
                    fn()
            ts = []
            for it in range(8):
                a, b = event_pair(torch)
                a.record()
                g.replay()
                b.record()
                torch.cuda.synchronize()
                if it >= 3:
                    ts.append(a.elapsed_time(b) / reps * 1e3)
            res[name + "_us"] = round(statistics.median(ts), 1)
            inst.plan_counts.copy_(after_plan)
        res.update(restore_list=info["dedup_restore"]["n_in"], restore_unique=info["dedup_restore"]["n_unique"],
                   stage_list=info["dedup_stage"]["n_in"], stage_unique=info["dedup_stage"]["n_unique"])
        inst.ctx.status(clear=True)
        out[str(n)] = res
        del inst
    return out


def schedule_sweep(torch, cs):
    """budget+schedule+plan latency for 1k..64k queued requests (plan-only, no tables): the three calls
    captured in a CUDA graph, 20 iterations per replay, median microseconds per iteration; launched call by
    call; 200 iterations of the churning sweep with the 5 % slot update inside the timed region (median, p99),
    launched call by call from Python and as ONE cascade_step call per iteration."""
    from paper_2608_06557_b200 import workload as wl
    from paper_2608_06557_b200.runner import Instance
    out = {}
    for n in (1024, 4096, 16384, 65536):
        sw = wl.SchedulerSweep(n, seed=0)
        inst = Instance(sw.workload(), alloc_pools=False)
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            inst.run_schedule(st)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        reps = 20
        with torch.cuda.graph(g, stream=st):
            for _ in range(reps):
                inst.run_schedule(st)
        ts = []
        for it in range(8):
            a, b = event_pair(torch)
            a.record()
            g.replay()
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) / reps * 1e3)
        # single iteration, launched call by call and bracketed by events (includes launch latency)
        single = []
        for it in range(13):
            a, b = event_pair(torch)
            a.record()
            inst.run_schedule()
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                single.append(a.elapsed_time(b) * 1e3)
        # the sweep as it would run: every iteration 5 % of the slots are rewritten (staged in pinned memory by
        # the host, scattered into the device queue by cascade_reqs_update inside the timed region), the clock
        # and the load move on, then budget + schedule + plan
        upd, upd_bytes = [], 0
        for it in range(203):
            slots = sw.step()
            w = sw.workload()
            upd_bytes = inst.stage_slot_update(w.reqs, slots)
            inst.set_clock(w.now_ns, w.D_act, w.K_act)
            a, b = event_pair(torch)
            a.record()
            inst.run_slot_update()
            inst.run_schedule()
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                upd.append(a.elapsed_time(b) * 1e3)
        # the same churning iterations through cascade_step: one C call issues slot update + budget + schedule + plan
        step_args = inst.step_args(with_update=True)
        one = []
        for it in range(203):
            slots = sw.step()
            w = sw.workload()
            inst.stage_slot_update(w.reqs, slots)
            inst.set_clock(w.now_ns, w.D_act, w.K_act)
            a, b = event_pair(torch)
            a.record()
            inst.run_step(step_args)
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                one.append(a.elapsed_time(b) * 1e3)
        one.sort()
        plain_args = inst.step_args()
        one_plain = []
        for it in range(103):
            a, b = event_pair(torch)
            a.record()
            inst.run_step(plain_args)
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                one_plain.append(a.elapsed_time(b) * 1e3)
        one_plain.sort()
        # the same iteration (last staged update) captured in a graph: device time without the Python launches
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=st):
            for _ in range(reps):
                inst.run_slot_update(st)
                inst.run_schedule(st)
        tg = []
        for it in range(8):
            a, b = event_pair(torch)
            a.record()
            g2.replay()
            b.record()
            torch.cuda.synchronize()
            if it >= 3:
                tg.append(a.elapsed_time(b) / reps * 1e3)
        single.sort()
        upd.sort()
        out[str(n)] = dict(graph_us=round(statistics.median(ts), 1), launched_us=round(statistics.median(single), 1),
                           graph_with_slot_update_us=round(statistics.median(tg), 1),
                           with_slot_update_us=round(statistics.median(upd), 1),
                           with_slot_update_p99_us=round(upd[int(0.99 * (len(upd) - 1))], 1),
                           one_call_us=round(statistics.median(one_plain), 1),
                           one_call_p99_us=round(one_plain[int(0.99 * (len(one_plain) - 1))], 1),
                           one_call_with_slot_update_us=round(statistics.median(one), 1),
                           one_call_with_slot_update_p99_us=round(one[int(0.99 * (len(one) - 1))], 1),
                           slot_update_bytes=upd_bytes)
        inst.ctx.status(clear=True)
        del inst
    return out


def ours_main(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    use_dist = "RANK" in os.environ and "MASTER_ADDR" in os.environ     # launched by torchrun, at any world size
    if use_dist:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    import __graft_entry__ as ge
    if rank == 0:
        ge.build()
    if use_dist:
        dist.barrier()
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance, alloc_pinned_pool, fill_pools

    dev = f"cuda:{local_rank}"
    K, W = args.steps, max(args.warmup, 0)
    # ---- inputs: W+K fresh batches, resident on the device before anything is timed ---------------
    batches = [make_batch(args, rank_seed(rank, s)) for s in range(W + K)]
    w0 = batches[0]
    bb = w0.block_bytes
    # one pinned allocation: the copy sweep's pool as stated (100 * 10^9 bytes, or what the box grants); the step
    # uses its first --host-gb
    want_sweep = 0 if args.no_sweeps or rank != 0 else int(args.host_sweep_gb * GB) // bb * bb
    # every rank of a multi-replica run pins its own pool on the same host: each takes its share of what is available
    big_pool, big_bytes = alloc_pinned_pool(max(want_sweep, w0.host_blocks * bb), share_of_available=0.7 / max(world, 1))
    if big_bytes < w0.host_blocks * bb:        # pinning was refused at full size: regenerate at the size we got
        args.host_gb = big_bytes / GB
        batches = [make_batch(args, rank_seed(rank, s)) for s in range(W + K)]
        w0 = batches[0]
    host_pool = big_pool[: w0.host_blocks * bb]
    hbm_pool = torch.empty(w0.layout["n_blocks"] * bb, dtype=torch.uint8, device=dev)
    fill_pools(hbm_pool, big_pool)
    ctx = cs.Context(w0.params, args.requests, local_rank)
    insts = [Instance(w, device=dev, ctx=ctx, hbm_pool=hbm_pool, host_pool=host_pool, alloc_pools=False)
             for w in batches]
    torch.cuda.synchronize()
    peaks = measure_link_peaks(torch, host_pool, hbm_pool)

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, then exactly K timed steps ------------------------------------------------------
    fused = not args.separate_copies
    FUSED_MOVE[0] = fused
    for i in range(W):
        insts[i].run_iteration(fused_move=fused)
    barrier()
    sampler = ClockSampler(local_rank)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    t_all = event_pair(torch)
    t_all[0].record()
    for i in range(K):
        inst = insts[W + i]
        ev[i][0].record()
        inst.run_schedule()
        ev[i][1].record()
        c = inst.ctx
        if fused:
            inst.run_move()
            ev[i][2].record()
        else:
            c.kv_evict(inst.layout, inst.hbm_pool, inst.host_pool, inst.host_blocks, False, inst.evict_src,
                       inst.evict_dst, inst.plan_counts[1:2], inst.evict_cap)
            ev[i][2].record()
            c.kv_restore(inst.layout, inst.hbm_pool, inst.host_pool, inst.host_blocks, False, inst.restore_src,
                         inst.restore_dst, inst.plan_counts[0:1], inst.restore_cap)
        ev[i][3].record()
    t_all[1].record()
    barrier()
    clocks = sampler.stop()
    ms_total = t_all[0].elapsed_time(t_all[1])
    status = ctx.status()[0]
    counts = [insts[W + i].plan_counts.cpu().numpy() for i in range(K)]
    n_restore = np.array([int(c[0]) for c in counts])
    n_evict = np.array([int(c[1]) for c in counts])
    moved = int((n_restore.sum() + n_evict.sum()) * bb)
    t_sched = np.array([ev[i][0].elapsed_time(ev[i][1]) for i in range(K)])
    t_evict = np.array([ev[i][1].elapsed_time(ev[i][2]) for i in range(K)])
    t_rest = np.array([ev[i][2].elapsed_time(ev[i][3]) for i in range(K)])
    # rate of every single step: the host link is shared with other tenants of the machine, a step that ran beside
    # somebody else's traffic shows here (the reported value stays the K-step total)
    t_step = t_sched + t_evict + t_rest
    big = (n_restore + n_evict) >= 64           # steps that move little say nothing about the link
    step_gbs = ((n_restore + n_evict) * bb / np.maximum(t_step, 1e-6) / 1e6)[big] if big.any() else np.zeros(1)
    if use_dist:
        ms_total, moved = aggregate_over_ranks(dist, ms_total, moved, dev)
    value = moved / (ms_total * 1e-3) / GB

    # ---- dominant kernel of the step and its roofline ----------------------------------------------
    ev_bytes, rs_bytes = int(n_evict.sum()) * bb, int(n_restore.sum()) * bb
    if fused:
        # one kernel moves both lists; the link carries the two directions at once, so the floor of a step is
        # the slower of (evicted bytes / D2H peak) and (restored bytes / H2D peak)
        t_move = float((t_evict + t_rest).sum())
        ideal_ms = sum(max(int(e) * bb / peaks["d2h"], int(r) * bb / peaks["h2d"]) for e, r in zip(n_evict, n_restore)) / 1e6
        dom_ach = (ev_bytes + rs_bytes) / (t_move * 1e-3) / GB if t_move else 0.0
        dom_peak = (ev_bytes + rs_bytes) / (ideal_ms * 1e-3) / GB if ideal_ms else 0.0
        dominant = "cascade_kv_move: kv_ring_kernel<evict> beside kv_copy_kernel<restore> (both link directions)"
        dom_launch_bytes = (ev_bytes + rs_bytes) / K
        traffic = int((NCU_DRAM_BYTES_PER_BLOCK["evict"] * n_evict.sum() + NCU_DRAM_BYTES_PER_BLOCK["restore"] * n_restore.sum()) / K)
        evict_gbs = restore_gbs = None
    else:
        evict_gbs = ev_bytes / (t_evict.sum() * 1e-3) / GB if ev_bytes else 0.0
        restore_gbs = rs_bytes / (t_rest.sum() * 1e-3) / GB if rs_bytes else 0.0
        is_ev = t_evict.sum() >= t_rest.sum()
        dominant = "kv_ring_kernel<evict>" if is_ev else "kv_ring_kernel<restore>"
        dom_ach = evict_gbs if is_ev else restore_gbs
        dom_peak = peaks["d2h"] if is_ev else peaks["h2d"]
        dom_launch_bytes = (ev_bytes if is_ev else rs_bytes) / K
        traffic = int(NCU_DRAM_BYTES_PER_BLOCK["evict" if is_ev else "restore"] * dom_launch_bytes / bb)
    roofline = dict(bound="host_link", kernel=dominant, achieved=round(dom_ach, 2), peak=round(dom_peak, 2),
                    unit="GB/s", frac=round(dom_ach / dom_peak, 4) if dom_peak else None,
                    traffic=traffic,
                    traffic_source="ncu captures of 128 blocks per direction, scaled by the blocks per launch",
                    algorithmic_bytes_per_launch=int(dom_launch_bytes),
                    link_peaks_GBps=dict(h2d=round(peaks["h2d"], 2), d2h=round(peaks["d2h"], 2)),
                    peak_source="pinned cudaMemcpyAsync of one contiguous 1 GiB buffer per direction, measured by "
                                "this run (MEASURED_PEAKS.json holds no host-link figure); for the fused kernel the "
                                "peak is the byte total over the slower direction's ideal time",
                    note="the bytes cross the host link, not HBM: the HBM-side traffic equals the algorithmic bytes")

    line = dict(metric=METRIC, value=round(value, 3), unit="GB/s", n_gpus=world, steps=K, warmup=W,
                ms_per_step=round(ms_total / K, 4), higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="u8", data="synthetic")

    if rank == 0:
        # ---- end to end: inputs start in pinned host memory, results are read back every step -------
        e2e = run_e2e(torch, args, batches[W:], insts[:2] if len(insts) > 1 else [insts[0], insts[0]], K)
        line["config"] = workload_config(args)
        line["run"] = dict(blocks_restored_per_step=float(n_restore.mean()), blocks_evicted_per_step=float(n_evict.mean()),
                           host_pool_bytes=int(host_pool.numel()), hbm_pool_bytes=int(hbm_pool.numel()),
                           status_bits=status,
                           step_GBps=dict(median=round(float(np.median(step_gbs)), 2), min=round(float(step_gbs.min()), 2),
                                          max=round(float(step_gbs.max()), 2), steps_counted=int(big.sum()),
                                          note="steps that move at least 64 blocks"))
        line["clocks"] = clocks
        line["e2e"] = e2e
        # budget, schedule, plan + 2 table rewrites, and the move's prepare + evict grid + restore grid
        line["gpu_launches"] = (8 if fused else 7) * K
        line["roofline"] = roofline
        line["kernels"] = dict(schedule_us_per_step=round(float(np.median(t_sched)) * 1e3, 1),
                               copies="fused cascade_kv_move" if fused else "cascade_kv_evict + cascade_kv_restore",
                               move_GBps=round(dom_ach, 2) if fused else None,
                               evict_GBps=round(evict_gbs, 2) if evict_gbs is not None else None,
                               restore_GBps=round(restore_gbs, 2) if restore_gbs is not None else None,
                               measured_peaks_GBps={k: round(v, 1) for k, v in peaks.items()})
        if not args.no_sweeps:
            stage_bytes = min(8 << 30, (hbm_pool.numel() // 4 // bb) * bb)
            # the staging buffer is carved from the tail of the HBM pool after the timed steps are over
            stage = hbm_pool[hbm_pool.numel() - stage_bytes:]
            lay = dict(w0.layout)
            lay_small = dict(lay, n_blocks=(hbm_pool.numel() - stage_bytes) // bb // 2)
            lay_small["chunk_stride"] = lay_small["n_blocks"] * lay["chunk_bytes"]
            sweep, sweep_median = copy_sweep(torch, cs, ctx, cs.make_layout(lay_small), lay_small, hbm_pool, big_pool,
                                             big_pool.numel() // bb, stage, peaks)
            line["run"]["copy_sweep_host_pool"] = dict(asked_bytes=int(args.host_sweep_gb * GB), pinned_bytes=int(big_bytes),
                                                       records=int(big_pool.numel() // bb))
            line["copy_sweep_GBps"] = sweep
            line["copy_sweep_median_GBps"] = sweep_median
            hbm_peak = load_hbm_peak()
            big = sweep.get("restore_hbm_4096", 0.0)
            line["roofline_hbm"] = dict(bound="hbm", kernel="kv_ring_kernel<restore>, device staging buffer, "
                                        "4096 blocks", achieved=big, peak=hbm_peak[0], unit="GB/s",
                                        frac=round(big / hbm_peak[0], 4),
                                        traffic=int(1028.25e6 / 256 * 4096),
                                        traffic_source="ncu capture of 256 staged blocks (537.0 MB read + 491.3 MB "
                                                       "written), scaled to 4096 blocks",
                                        algorithmic_bytes_per_launch=int(2 * 4096 * bb), peak_source=hbm_peak[1])
            del insts
            line["schedule_latency_us"] = schedule_sweep(torch, cs)
            line["deep_tier_us"] = deep_sweep(torch, cs)
            # the four targets the build was given, side by side with what this run measured
            sl = line["schedule_latency_us"]
            small = sweep["graph_timed_small_calls"]
            line["targets"] = dict(
                restore_fraction_of_h2d_peak=dict(target=0.80, measured=round(sweep["restore_host_256"] / peaks["h2d"], 3),
                                                  at_16_blocks=small["restore_host_16_fraction_of_1GiB_peak"],
                                                  at_1_block=small["restore_host_1_fraction_of_1GiB_peak"],
                                                  at_1_block_of_same_size_copy=small["restore_host_1_fraction_of_same_size_copy"]),
                evict_fraction_of_d2h_peak=dict(target=0.80, measured=round(sweep["evict_host_256"] / peaks["d2h"], 3),
                                                at_16_blocks=small["evict_host_16_fraction_of_1GiB_peak"],
                                                at_1_block=small["evict_host_1_fraction_of_1GiB_peak"]),
                hbm_scatter_fraction_of_hbm_peak=dict(target=0.70, measured=round(sweep["restore_hbm_4096"] / hbm_peak[0], 3),
                                                      at_256_blocks=round(sweep["restore_hbm_256"] / hbm_peak[0], 3),
                                                      at_16_blocks=round(small["restore_hbm_16"]["GBps"] / hbm_peak[0], 3),
                                                      one_block_latency_us=small["restore_hbm_1"]["us"]),
                budget_schedule_plan_16k_us=dict(target=100.0, measured=sl["16384"]["graph_us"],
                                                 launched_from_python=sl["16384"]["launched_us"],
                                                 one_call=sl["16384"]["one_call_us"],
                                                 one_call_p99=sl["16384"]["one_call_p99_us"],
                                                 one_call_with_slot_update=sl["16384"]["one_call_with_slot_update_us"],
                                                 one_call_with_slot_update_p99=sl["16384"]["one_call_with_slot_update_p99_us"]),
                parity="bit-exact against the CPU oracle: see tests/ (-m gpu)")
        line["cpu_baseline"] = {k: v for k, v in run_oracle_arm(args, args.cpu_seconds, first_seed=W).items()
                                if k in ("value", "unit", "cores", "kind", "sample", "host")}
        if not args.no_sweeps:
            line["cpu_baseline"]["schedule_latency_us"] = oracle_schedule_latency()
        print(json.dumps(line))
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def load_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "MEASURED_PEAKS.json (of measured)"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback 6.65 TB/s (of fallback)"


FUSED_MOVE = [True]


def run_e2e(torch, args, batches, two, K):
    """The same metric through the public API with HOST inputs: every step copies that step's request
    arrays, block tables and free lists from pinned host memory, runs the calls and reads the per-request
    results and counts back to the host, which waits for them before it goes on.  Two sets of device buffers
    (`two`) alternate, so the inputs of step i+1 travel on a second stream while step i runs."""
    keys_req = ("arrival_ns", "prompt", "pred_out", "n0", "n1", "n2", "id", "cls", "flags")
    pinned = []
    for w in batches[:K]:
        p = {k: torch.from_numpy(np.ascontiguousarray(w.reqs[k]).view(np.int32) if w.reqs[k].dtype == np.uint32
                                 else np.ascontiguousarray(w.reqs[k])).pin_memory() for k in keys_req}
        p["hbm_tbl"] = torch.from_numpy(w.hbm_tbl).pin_memory()
        p["host_tbl"] = torch.from_numpy(w.host_tbl).pin_memory()
        p["hbm_free"] = torch.from_numpy(w.hbm_free).pin_memory()
        p["host_free"] = torch.from_numpy(w.host_free).pin_memory()
        p["counts"] = torch.tensor([w.hbm_free_count, w.host_free_count], dtype=torch.int32).pin_memory()
        pinned.append((w, p))
    n = two[0].n
    out_host = dict(grant=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    x1=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    x2=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    tokens_run=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    action=torch.empty(n, dtype=torch.uint8, pin_memory=True),
                    counts=torch.empty(12, dtype=torch.int32, pin_memory=True))
    h2d = sum(t.numel() * t.element_size() for t in pinned[0][1].values())
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())
    main, up = torch.cuda.current_stream(), torch.cuda.Stream()
    uploaded = [torch.cuda.Event(), torch.cuda.Event()]
    finished = [torch.cuda.Event(), torch.cuda.Event()]
    free_counts = [torch.empty(2, dtype=torch.int32, device=two[0].device) for _ in range(2)]

    def upload(j, w, p):
        inst = two[j % 2]
        if j >= 2:
            up.wait_event(finished[j % 2])          # the step that last used these buffers is over
        with torch.cuda.stream(up):
            for k in keys_req:
                dst = inst.reqs[k][:n]
                dst.view(torch.int32).copy_(p[k], non_blocking=True) if dst.dtype == torch.uint32 else \
                    dst.copy_(p[k], non_blocking=True)
            inst.hbm_tbl.copy_(p["hbm_tbl"], non_blocking=True)
            inst.host_tbl.copy_(p["host_tbl"], non_blocking=True)
            inst.hbm_free.copy_(p["hbm_free"], non_blocking=True)
            inst.host_free.copy_(p["host_free"], non_blocking=True)
            free_counts[j % 2].copy_(p["counts"], non_blocking=True)
            inst.hbm_free_count.copy_(free_counts[j % 2][0:1], non_blocking=True)
            inst.host_free_count.copy_(free_counts[j % 2][1:2], non_blocking=True)
            uploaded[j % 2].record(up)

    step_args = [inst.step_args(with_move=True) if FUSED_MOVE[0] else None for inst in two]

    def enqueue(j, w):
        inst = two[j % 2]
        main.wait_event(uploaded[j % 2])
        inst.set_clock(w.now_ns, w.D_act, w.K_act)
        if FUSED_MOVE[0]:
            inst.run_step(step_args[j % 2])         # the whole iteration as one call of the C ABI
        else:
            inst.run_iteration(fused_move=False)
        out_host["grant"].copy_(inst.grant[:n], non_blocking=True)
        out_host["x1"].copy_(inst.x1[:n], non_blocking=True)
        out_host["x2"].copy_(inst.x2[:n], non_blocking=True)
        out_host["tokens_run"].copy_(inst.tokens_run[:n], non_blocking=True)
        out_host["action"].copy_(inst.action[:n], non_blocking=True)
        out_host["counts"].copy_(inst.plan_counts, non_blocking=True)
        finished[j % 2].record(main)

    def finish():
        main.synchronize()                          # the caller needs the plan before it goes on
        return int(out_host["counts"][0]) + int(out_host["counts"][1])

    upload(0, *pinned[0])                           # untimed warm-up of the code path
    enqueue(0, pinned[0][0])
    finish()
    torch.cuda.synchronize()
    moved = 0
    a, b = event_pair(torch)
    a.record()
    upload(0, *pinned[0])
    for j, (w, p) in enumerate(pinned):
        enqueue(j, w)
        if j + 1 < len(pinned):
            upload(j + 1, *pinned[j + 1])           # queued behind nothing: it runs beside step j
        moved += finish() * two[0].block_bytes
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b)
    return dict(value=round(moved / (ms * 1e-3) / GB, 3), unit="GB/s", h2d_bytes_per_step=int(h2d),
                d2h_bytes_per_step=int(d2h), ms_per_step=round(ms / len(pinned), 4),
                note="inputs of step i+1 are uploaded on a second stream while step i runs; the host waits for "
                     "every step's results")


# --------------------------------------------------------------------------------------------
# small cases: one kernel family, a few launches (what the ncu captures under profiles/ run)
# --------------------------------------------------------------------------------------------
def run_case(args):
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200 import workload as wl
    from paper_2608_06557_b200.runner import Instance

    def timed(fn, reps=5):
        out = []
        for _ in range(reps):
            a, b = event_pair(torch)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            out.append(a.elapsed_time(b) * 1e3)
        return out

    n_chunks, chunk_bytes = 64, 32 * 1024
    bb = n_chunks * chunk_bytes
    case = args.case
    if case in ("copy-hbm", "copy-host"):
        n = args.case_n or 256
        on_device = case == "copy-hbm"
        n_hbm, n_rec = 2 * n + 64, n + 64
        lay = wl.kv_layout(n_hbm, n_chunks, chunk_bytes)
        hbm = torch.empty(n_hbm * bb, dtype=torch.uint8, device="cuda").fill_(1)
        rec = (torch.empty(n_rec * bb, dtype=torch.uint8, device="cuda") if on_device
               else torch.empty(n_rec * bb, dtype=torch.uint8, pin_memory=True)).fill_(2)
        ctx = cs.Context(wl.default_params(), 16, 0)
        layout = cs.make_layout(lay)
        src, dst = wl.copy_lists(7, n, n_rec, n_hbm)
        s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
        torch.cuda.synchronize()
        t_r = timed(lambda: ctx.kv_restore(layout, hbm, rec, n_rec, on_device, s, d, None, n))
        t_e = timed(lambda: ctx.kv_evict(layout, hbm, rec, n_rec, on_device, d, s, None, n))
        mult = 2 if on_device else 1
        for name, ts in (("restore", t_r), ("evict", t_e)):
            print(f"{name}: {n} blocks x {bb} B, us per launch {[round(t, 1) for t in ts]}, "
                  f"best {mult * n * bb / min(ts) / 1e3:.1f} GB/s ({'read+write' if mult == 2 else 'link'} bytes)")
        print("status", ctx.status())
    elif case in ("move", "staged"):
        # n blocks evicted and n restored by one call; half of the restores reuse evicted blocks
        n = args.case_n or 128
        n_hbm, n_rec = 3 * n + 64, 3 * n + 64
        lay = wl.kv_layout(n_hbm, n_chunks, chunk_bytes)
        hbm = torch.empty(n_hbm * bb, dtype=torch.uint8, device="cuda").fill_(1)
        rec = torch.empty(n_rec * bb, dtype=torch.uint8, pin_memory=True).fill_(2)
        ctx = cs.Context(wl.default_params(), 16, 0)
        layout = cs.make_layout(lay)
        rng = np.random.default_rng(3)
        hp, op = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_rec).astype(np.int32)
        es, ed, rs = hp[:n], op[:n], op[n:2 * n]
        rd = np.concatenate([es[::-1][: n // 2], hp[n:2 * n - n // 2]]).astype(np.int32)
        t = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in (es, ed, rs, rd)]
        if case == "move":
            scratch = torch.empty(cs.kv_move_scratch_len(n, n), dtype=torch.int32, device="cuda")
            fn = lambda: ctx.kv_move(layout, hbm, rec, n_rec, t[0], t[1], None, n, t[2], t[3], None, n, scratch)
        else:
            staging = torch.empty(2 * n * bb, dtype=torch.uint8, device="cuda")
            mailbox = torch.empty(cs.kv_mailbox_len(n, n), dtype=torch.int32, pin_memory=True)
            fn = lambda: ctx.kv_move_staged(layout, hbm, rec, n_rec, t[0], t[1], None, n, t[2], t[3], None, n, staging,
                                            2 * n, mailbox)
        torch.cuda.synchronize()
        ts = timed(fn)
        print(f"{case}: {n} evicted + {n} restored blocks x {bb} B, us per call {[round(x, 1) for x in ts]}, "
              f"best {2 * n * bb / min(ts) / 1e3:.1f} GB/s over the link (both directions)")
        print("status", ctx.status())
    elif case == "schedule":
        n = args.case_n or 16384
        sw = wl.SchedulerSweep(n, seed=0)
        inst = Instance(sw.workload(), alloc_pools=False)
        ts = timed(inst.run_schedule, reps=8)
        print(f"budget+schedule+plan, {n} requests, us per iteration (event-bracketed, launched call by call): "
              f"{[round(t, 1) for t in ts]}")
        print("status", inst.ctx.status())
    elif case == "deep":
        # three independent iterations (seeds 0..2) of the shared-prefix workload: plan, merge of the restore list,
        # stage plan, merge of the stage list, evict + restore, stage copy (16 KiB blocks)
        n = args.case_n or 1024
        for seed in range(3):
            w = wl.config_deep_shared(seed, n=n, n_hbm=16 * n, n_host=16 * n, n_deep=32 * n, hbm_free_target=8 * n)
            w.params["plan_first"] = 1
            inst = Instance(w)
            inst.enable_deep(w)
            inst.hbm_pool.fill_(1)
            inst.host_pool.fill_(2)
            inst.deep_pool.fill_(3)
            torch.cuda.synchronize()
            ts = timed(lambda: inst.run_iteration_deep(10**9, 0), reps=1)
            d = inst.fetch_deep()
            print(f"seed {seed}: {n} requests, iteration {ts[0]:.1f} us; restore list {d['dedup_restore']['n_in']} -> "
                  f"{d['dedup_restore']['n_unique']}, stage list {d['dedup_stage']['n_in']} -> "
                  f"{d['dedup_stage']['n_unique']}, status {inst.ctx.status()}")
            del inst


def main():
    args = parse_args()
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        reference_main(args)
    else:
        ours_main(args)


if __name__ == "__main__":
    main()
