#!/usr/bin/env python
"""Benchmark of the Cascade scheduling + KV-tier step on B200.

A step is one pass of the whole hot path (budget -> schedule -> tier plan -> KV evict -> KV restore)
over one batch of synthetic input in the Llama-3-8B-shaped configuration: 1024 queued requests,
2 MiB KV blocks, a 60 GB paged HBM pool and a 40 GB pinned host pool.  Every step works on a fresh
seeded batch (request arrays, block tables, free lists) that is already resident in HBM when the
timed region starts; the KV bytes a step moves cross the host link inside the copy kernels.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line.  With --gpus N > 1 (launched by torchrun) every rank runs an independent
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
# dram__bytes_read.sum + dram__bytes_write.sum per 2 MiB block of the host-link copy kernel, from the
# 128-block ncu captures summarised in profiles/kv_copy_bulk_kernel_pinned_host_128_blocks.md; the traffic
# grows in proportion to the blocks moved, so a launch's traffic is this figure times its block count
# (the restore figure is low because part of the written lines is still in L2 when the kernel ends)
NCU_DRAM_BYTES_PER_BLOCK = {"evict": (268_630_272 + 3_547_648) / 128, "restore": (99_840 + 209_025_792) / 128}
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


def run_oracle_arm(args, seconds, first_seed=0, max_steps=None, warmup=1):
    try:
        os.sched_setaffinity(0, {sorted(os.sched_getaffinity(0))[0]})
    except OSError:
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
                ms_per_step=total_t / steps * 1e3, steps=steps)


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
                config=workload_config(args, None),
                cpu_baseline=dict(value=res["value"], unit="GB/s", cores=1, kind="oracle", sample=res["sample"]),
                e2e=dict(value=res["value"], unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def workload_config(args, extra):
    cfg = dict(workload="llama3-8b-shaped KV step: %d requests, 3 SLO classes, 2 MiB blocks (64 x 32 KiB), "
                        "HBM pool %.0f GB, pinned host pool %.0f GB, token budget 8192, one fresh seeded batch per step"
                        % (args.requests, args.hbm_gb, args.host_gb),
               l2="every step moves far more than the 126 MB L2 across the host link; inputs larger than L2",
               replicas=args.gpus)
    if extra:
        cfg.update(extra)
    return cfg


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


def copy_sweep(torch, cs, ctx, layout, lay, hbm_pool, host_pool, host_blocks, stage):
    """Evict / restore bandwidth for 1, 16, 256 and 4096 scattered blocks per call, through the pinned
    host pool (host link) and through a device staging buffer (HBM): 3 warm-ups, then 20 timed calls (10 for
    4096 blocks over the host link); best and median."""
    from paper_2608_06557_b200 import workload as wl
    bb = lay["n_chunks"] * lay["chunk_bytes"]
    out, median = {}, {}
    stage_blocks = stage.numel() // bb
    for n in (1, 16, 256, 4096):
        for name, rec, nrec, isdev in (("host", host_pool, host_blocks, False), ("hbm", stage, stage_blocks, True)):
            m = min(n, nrec, lay["n_blocks"])
            src, dst = wl.copy_lists(100 + n, m, nrec, lay["n_blocks"])
            s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
            for kind in ("evict", "restore"):
                ts = []
                for it in range(3 + (20 if n <= 256 or isdev else 10)):
                    a, b = event_pair(torch)
                    a.record()
                    if kind == "evict":
                        ctx.kv_evict(layout, hbm_pool, rec, nrec, isdev, d, s, None, m)
                    else:
                        ctx.kv_restore(layout, hbm_pool, rec, nrec, isdev, s, d, None, m)
                    b.record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        ts.append(a.elapsed_time(b))
                scale = (2 if isdev else 1) * m * bb / 1e6
                out[f"{kind}_{name}_{n}"] = round(scale / min(ts), 1)
                median[f"{kind}_{name}_{n}"] = round(scale / statistics.median(ts), 1)
    # both directions at once: n blocks evicted and n restored by one cascade_kv_move, half of the restores
    # into blocks the same call evicts
    for n in (16, 256, 2048):
        m = min(n, host_blocks // 2, lay["n_blocks"] // 2)
        rng = np.random.default_rng(n)
        hp, op = rng.permutation(lay["n_blocks"]).astype(np.int32), rng.permutation(host_blocks).astype(np.int32)
        es, ed, rs = hp[:m], op[:m], op[m:2 * m]
        rd = np.concatenate([es[::-1][: m // 2], hp[m:2 * m - m // 2]]).astype(np.int32)
        t = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in (es, ed, rs, rd)]
        scratch = torch.empty(cs.kv_move_scratch_len(m, m), dtype=torch.int32, device="cuda")
        best = 1e30
        for it in range(6):
            a, b = event_pair(torch)
            a.record()
            ctx.kv_move(layout, hbm_pool, host_pool, host_blocks, t[0], t[1], None, m, t[2], t[3], None, m, scratch)
            b.record()
            torch.cuda.synchronize()
            if it >= 2:
                best = min(best, a.elapsed_time(b))
        out[f"move_host_{n}+{n}"] = round(2 * m * bb / best / 1e6, 1)
    # first hop of the deep-tier path: pinned "deep" records -> pinned host records (the bytes cross the host
    # link twice, once in each direction)
    m = min(256, host_blocks)
    deep = torch.empty(m * bb, dtype=torch.uint8, pin_memory=True)
    src, dst = wl.copy_lists(77, m, m, host_blocks)
    s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
    best = 1e30
    for it in range(6):
        a, b = event_pair(torch)
        a.record()
        ctx.kv_stage(deep, m, host_pool, host_blocks, bb, s, d, None, m)
        b.record()
        torch.cuda.synchronize()
        if it >= 2:
            best = min(best, a.elapsed_time(b))
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
    call; and 200 iterations of the churning sweep with the 5 % slot update inside the timed region (median, p99)."""
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
    host_pool, host_bytes = alloc_pinned_pool(w0.host_blocks * bb)
    if host_bytes != w0.host_blocks * bb:      # pinning was refused at full size: regenerate at the size we got
        args.host_gb = host_bytes / GB
        batches = [make_batch(args, rank_seed(rank, s)) for s in range(W + K)]
        w0 = batches[0]
        host_pool = host_pool[: w0.host_blocks * bb]
    hbm_pool = torch.empty(w0.layout["n_blocks"] * bb, dtype=torch.uint8, device=dev)
    fill_pools(hbm_pool, host_pool)
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
        dominant = "kv_move_kernel (evict + restore, both link directions)"
        dom_launch_bytes = (ev_bytes + rs_bytes) / K
        traffic = int((NCU_DRAM_BYTES_PER_BLOCK["evict"] * n_evict.sum() + NCU_DRAM_BYTES_PER_BLOCK["restore"] * n_restore.sum()) / K)
        evict_gbs = restore_gbs = None
    else:
        evict_gbs = ev_bytes / (t_evict.sum() * 1e-3) / GB if ev_bytes else 0.0
        restore_gbs = rs_bytes / (t_rest.sum() * 1e-3) / GB if rs_bytes else 0.0
        is_ev = t_evict.sum() >= t_rest.sum()
        dominant = "kv_copy_bulk_kernel<evict>" if is_ev else "kv_copy_bulk_kernel<restore>"
        dom_ach = evict_gbs if is_ev else restore_gbs
        dom_peak = peaks["d2h"] if is_ev else peaks["h2d"]
        dom_launch_bytes = (ev_bytes if is_ev else rs_bytes) / K
        traffic = int(NCU_DRAM_BYTES_PER_BLOCK["evict" if is_ev else "restore"] * dom_launch_bytes / bb)
    roofline = dict(bound="host_link", kernel=dominant, achieved=round(dom_ach, 2), peak=round(dom_peak, 2),
                    unit="GB/s", frac=round(dom_ach / dom_peak, 4) if dom_peak else None,
                    traffic=traffic,
                    traffic_source="ncu captures of 128 blocks per direction, scaled by the blocks per launch",
                    algorithmic_bytes_per_launch=int(dom_launch_bytes),
                    peak_source="pinned cudaMemcpyAsync of one contiguous 1 GiB buffer per direction, measured by "
                                "this run (MEASURED_PEAKS.json holds no host-link figure); for the fused kernel the "
                                "peak is the byte total over the slower direction's ideal time",
                    note="the bytes cross the host link, not HBM: the HBM-side traffic equals the algorithmic bytes")

    line = dict(metric=METRIC, value=round(value, 3), unit="GB/s", n_gpus=world, steps=K, warmup=W,
                ms_per_step=round(ms_total / K, 4), higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="u8", data="synthetic")

    if rank == 0:
        # ---- end to end: inputs start in pinned host memory, results are read back every step -------
        e2e = run_e2e(torch, args, batches[W:], insts[0], K)
        extra = dict(blocks_restored_per_step=float(n_restore.mean()), blocks_evicted_per_step=float(n_evict.mean()),
                     host_pool_bytes=int(host_pool.numel()), hbm_pool_bytes=int(hbm_pool.numel()),
                     status_bits=status)
        line["config"] = workload_config(args, extra)
        line["clocks"] = clocks
        line["e2e"] = e2e
        line["gpu_launches"] = 7 * K
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
            sweep, sweep_median = copy_sweep(torch, cs, ctx, cs.make_layout(lay_small), lay_small, hbm_pool, host_pool,
                                             w0.host_blocks, stage)
            line["copy_sweep_GBps"] = sweep
            line["copy_sweep_median_GBps"] = sweep_median
            hbm_peak = load_hbm_peak()
            big = sweep.get("restore_hbm_4096", 0.0)
            line["roofline_hbm"] = dict(bound="hbm", kernel="kv_copy_bulk_kernel<restore>, device staging buffer, "
                                        "4096 blocks", achieved=big, peak=hbm_peak[0], unit="GB/s",
                                        frac=round(big / hbm_peak[0], 4),
                                        traffic=int(1027.4e6 / 256 * 4096),
                                        traffic_source="ncu capture of 256 staged blocks (537.0 MB read + 490.4 MB "
                                                       "written), scaled to 4096 blocks",
                                        algorithmic_bytes_per_launch=int(2 * 4096 * bb), peak_source=hbm_peak[1])
            del insts
            line["schedule_latency_us"] = schedule_sweep(torch, cs)
            line["deep_tier_us"] = deep_sweep(torch, cs)
            # the four targets the build was given, side by side with what this run measured
            sl = line["schedule_latency_us"]
            line["targets"] = dict(
                restore_fraction_of_h2d_peak=dict(target=0.80, measured=round(sweep["restore_host_256"] / peaks["h2d"], 3)),
                evict_fraction_of_d2h_peak=dict(target=0.80, measured=round(sweep["evict_host_256"] / peaks["d2h"], 3)),
                hbm_scatter_fraction_of_hbm_peak=dict(target=0.70, measured=round(sweep["restore_hbm_4096"] / hbm_peak[0], 3)),
                budget_schedule_plan_16k_us=dict(target=100.0, measured=sl["16384"]["graph_us"],
                                                 launched_from_python=sl["16384"]["launched_us"]),
                parity="bit-exact against the CPU oracle: see tests/ (-m gpu)")
        line["cpu_baseline"] = {k: v for k, v in run_oracle_arm(args, args.cpu_seconds, first_seed=W).items()
                                if k in ("value", "unit", "cores", "kind", "sample")}
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


def run_e2e(torch, args, batches, inst, K):
    """The same metric through the public API with HOST inputs: every step copies that step's request
    arrays, block tables and free lists from pinned host memory, runs the five calls and reads the
    per-request results and counts back to the host."""
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
    n = inst.n
    out_host = dict(grant=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    x1=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    x2=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    tokens_run=torch.empty(n, dtype=torch.int32, pin_memory=True),
                    action=torch.empty(n, dtype=torch.uint8, pin_memory=True),
                    counts=torch.empty(12, dtype=torch.int32, pin_memory=True))
    h2d = sum(t.numel() * t.element_size() for t in pinned[0][1].values())
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())
    free_counts = torch.empty(2, dtype=torch.int32, device=inst.device)
    moved = 0

    def step(w, p):
        for k in keys_req:
            dst = inst.reqs[k][:n]
            dst.view(torch.int32).copy_(p[k], non_blocking=True) if dst.dtype == torch.uint32 else \
                dst.copy_(p[k], non_blocking=True)
        inst.hbm_tbl.copy_(p["hbm_tbl"], non_blocking=True)
        inst.host_tbl.copy_(p["host_tbl"], non_blocking=True)
        inst.hbm_free.copy_(p["hbm_free"], non_blocking=True)
        inst.host_free.copy_(p["host_free"], non_blocking=True)
        free_counts.copy_(p["counts"], non_blocking=True)
        inst.hbm_free_count.copy_(free_counts[0:1], non_blocking=True)
        inst.host_free_count.copy_(free_counts[1:2], non_blocking=True)
        inst.set_clock(w.now_ns, w.D_act, w.K_act)
        inst.run_iteration(fused_move=FUSED_MOVE[0])
        out_host["grant"].copy_(inst.grant[:n], non_blocking=True)
        out_host["x1"].copy_(inst.x1[:n], non_blocking=True)
        out_host["x2"].copy_(inst.x2[:n], non_blocking=True)
        out_host["tokens_run"].copy_(inst.tokens_run[:n], non_blocking=True)
        out_host["action"].copy_(inst.action[:n], non_blocking=True)
        out_host["counts"].copy_(inst.plan_counts, non_blocking=True)
        torch.cuda.synchronize()       # the caller needs the plan before it can build the next batch
        return int(out_host["counts"][0]) + int(out_host["counts"][1])

    step(*pinned[0])                    # untimed warm-up of the code path
    torch.cuda.synchronize()
    a, b = event_pair(torch)
    a.record()
    for w, p in pinned:
        moved += step(w, p) * inst.block_bytes
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b)
    return dict(value=round(moved / (ms * 1e-3) / GB, 3), unit="GB/s", h2d_bytes_per_step=int(h2d),
                d2h_bytes_per_step=int(d2h), ms_per_step=round(ms / len(pinned), 4))


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_main(args)
    else:
        ours_main(args)


if __name__ == "__main__":
    main()
