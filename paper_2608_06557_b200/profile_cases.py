"""Small, self-contained invocations of single kernels, sized for an `ncu` capture.

    python -m paper_2608_06557_b200.profile_cases copy-hbm   [blocks]   # staging buffer <-> paged pool (HBM bound)
    python -m paper_2608_06557_b200.profile_cases copy-host  [blocks]   # pinned host pool <-> paged pool (host link)
    python -m paper_2608_06557_b200.profile_cases move       [blocks]   # fused evict + restore, both link directions
    python -m paper_2608_06557_b200.profile_cases schedule   [requests] # budget + schedule + tier plan, plan-only
    python -m paper_2608_06557_b200.profile_cases deep       [requests] # whole iteration with the deep-tier stage and
                                                                        # the shared-block merge (16 KiB blocks)

Each case holds at most a few GB on the device, moves more than the 126 MB L2 per launch and
launches its kernel five times, printing the CUDA-event time of every launch.
"""
from __future__ import annotations

import sys

import torch

from . import cascade as cs
from . import workload as wl
from .runner import Instance


def _timed(fn, reps=5):
    out = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        out.append(a.elapsed_time(b) * 1e3)
    return out


def copy_case(record_on_device: bool, n: int):
    n_chunks, chunk_bytes = 64, 32 * 1024
    bb = n_chunks * chunk_bytes
    n_hbm, n_rec = 2 * n + 64, n + 64
    lay = wl.kv_layout(n_hbm, n_chunks, chunk_bytes)
    hbm = torch.empty(n_hbm * bb, dtype=torch.uint8, device="cuda").fill_(1)
    if record_on_device:
        rec = torch.empty(n_rec * bb, dtype=torch.uint8, device="cuda").fill_(2)
    else:
        rec = torch.empty(n_rec * bb, dtype=torch.uint8, pin_memory=True).fill_(2)
    ctx = cs.Context(wl.default_params(), 16, 0)
    layout = cs.make_layout(lay)
    src, dst = wl.copy_lists(7, n, n_rec, n_hbm)
    s, d = torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda()
    torch.cuda.synchronize()
    t_r = _timed(lambda: ctx.kv_restore(layout, hbm, rec, n_rec, record_on_device, s, d, None, n))
    t_e = _timed(lambda: ctx.kv_evict(layout, hbm, rec, n_rec, record_on_device, d, s, None, n))
    mult = 2 if record_on_device else 1
    for name, ts in (("restore", t_r), ("evict", t_e)):
        best = min(ts)
        print(f"{name}: {n} blocks x {bb} B, us per launch {[round(t, 1) for t in ts]}, "
              f"best {mult * n * bb / best / 1e3:.1f} GB/s ({'read+write' if mult == 2 else 'link'} bytes)")
    print("status", ctx.status())


def move_case(n: int):
    """n blocks evicted and n restored by one cascade_kv_move; half of the restores reuse evicted blocks."""
    import numpy as np
    n_chunks, chunk_bytes = 64, 32 * 1024
    bb = n_chunks * chunk_bytes
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
    scratch = torch.empty(2 * n, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    ts = _timed(lambda: ctx.kv_move(layout, hbm, rec, n_rec, t[0], t[1], None, n, t[2], t[3], None, n, scratch))
    print(f"move: {n} evicted + {n} restored blocks x {bb} B, us per call {[round(x, 1) for x in ts]}, "
          f"best {2 * n * bb / min(ts) / 1e3:.1f} GB/s over the link (both directions)")
    print("status", ctx.status())


def schedule_case(n: int):
    sw = wl.SchedulerSweep(n, seed=0)
    inst = Instance(sw.workload(), alloc_pools=False)
    ts = _timed(inst.run_schedule, reps=8)
    print(f"budget+schedule+plan, {n} requests, us per iteration (event-bracketed, launched call by call): "
          f"{[round(t, 1) for t in ts]}")
    print("status", inst.ctx.status())


def deep_case(n: int):
    """Three independent iterations (seeds 0..2) of the shared-prefix workload: plan, merge of the restore
    list, stage plan, merge of the stage list, evict + restore, stage copy."""
    for seed in range(3):
        w = wl.config_deep_shared(seed, n=n, n_hbm=16 * n, n_host=16 * n, n_deep=32 * n, hbm_free_target=8 * n)
        w.params["plan_first"] = 1
        inst = Instance(w)
        inst.enable_deep(w)
        inst.hbm_pool.fill_(1)
        inst.host_pool.fill_(2)
        inst.deep_pool.fill_(3)
        torch.cuda.synchronize()
        ts = _timed(lambda: inst.run_iteration_deep(10**9, 0), reps=1)
        d = inst.fetch_deep()
        print(f"seed {seed}: {n} requests, iteration {ts[0]:.1f} us; restore list {d['dedup_restore']['n_in']} -> "
              f"{d['dedup_restore']['n_unique']}, stage list {d['dedup_stage']['n_in']} -> {d['dedup_stage']['n_unique']}, "
              f"status {inst.ctx.status()}")
        del inst


def main(argv):
    case = argv[1] if len(argv) > 1 else "copy-hbm"
    if case == "copy-hbm":
        copy_case(True, int(argv[2]) if len(argv) > 2 else 256)
    elif case == "copy-host":
        copy_case(False, int(argv[2]) if len(argv) > 2 else 256)
    elif case == "move":
        move_case(int(argv[2]) if len(argv) > 2 else 128)
    elif case == "schedule":
        schedule_case(int(argv[2]) if len(argv) > 2 else 16384)
    elif case == "deep":
        deep_case(int(argv[2]) if len(argv) > 2 else 1024)
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main(sys.argv)
