"""Shared test plumbing: run one iteration of a Workload through the CPU oracle."""
import copy

import numpy as np

import oracle


def oracle_iteration(w, with_tables=True, restore_cap=None, evict_cap=None):
    """budget -> schedule -> tier plan on the oracle.  Returns a dict of every output; the
    workload's tables and free lists are copied first, so ``w`` itself is left untouched."""
    p = oracle.make_params(w.params)
    budget, key, st_b = oracle.budget(p, w.reqs, w.now_ns, w.D_act, w.K_act)
    order, grant, sc, st_s = oracle.schedule(p, w.reqs, key, w.D_act, budget, w.K_act)
    grant_sched = grant.copy()
    if with_tables and w.hbm_tbl is not None:
        pools = oracle.Pools(hbm_tbl=w.hbm_tbl.copy(), host_tbl=w.host_tbl.copy(), hbm_free=w.hbm_free.copy(),
                             hbm_free_count=w.hbm_free_count, host_free=w.host_free.copy(),
                             host_free_count=w.host_free_count,
                             restore_cap=restore_cap if restore_cap is not None else len(w.hbm_free),
                             evict_cap=evict_cap if evict_cap is not None else len(w.host_free))
    else:
        pools = oracle.Pools(None, None, None, w.hbm_free_count, None, w.host_free_count, 0, 0)
    plan = oracle.tier_plan(p, w.reqs, budget, order, grant, w.D_act, w.K_act, pools)
    return dict(budget=budget, key=key, order=order, grant_sched=grant_sched, grant=grant, sched_counts=sc,
                plan=plan, pools=pools, status=st_b | st_s | plan["status"])


def clone_workload(w):
    return copy.deepcopy(w)


def guard_pattern(n_bytes, tag):
    return np.full(n_bytes, tag, np.uint8)


def load_gpu_filler():
    """Builds (if needed) and loads tests/gpu_filler.cu: a test-only kernel that keeps SMs busy for a
    bounded time.  Returns the ctypes library."""
    import ctypes
    import os
    import subprocess
    here = os.path.dirname(os.path.abspath(__file__))
    src, lib = os.path.join(here, "gpu_filler.cu"), os.path.join(here, "libgpu_filler.so")
    if not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(src):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = lib + f".{os.getpid()}.tmp"
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-shared", "-Xcompiler",
                               "-fPIC", "-o", tmp, src])
        os.replace(tmp, lib)
    f = ctypes.CDLL(lib)
    f.filler_launch.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p]
    f.filler_launch.restype = ctypes.c_int
    return f
