"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not product code).

Only tests, ``__graft_entry__.smoke()`` and the CPU-baseline leg of ``bench.py`` may import
this package.  It compiles ``cascade_oracle.cpp`` with g++ on first use and marshals numpy
arrays to it; none of the method's arithmetic lives here.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_HDR = os.path.join(_HERE, "cascade_oracle.h")
# CASCADE_ORACLE_SRC points the tests at an altered copy of the source (the mutation check of the pins);
# its library is built next to that copy, never over the real one
_SRC = os.environ.get("CASCADE_ORACLE_SRC") or os.path.join(_HERE, "cascade_oracle.cpp")
_LIB = (os.path.splitext(_SRC)[0] + ".so") if os.environ.get("CASCADE_ORACLE_SRC") else os.path.join(_HERE, "liboracle.so")

MAX_CLASSES = 8
FLAG_HBM_PRIVATE, FLAG_RUNNING = 1, 2
ACT_NONE, ACT_RETAIN, ACT_EVICT, ACT_DROP = 0, 1, 2, 3
ST_EBOUNDS, ST_ENOSPC, ST_EPRECOND, ST_ELISTCAP = 1, 2, 8, 16


class OrcParams(C.Structure):
    _fields_ = [
        ("bt", C.c_int32), ("chunk_shift", C.c_int32), ("max_batch", C.c_int32), ("max_ctx_avg", C.c_int32),
        ("gamma_q16", C.c_int32), ("n_classes", C.c_int32), ("token_budget", C.c_int32),
        ("tier2_reserve", C.c_int32),
        ("c_tok_q20", C.c_int64), ("c_attn_q20", C.c_int64), ("c_iter_q20", C.c_int64),
        ("c_dseq_q20", C.c_int64), ("c_dkv_q20", C.c_int64),
        ("delta_ns", C.c_int64 * 3), ("blk_ns", C.c_int64 * 3),
        ("ttft_ns", C.c_int64 * MAX_CLASSES), ("tpot_ns", C.c_int64 * MAX_CLASSES),
        ("policy", C.c_int32), ("plan_first", C.c_int32),
    ]


POLICY_BUDGET, POLICY_FCFS, POLICY_EDF, POLICY_SJF = 0, 1, 2, 3


class OrcSchedCounts(C.Structure):
    _fields_ = [("n_tier1", C.c_int32), ("n_admitted", C.c_int32), ("tokens_granted", C.c_int64)]


class OrcPlanCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "n_restore", "n_evict", "n_drop_blocks", "n_victims", "n_unadmitted", "n_admitted", "hbm_need",
        "deficit", "hbm_free_after", "host_free_after")] + [("tokens_run", C.c_int64)]


def build(force: bool = False) -> str:
    """Compile the oracle into ``oracle/liboracle.so`` (g++ -O2, no SIMD flags)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".{os.getpid()}.tmp"
        extra = os.environ.get("CASCADE_ORACLE_CXXFLAGS", "").split()   # e.g. -fsanitize=undefined for the UB check
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-I", _HERE] + extra +
                              ["-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_restore_time.restype = C.c_int64
        _lib.orc_restore_time.argtypes = [C.POINTER(OrcParams), C.c_int, C.c_int64]
        _lib.orc_max_restorable.restype = C.c_int64
        _lib.orc_max_restorable.argtypes = [C.POINTER(OrcParams), C.c_int, C.c_int64, C.c_int64]
        _lib.orc_plan_cost_q20.restype = C.c_int64
        _lib.orc_plan_cost_q20.argtypes = [C.POINTER(OrcParams), C.c_int32, C.c_int64, C.c_int32, C.c_int32,
                                           C.c_int32, C.c_int32]
        for name in ("orc_budget", "orc_schedule", "orc_tier_plan", "orc_kv_restore", "orc_kv_evict"):
            getattr(_lib, name).restype = C.c_uint32
    return _lib


def make_params(d: dict) -> OrcParams:
    """Build the oracle's parameter block from a plain dict (see workload.default_params)."""
    p = OrcParams()
    for k in ("bt", "chunk_shift", "max_batch", "max_ctx_avg", "gamma_q16", "token_budget", "tier2_reserve",
              "c_tok_q20", "c_attn_q20", "c_iter_q20", "c_dseq_q20", "c_dkv_q20"):
        setattr(p, k, int(d[k]))
    p.n_classes = len(d["ttft_ns"])
    for k in (1, 2):
        p.delta_ns[k] = int(d["delta_ns"][k])
        p.blk_ns[k] = int(d["blk_ns"][k])
    for i, v in enumerate(d["ttft_ns"]):
        p.ttft_ns[i] = int(v)
    for i, v in enumerate(d["tpot_ns"]):
        p.tpot_ns[i] = int(v)
    p.policy = int(d.get("policy", 0))
    p.plan_first = int(d.get("plan_first", 0))
    return p


def _ptr(a, ctype):
    if a is None:
        return C.cast(None, C.POINTER(ctype))
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ctype))


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def restore_time(p: OrcParams, k: int, x: int) -> int:
    return int(lib().orc_restore_time(C.byref(p), k, x))


def max_restorable(p: OrcParams, k: int, rem_ns: int, nk: int) -> int:
    return int(lib().orc_max_restorable(C.byref(p), k, rem_ns, nk))


def plan_cost_q20(p: OrcParams, D_act: int, K_act: int, prompt: int, n0: int, x1: int, x2: int) -> int:
    return int(lib().orc_plan_cost_q20(C.byref(p), D_act, K_act, prompt, n0, x1, x2))


def budget(p: OrcParams, reqs: dict, now_ns: int, D_act: int, K_act: int):
    """Steps B1-B6.  Returns (budget int64[n], key uint64[n], status bits)."""
    n = len(reqs["prompt"])
    out_b = np.empty(n, np.int64)
    out_k = np.empty(n, np.uint64)
    a = {k: _arr(reqs[k], dt) for k, dt in (("arrival_ns", np.int64), ("prompt", np.int32), ("pred_out", np.int32),
                                            ("n0", np.int32), ("n1", np.int32), ("n2", np.int32),
                                            ("id", np.uint32), ("cls", np.uint8))}
    st = lib().orc_budget(C.byref(p), C.c_int(n), _ptr(a["arrival_ns"], C.c_int64), _ptr(a["prompt"], C.c_int32),
                          _ptr(a["pred_out"], C.c_int32), _ptr(a["n0"], C.c_int32), _ptr(a["n1"], C.c_int32),
                          _ptr(a["n2"], C.c_int32), _ptr(a["id"], C.c_uint32), _ptr(a["cls"], C.c_uint8),
                          C.c_int64(now_ns), C.c_int32(D_act), C.c_int64(K_act),
                          _ptr(out_b, C.c_int64), _ptr(out_k, C.c_uint64))
    return out_b, out_k, int(st)


def latency_regimes(p: OrcParams, reqs: dict, D_act: int, K_act: int):
    """The estimator's four regimes, int64 [n, 4] (ns).  Returns (array, status bits)."""
    n = len(reqs["prompt"])
    a = {k: _arr(reqs[k], np.int32) for k in ("prompt", "n0", "n1", "n2")}
    out = np.empty((n, 4), np.int64)
    lib().orc_latency_regimes.restype = C.c_uint32
    st = lib().orc_latency_regimes(C.byref(p), C.c_int(n), _ptr(a["prompt"], C.c_int32), _ptr(a["n0"], C.c_int32),
                                   _ptr(a["n1"], C.c_int32), _ptr(a["n2"], C.c_int32), C.c_int32(D_act),
                                   C.c_int64(K_act), _ptr(out, C.c_int64))
    return out, int(st)


def schedule(p: OrcParams, reqs: dict, key: np.ndarray, D_act: int, budget_: np.ndarray | None = None, K_act: int = 0):
    """Steps S1-S3.  Returns (order uint32[n], grant int32[n], counts dict, status bits).
    ``budget_`` and ``K_act`` are needed only when the parameters select plan-first admission."""
    n = len(reqs["prompt"])
    order = np.empty(n, np.uint32)
    grant = np.empty(n, np.int32)
    cnt = OrcSchedCounts()
    a = {k: _arr(reqs[k], np.int32) for k in ("prompt", "n0", "n1", "n2")}
    key = _arr(key, np.uint64)
    st = lib().orc_schedule(C.byref(p), C.c_int(n), _ptr(key, C.c_uint64), _ptr(a["prompt"], C.c_int32),
                            _ptr(a["n0"], C.c_int32), _ptr(a["n1"], C.c_int32), _ptr(a["n2"], C.c_int32),
                            C.c_int32(D_act), _ptr(order, C.c_uint32), _ptr(grant, C.c_int32), C.byref(cnt),
                            _ptr(None if budget_ is None else _arr(budget_, np.int64), C.c_int64), C.c_int64(K_act))
    counts = {k: int(getattr(cnt, k)) for k, _ in OrcSchedCounts._fields_}
    return order, grant, counts, int(st)


@dataclass
class Pools:
    """Block tables and free lists (numpy, modified in place by tier_plan)."""
    hbm_tbl: np.ndarray | None        # int32 [n, maxb], -1 = no block
    host_tbl: np.ndarray | None       # int32 [n, maxb]
    hbm_free: np.ndarray | None       # int32 [hbm_free_cap]; a stack, top = [count-1]
    hbm_free_count: int = 0
    host_free: np.ndarray | None = None
    host_free_count: int = 0
    restore_cap: int = 0
    evict_cap: int = 0
    extra: dict = field(default_factory=dict)


def tier_plan(p: OrcParams, reqs: dict, budget_: np.ndarray, order: np.ndarray, grant: np.ndarray,
              D_act: int, K_act: int, pools: Pools):
    """Steps P1-P6 and K1.  ``grant`` and ``pools`` are updated in place.

    Returns a dict with x1, x2, tokens_run, action, restore_src/dst, evict_src/dst (trimmed to
    their counts), counts and status bits."""
    n = len(reqs["prompt"])
    a = {k: _arr(reqs[k], np.int32) for k in ("prompt", "n0", "n1", "n2")}
    flags = _arr(reqs["flags"], np.uint8)
    budget_ = _arr(budget_, np.int64)
    order = _arr(order, np.uint32)
    assert grant.dtype == np.int32 and grant.flags["C_CONTIGUOUS"]
    x1 = np.empty(n, np.int32)
    x2 = np.empty(n, np.int32)
    run = np.empty(n, np.int32)
    action = np.empty(n, np.uint8)
    with_tables = pools.hbm_tbl is not None
    maxb = pools.hbm_tbl.shape[1] if with_tables else 0
    rs = np.full(max(pools.restore_cap, 1), -1, np.int32)
    rd = np.full(max(pools.restore_cap, 1), -1, np.int32)
    es = np.full(max(pools.evict_cap, 1), -1, np.int32)
    ed = np.full(max(pools.evict_cap, 1), -1, np.int32)
    hc = C.c_int32(pools.hbm_free_count)
    oc = C.c_int32(pools.host_free_count)
    cnt = OrcPlanCounts()
    st = lib().orc_tier_plan(
        C.byref(p), C.c_int(n), _ptr(a["prompt"], C.c_int32), _ptr(a["n0"], C.c_int32), _ptr(a["n1"], C.c_int32),
        _ptr(a["n2"], C.c_int32), _ptr(flags, C.c_uint8), _ptr(budget_, C.c_int64), _ptr(order, C.c_uint32),
        _ptr(grant, C.c_int32), C.c_int32(D_act), C.c_int64(K_act),
        _ptr(pools.hbm_tbl, C.c_int32), _ptr(pools.host_tbl, C.c_int32), C.c_int32(maxb),
        _ptr(pools.hbm_free, C.c_int32), C.byref(hc),
        C.c_int32(0 if pools.hbm_free is None else len(pools.hbm_free)),
        _ptr(pools.host_free, C.c_int32), C.byref(oc),
        C.c_int32(0 if pools.host_free is None else len(pools.host_free)),
        _ptr(x1, C.c_int32), _ptr(x2, C.c_int32), _ptr(run, C.c_int32), _ptr(action, C.c_uint8),
        _ptr(rs, C.c_int32), _ptr(rd, C.c_int32), C.c_int32(pools.restore_cap),
        _ptr(es, C.c_int32), _ptr(ed, C.c_int32), C.c_int32(pools.evict_cap), C.byref(cnt))
    pools.hbm_free_count = int(hc.value)
    pools.host_free_count = int(oc.value)
    counts = {k: int(getattr(cnt, k)) for k, _ in OrcPlanCounts._fields_}
    nr = min(counts["n_restore"], pools.restore_cap)
    ne = min(counts["n_evict"], pools.evict_cap)
    return dict(x1=x1, x2=x2, tokens_run=run, action=action, restore_src=rs[:nr], restore_dst=rd[:nr],
                evict_src=es[:ne], evict_dst=ed[:ne], counts=counts, status=int(st))


class OrcPrefetchCounts(C.Structure):
    _fields_ = [("n_prefetch", C.c_int32), ("n_requests", C.c_int32), ("hbm_free_after", C.c_int32),
                ("n_restore_total", C.c_int32), ("link_ns_left", C.c_int64)]


def prefetch_plan(p: OrcParams, reqs: dict, budget_: np.ndarray, order: np.ndarray, grant: np.ndarray,
                  action: np.ndarray, x1: np.ndarray, D_act: int, K_act: int, link_budget_ns: int, hbm_reserve: int,
                  pools: Pools, restore_src: np.ndarray, restore_dst: np.ndarray, n_restore: int | None = None):
    """Budget-bounded prefetch for queued requests.  ``pools`` (HBM table, HBM free list and its count) is
    updated in place; the restore list passed in is extended.  Returns a dict with pf (blocks per request),
    the extended restore_src/dst, counts and status bits."""
    n = len(reqs["prompt"])
    a = {k: _arr(reqs[k], np.int32) for k in ("prompt", "n0", "n1", "n2")}
    with_tables = pools.hbm_tbl is not None
    maxb = pools.hbm_tbl.shape[1] if with_tables else 0
    cap = max(pools.restore_cap, 1)
    rs = np.full(cap, -1, np.int32)
    rd = np.full(cap, -1, np.int32)
    rs[: len(restore_src)] = restore_src
    rd[: len(restore_dst)] = restore_dst
    nrest = C.c_int32(len(restore_src) if n_restore is None else n_restore)
    hc = C.c_int32(pools.hbm_free_count)
    pf = np.empty(n, np.int32)
    cnt = OrcPrefetchCounts()
    lib().orc_prefetch_plan.restype = C.c_uint32
    st = lib().orc_prefetch_plan(
        C.byref(p), C.c_int(n), _ptr(a["prompt"], C.c_int32), _ptr(a["n0"], C.c_int32), _ptr(a["n1"], C.c_int32),
        _ptr(a["n2"], C.c_int32), _ptr(_arr(budget_, np.int64), C.c_int64), _ptr(_arr(order, np.uint32), C.c_uint32),
        _ptr(_arr(grant, np.int32), C.c_int32), _ptr(_arr(action, np.uint8), C.c_uint8),
        _ptr(_arr(x1, np.int32), C.c_int32), C.c_int32(D_act), C.c_int64(K_act), C.c_int64(link_budget_ns),
        C.c_int32(hbm_reserve), _ptr(pools.hbm_tbl, C.c_int32), _ptr(pools.host_tbl, C.c_int32), C.c_int32(maxb),
        _ptr(pools.hbm_free, C.c_int32), C.byref(hc),
        C.c_int32(0 if pools.hbm_free is None else len(pools.hbm_free)),
        _ptr(rs, C.c_int32), _ptr(rd, C.c_int32), C.c_int32(pools.restore_cap), C.byref(nrest),
        _ptr(pf, C.c_int32), C.byref(cnt))
    pools.hbm_free_count = int(hc.value)
    counts = {k: int(getattr(cnt, k)) for k, _ in OrcPrefetchCounts._fields_}
    nr = min(counts["n_restore_total"], pools.restore_cap)
    return dict(pf=pf, restore_src=rs[:nr], restore_dst=rd[:nr], counts=counts, status=int(st))


def _layout_args(layout: dict):
    return (C.c_int64(layout["n_blocks"]), C.c_int32(layout["n_chunks"]), C.c_int64(layout["chunk_bytes"]),
            C.c_int64(layout["chunk_stride"]), C.c_int64(layout["block_stride"]))


def kv_restore(hbm_pool: np.ndarray, layout: dict, host_pool: np.ndarray, host_blocks: int,
               src_ids: np.ndarray, dst_ids: np.ndarray) -> int:
    """Step K2, host record -> paged HBM block, on uint8 numpy mirrors of the pools."""
    src = _arr(src_ids, np.int32)
    dst = _arr(dst_ids, np.int32)
    assert hbm_pool.dtype == np.uint8 and host_pool.dtype == np.uint8
    return int(lib().orc_kv_restore(_ptr(hbm_pool, C.c_uint8), *_layout_args(layout), _ptr(host_pool, C.c_uint8),
                                    C.c_int64(host_blocks), _ptr(src, C.c_int32), _ptr(dst, C.c_int32),
                                    C.c_int(len(src))))


def kv_evict(hbm_pool: np.ndarray, layout: dict, host_pool: np.ndarray, host_blocks: int,
             src_ids: np.ndarray, dst_ids: np.ndarray) -> int:
    """Step K2, paged HBM block -> host record."""
    src = _arr(src_ids, np.int32)
    dst = _arr(dst_ids, np.int32)
    assert hbm_pool.dtype == np.uint8 and host_pool.dtype == np.uint8
    return int(lib().orc_kv_evict(_ptr(hbm_pool, C.c_uint8), *_layout_args(layout), _ptr(host_pool, C.c_uint8),
                                  C.c_int64(host_blocks), _ptr(src, C.c_int32), _ptr(dst, C.c_int32),
                                  C.c_int(len(src))))


class OrcStageCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_stage", "n_requests", "n_short", "host_free_after")] + \
               [("link_ns_left", C.c_int64)]


def stage_plan(p: OrcParams, reqs: dict, budget_: np.ndarray, order: np.ndarray, action: np.ndarray, D_act: int,
               K_act: int, link_budget_ns: int, host_reserve: int, pools: Pools, deep_tbl: np.ndarray | None,
               stage_cap: int):
    """First hop of the deep-tier path.  ``pools.host_tbl`` and the host free count are updated in place.
    Returns a dict with staged (blocks per slot), stage_src/dst (trimmed), counts and status bits."""
    n = len(reqs["prompt"])
    a = {k: _arr(reqs[k], np.int32) for k in ("prompt", "n0", "n1", "n2")}
    with_tables = pools.host_tbl is not None
    maxb = pools.host_tbl.shape[1] if with_tables else 0
    ss = np.full(max(stage_cap, 1), -1, np.int32)
    sd = np.full(max(stage_cap, 1), -1, np.int32)
    staged = np.empty(n, np.int32)
    oc = C.c_int32(pools.host_free_count)
    cnt = OrcStageCounts()
    lib().orc_stage_plan.restype = C.c_uint32
    st = lib().orc_stage_plan(
        C.byref(p), C.c_int(n), _ptr(a["prompt"], C.c_int32), _ptr(a["n0"], C.c_int32), _ptr(a["n1"], C.c_int32),
        _ptr(a["n2"], C.c_int32), _ptr(_arr(budget_, np.int64), C.c_int64), _ptr(_arr(order, np.uint32), C.c_uint32),
        _ptr(_arr(action, np.uint8), C.c_uint8), C.c_int32(D_act), C.c_int64(K_act), C.c_int64(link_budget_ns),
        C.c_int32(host_reserve), _ptr(pools.host_tbl, C.c_int32), _ptr(deep_tbl, C.c_int32), C.c_int32(maxb),
        _ptr(pools.host_free, C.c_int32), C.byref(oc),
        C.c_int32(0 if pools.host_free is None else len(pools.host_free)), _ptr(ss, C.c_int32), _ptr(sd, C.c_int32),
        C.c_int32(stage_cap), _ptr(staged, C.c_int32), C.byref(cnt))
    pools.host_free_count = int(oc.value)
    counts = {k: int(getattr(cnt, k)) for k, _ in OrcStageCounts._fields_}
    ns = min(counts["n_stage"], stage_cap)
    return dict(staged=staged, stage_src=ss[:ns], stage_dst=sd[:ns], counts=counts, status=int(st))


class OrcDedupCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_in", "n_unique", "n_surplus", "n_shared_requests", "max_share",
                                         "free_after")]


def dedup(lo_a, lo_b, len_a, len_b, src_tbl: np.ndarray, dst_tbl: np.ndarray, list_src, list_dst, list_count: int,
          n_src_ids: int, n_dst_ids: int, free_list: np.ndarray, free_count: int, ref: np.ndarray):
    """One copy per distinct source block.  ``dst_tbl``, ``free_list`` and ``ref`` are updated in place.
    Returns a dict with out_src/out_dst (trimmed), shared (per slot), free_count, counts and status bits."""
    n, maxb = src_tbl.shape
    assert dst_tbl.shape == src_tbl.shape and dst_tbl.dtype == np.int32 and dst_tbl.flags["C_CONTIGUOUS"]
    assert free_list.dtype == np.int32 and ref.dtype == np.int32
    ls, ld = _arr(list_src, np.int32), _arr(list_dst, np.int32)
    cap = len(ls)
    os_ = np.full(max(cap, 1), -1, np.int32)
    od = np.full(max(cap, 1), -1, np.int32)
    shared = np.empty(n, np.uint8)
    fc = C.c_int32(free_count)
    cnt = OrcDedupCounts()
    lib().orc_dedup.restype = C.c_uint32
    st = lib().orc_dedup(
        C.c_int(n), _ptr(_arr(lo_a, np.int32), C.c_int32), _ptr(None if lo_b is None else _arr(lo_b, np.int32), C.c_int32),
        _ptr(_arr(len_a, np.int32), C.c_int32), _ptr(None if len_b is None else _arr(len_b, np.int32), C.c_int32),
        _ptr(_arr(src_tbl, np.int32), C.c_int32), _ptr(dst_tbl, C.c_int32), C.c_int32(maxb), _ptr(ls, C.c_int32),
        _ptr(ld, C.c_int32), C.c_int32(list_count), C.c_int32(cap), _ptr(os_, C.c_int32), _ptr(od, C.c_int32),
        C.c_int32(n_src_ids), C.c_int32(n_dst_ids), _ptr(free_list, C.c_int32), C.byref(fc),
        C.c_int32(len(free_list)), _ptr(ref, C.c_int32), _ptr(shared, C.c_uint8), C.byref(cnt))
    counts = {k: int(getattr(cnt, k)) for k, _ in OrcDedupCounts._fields_}
    nu = counts["n_unique"]
    return dict(out_src=os_[:nu], out_dst=od[:nu], shared=shared, free_count=int(fc.value), counts=counts,
                status=int(st))


def kv_stage(deep_pool: np.ndarray, deep_blocks: int, host_pool: np.ndarray, host_blocks: int, block_bytes: int,
             src_ids: np.ndarray, dst_ids: np.ndarray) -> int:
    """Deep-tier record -> host record (both pools record-major)."""
    src = _arr(src_ids, np.int32)
    dst = _arr(dst_ids, np.int32)
    assert deep_pool.dtype == np.uint8 and host_pool.dtype == np.uint8
    lib().orc_kv_stage.restype = C.c_uint32
    return int(lib().orc_kv_stage(_ptr(deep_pool, C.c_uint8), C.c_int64(deep_blocks), _ptr(host_pool, C.c_uint8),
                                  C.c_int64(host_blocks), C.c_int64(block_bytes), _ptr(src, C.c_int32),
                                  _ptr(dst, C.c_int32), C.c_int(len(src))))
