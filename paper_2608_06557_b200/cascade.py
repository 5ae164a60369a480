"""Thin ctypes binding over libcascade.so (argument marshalling only).

Every step of the path runs in the library's CUDA kernels; there is no CPU fallback.  Importing
this module fails loudly if the library has not been built (``python -m paper_2608_06557_b200.build``).
PyTorch appears only as the owner of device memory, pinned host memory and streams: a tensor
argument is reduced to ``tensor.data_ptr()`` before the call.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcascade.so")

MAX_CLASSES = 8
MAX_REQUESTS = 65536
OK, EINVAL, ERANGE, ECUDA, ENOMEM, ETOOBIG = 0, -1, -2, -3, -4, -5
NOALLOC_MAX_REQUESTS = 8192
ST_EBOUNDS, ST_ENOSPC, ST_ETIMEOUT, ST_EPRECOND, ST_ELISTCAP = 1, 2, 4, 8, 16
FLAG_HBM_PRIVATE, FLAG_RUNNING = 1, 2
ACT_NONE, ACT_RETAIN, ACT_EVICT, ACT_DROP = 0, 1, 2, 3

EXPORTS = ("cascade_create", "cascade_destroy", "cascade_set_params", "cascade_budget", "cascade_schedule",
           "cascade_tier_plan", "cascade_kv_restore", "cascade_kv_evict", "cascade_status", "cascade_version",
           "cascade_tier_plan_noalloc", "cascade_latency_regimes", "cascade_prefetch_plan", "cascade_kv_move",
           "cascade_stage_plan", "cascade_kv_stage", "cascade_dedup", "cascade_reqs_update",
           "cascade_kv_move_scratch_len", "cascade_kv_mailbox_len", "cascade_kv_move_staged", "cascade_step")


class Params(C.Structure):
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


class Reqs(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("arrival_ns", "prompt", "pred_out", "n0", "n1", "n2", "id", "cls", "flags")]


class SchedCounts(C.Structure):
    _fields_ = [("n_tier1", C.c_int32), ("n_admitted", C.c_int32), ("tokens_granted", C.c_int64)]


class PlanCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "n_restore", "n_evict", "n_drop_blocks", "n_victims", "n_unadmitted", "n_admitted", "hbm_need",
        "deficit", "hbm_free_after", "host_free_after")] + [("tokens_run", C.c_int64)]


class Pools(C.Structure):
    _fields_ = [("hbm_tbl", C.c_void_p), ("host_tbl", C.c_void_p), ("maxb", C.c_int32),
                ("hbm_free", C.c_void_p), ("hbm_free_count", C.c_void_p), ("hbm_free_cap", C.c_int32),
                ("host_free", C.c_void_p), ("host_free_count", C.c_void_p), ("host_free_cap", C.c_int32)]


class Plan(C.Structure):
    _fields_ = [("x1", C.c_void_p), ("x2", C.c_void_p), ("tokens_run", C.c_void_p), ("action", C.c_void_p),
                ("restore_src", C.c_void_p), ("restore_dst", C.c_void_p), ("restore_cap", C.c_int32),
                ("evict_src", C.c_void_p), ("evict_dst", C.c_void_p), ("evict_cap", C.c_int32),
                ("counts", C.c_void_p)]


class StageCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_stage", "n_requests", "n_short", "host_free_after")] + \
               [("link_ns_left", C.c_int64)]


class Stage(C.Structure):
    _fields_ = [("deep_tbl", C.c_void_p), ("stage_src", C.c_void_p), ("stage_dst", C.c_void_p),
                ("stage_cap", C.c_int32), ("staged", C.c_void_p), ("counts", C.c_void_p)]


class DedupCounts(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_in", "n_unique", "n_surplus", "n_shared_requests", "max_share",
                                         "free_after")]


class DedupArgs(C.Structure):
    _fields_ = [("lo_a", C.c_void_p), ("lo_b", C.c_void_p), ("len_a", C.c_void_p), ("len_b", C.c_void_p),
                ("src_tbl", C.c_void_p), ("dst_tbl", C.c_void_p), ("maxb", C.c_int32),
                ("list_src", C.c_void_p), ("list_dst", C.c_void_p), ("list_count", C.c_void_p),
                ("list_cap", C.c_int32), ("out_src", C.c_void_p), ("out_dst", C.c_void_p),
                ("n_src_ids", C.c_int32), ("n_dst_ids", C.c_int32), ("free_list", C.c_void_p),
                ("free_count", C.c_void_p), ("free_cap", C.c_int32), ("ref", C.c_void_p), ("shared", C.c_void_p),
                ("scratch", C.c_void_p), ("scratch_len", C.c_int64), ("counts", C.c_void_p)]


def dedup_scratch_len(n_src_ids: int, list_cap: int) -> int:
    """int32 entries cascade_dedup needs in its caller-owned scratch."""
    return 2 * n_src_ids + (list_cap + 1023) // 1024 + 8


def make_dedup_args(**kw) -> DedupArgs:
    """DedupArgs from keyword arguments: tensors become device addresses, integers stay integers."""
    a = DedupArgs()
    for k, ctype in DedupArgs._fields_:
        v = kw.get(k)
        setattr(a, k, _p(v) if ctype is C.c_void_p else int(v))
    return a


class StepArgs(C.Structure):
    _fields_ = [("reqs", C.POINTER(Reqs)), ("n", C.c_int32), ("D_act", C.c_int32), ("K_act", C.c_int64),
                ("now_ns", C.c_int64), ("upd_src", C.POINTER(Reqs)), ("upd_slots", C.c_void_p), ("upd_m", C.c_int32),
                ("upd_cap", C.c_int32), ("budget", C.c_void_p), ("key", C.c_void_p), ("order", C.c_void_p),
                ("grant", C.c_void_p), ("sched_counts", C.c_void_p), ("pools", C.POINTER(Pools)),
                ("plan", C.POINTER(Plan)), ("layout", C.c_void_p), ("hbm_pool", C.c_void_p),
                ("host_pool", C.c_void_p), ("host_blocks", C.c_int64), ("move_scratch", C.c_void_p)]


class KvLayout(C.Structure):
    _fields_ = [("n_blocks", C.c_int64), ("n_chunks", C.c_int32), ("reserved", C.c_int32),
                ("chunk_bytes", C.c_int64), ("chunk_stride", C.c_int64), ("block_stride", C.c_int64)]


class Status(C.Structure):
    _fields_ = [("bits", C.c_uint32), ("cuda_error", C.c_int32)]


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2608_06557_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.cascade_create.argtypes = [C.POINTER(vp), C.POINTER(Params), C.c_int, C.c_int]
    lib.cascade_destroy.argtypes = [vp]
    lib.cascade_destroy.restype = None
    lib.cascade_set_params.argtypes = [vp, C.POINTER(Params)]
    lib.cascade_budget.argtypes = [vp, C.POINTER(Reqs), C.c_int, i64, i32, i64, vp, vp, vp]
    lib.cascade_latency_regimes.argtypes = [vp, C.POINTER(Reqs), C.c_int, i32, i64, vp, vp]
    lib.cascade_prefetch_plan.argtypes = [vp, C.POINTER(Reqs), vp, vp, vp, vp, C.c_int, i32, i64, i64, i32,
                                          C.POINTER(Pools), C.POINTER(Plan), vp, vp, vp]
    lib.cascade_schedule.argtypes = [vp, C.POINTER(Reqs), vp, C.c_int, i32, vp, vp, vp, vp]
    lib.cascade_tier_plan.argtypes = [vp, C.POINTER(Reqs), vp, vp, vp, C.c_int, i32, i64, C.POINTER(Pools),
                                      C.POINTER(Plan), vp]
    lib.cascade_kv_restore.argtypes = [vp, C.POINTER(KvLayout), vp, vp, i64, C.c_int, vp, vp, vp, C.c_int, vp]
    lib.cascade_kv_evict.argtypes = [vp, C.POINTER(KvLayout), vp, vp, i64, C.c_int, vp, vp, vp, C.c_int, vp]
    lib.cascade_status.argtypes = [vp, C.POINTER(Status), C.c_int, vp]
    lib.cascade_kv_move.argtypes = [vp, C.POINTER(KvLayout), vp, vp, i64, vp, vp, vp, C.c_int, vp, vp, vp, C.c_int,
                                    vp, vp]
    lib.cascade_kv_move_scratch_len.argtypes = [C.c_int, C.c_int]
    lib.cascade_kv_mailbox_len.argtypes = [C.c_int, C.c_int]
    lib.cascade_kv_move_staged.argtypes = [vp, C.POINTER(KvLayout), vp, vp, i64, vp, vp, vp, C.c_int, vp, vp, vp, C.c_int,
                                           vp, i64, vp, vp]
    lib.cascade_step.argtypes = [vp, C.POINTER(StepArgs), vp]
    lib.cascade_reqs_update.argtypes = [vp, C.POINTER(Reqs), C.c_int, C.POINTER(Reqs), vp, C.c_int, vp]
    lib.cascade_stage_plan.argtypes = [vp, C.POINTER(Reqs), vp, vp, vp, C.c_int, i32, i64, i64, i32, C.POINTER(Pools),
                                       C.POINTER(Stage), vp]
    lib.cascade_kv_stage.argtypes = [vp, vp, i64, vp, i64, i64, vp, vp, vp, C.c_int, vp]
    lib.cascade_dedup.argtypes = [vp, C.POINTER(DedupArgs), C.c_int, vp]
    lib.cascade_tier_plan_noalloc.argtypes = [C.POINTER(Params), C.POINTER(Reqs), vp, vp, vp, C.c_int, i32, i64,
                                              C.POINTER(Pools), C.POINTER(Plan), vp, vp]
    for name in EXPORTS:
        if name != "cascade_destroy":
            getattr(lib, name).restype = C.c_int
    lib.cascade_kv_move_scratch_len.restype = C.c_int64
    lib.cascade_kv_mailbox_len.restype = C.c_int64
    return lib


_lib = load_library()


def make_params(d: dict) -> Params:
    """Parameter block from a plain dict (keys as in workload.default_params)."""
    p = Params()
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


def make_layout(d: dict) -> KvLayout:
    return KvLayout(int(d["n_blocks"]), int(d["n_chunks"]), 0, int(d["chunk_bytes"]), int(d["chunk_stride"]),
                    int(d["block_stride"]))


def _p(x):
    """Device address of a tensor (or an int address, or None)."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class CascadeError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != OK:
        names = {EINVAL: "CASCADE_EINVAL", ERANGE: "CASCADE_ERANGE", ECUDA: "CASCADE_ECUDA", ENOMEM: "CASCADE_ENOMEM",
                 ETOOBIG: "CASCADE_ETOOBIG"}
        raise CascadeError(f"{what} failed: {names.get(rc, rc)}")


def kv_move_scratch_len(n_evict_max: int, n_restore_max: int) -> int:
    """int32 entries cascade_kv_move needs in its caller-owned scratch."""
    return int(_lib.cascade_kv_move_scratch_len(n_evict_max, n_restore_max))


def kv_mailbox_len(n_evict_max: int, n_restore_max: int) -> int:
    """int32 entries of the pinned mailbox cascade_kv_move_staged publishes the lists into."""
    return int(_lib.cascade_kv_mailbox_len(n_evict_max, n_restore_max))


def make_reqs(t: dict) -> Reqs:
    """Struct of device pointers from a dict of tensors (arrival_ns, prompt, ..., flags)."""
    return Reqs(*[_p(t[k]) for k, _ in Reqs._fields_])


class Context:
    """Owns one cascade_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, params: dict | Params, max_requests: int, device: int = 0):
        self.params = params if isinstance(params, Params) else make_params(params)
        self._h = C.c_void_p()
        _check(_lib.cascade_create(C.byref(self._h), C.byref(self.params), max_requests, device), "cascade_create")
        self.max_requests = max_requests
        self.device = device

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value and _lib is not None:
            _lib.cascade_destroy(self._h)
            self._h = C.c_void_p()

    __del__ = close

    def set_params(self, params: dict | Params):
        new = params if isinstance(params, Params) else make_params(params)
        _check(_lib.cascade_set_params(self._h, C.byref(new)), "cascade_set_params")
        self.params = new

    def reqs_update(self, dst: Reqs, cap, src: Reqs, slots, m, stream=None):
        _check(_lib.cascade_reqs_update(self._h, C.byref(dst), cap, C.byref(src), _p(slots), m, _stream(stream)),
               "cascade_reqs_update")

    def budget(self, reqs: Reqs, n, now_ns, D_act, K_act, budget_out, key_out, stream=None):
        _check(_lib.cascade_budget(self._h, C.byref(reqs), n, now_ns, D_act, K_act, _p(budget_out), _p(key_out),
                                   _stream(stream)), "cascade_budget")

    def latency_regimes(self, reqs: Reqs, n, D_act, K_act, lat4_out, stream=None):
        _check(_lib.cascade_latency_regimes(self._h, C.byref(reqs), n, D_act, K_act, _p(lat4_out), _stream(stream)),
               "cascade_latency_regimes")

    def schedule(self, reqs: Reqs, key, n, D_act, order_out, grant_out, counts_dev, stream=None):
        _check(_lib.cascade_schedule(self._h, C.byref(reqs), _p(key), n, D_act, _p(order_out), _p(grant_out),
                                     _p(counts_dev), _stream(stream)), "cascade_schedule")

    def tier_plan(self, reqs: Reqs, budget, order, grant, n, D_act, K_act, pools: Pools, plan: Plan, stream=None):
        _check(_lib.cascade_tier_plan(self._h, C.byref(reqs), _p(budget), _p(order), _p(grant), n, D_act, K_act,
                                      C.byref(pools), C.byref(plan), _stream(stream)), "cascade_tier_plan")

    def prefetch_plan(self, reqs: Reqs, budget, order, grant, action, n, D_act, K_act, link_budget_ns, hbm_reserve,
                      pools: Pools, plan: Plan, pf_out, counts_dev, stream=None):
        _check(_lib.cascade_prefetch_plan(self._h, C.byref(reqs), _p(budget), _p(order), _p(grant), _p(action), n,
                                          D_act, K_act, link_budget_ns, hbm_reserve, C.byref(pools), C.byref(plan),
                                          _p(pf_out), _p(counts_dev), _stream(stream)), "cascade_prefetch_plan")

    def kv_restore(self, layout: KvLayout, hbm_pool, src_pool, src_blocks, src_is_device, src_ids, dst_ids,
                   n_copies_dev, n_copies_max, stream=None):
        _check(_lib.cascade_kv_restore(self._h, C.byref(layout), _p(hbm_pool), _p(src_pool), src_blocks,
                                       int(src_is_device), _p(src_ids), _p(dst_ids), _p(n_copies_dev), n_copies_max,
                                       _stream(stream)), "cascade_kv_restore")

    def kv_evict(self, layout: KvLayout, hbm_pool, dst_pool, dst_blocks, dst_is_device, src_ids, dst_ids,
                 n_copies_dev, n_copies_max, stream=None):
        _check(_lib.cascade_kv_evict(self._h, C.byref(layout), _p(hbm_pool), _p(dst_pool), dst_blocks,
                                     int(dst_is_device), _p(src_ids), _p(dst_ids), _p(n_copies_dev), n_copies_max,
                                     _stream(stream)), "cascade_kv_evict")

    def kv_move(self, layout: KvLayout, hbm_pool, host_pool, host_blocks, evict_src, evict_dst, n_evict_dev,
                n_evict_max, restore_src, restore_dst, n_restore_dev, n_restore_max, scratch, stream=None):
        _check(_lib.cascade_kv_move(self._h, C.byref(layout), _p(hbm_pool), _p(host_pool), host_blocks,
                                    _p(evict_src), _p(evict_dst), _p(n_evict_dev), n_evict_max, _p(restore_src),
                                    _p(restore_dst), _p(n_restore_dev), n_restore_max, _p(scratch),
                                    _stream(stream)), "cascade_kv_move")

    def kv_move_staged(self, layout: KvLayout, hbm_pool, host_pool, host_blocks, evict_src, evict_dst, n_evict_dev,
                       n_evict_max, restore_src, restore_dst, n_restore_dev, n_restore_max, staging, staging_blocks,
                       mailbox, stream=None):
        _check(_lib.cascade_kv_move_staged(self._h, C.byref(layout), _p(hbm_pool), _p(host_pool), host_blocks,
                                           _p(evict_src), _p(evict_dst), _p(n_evict_dev), n_evict_max,
                                           _p(restore_src), _p(restore_dst), _p(n_restore_dev), n_restore_max,
                                           _p(staging), staging_blocks, _p(mailbox), _stream(stream)),
               "cascade_kv_move_staged")

    def step(self, args: StepArgs, stream=None):
        _check(_lib.cascade_step(self._h, C.byref(args), _stream(stream)), "cascade_step")

    def stage_plan(self, reqs: Reqs, budget, order, action, n, D_act, K_act, link_budget_ns, host_reserve,
                   pools: Pools, stage: Stage, stream=None):
        _check(_lib.cascade_stage_plan(self._h, C.byref(reqs), _p(budget), _p(order), _p(action), n, D_act, K_act,
                                       link_budget_ns, host_reserve, C.byref(pools), C.byref(stage),
                                       _stream(stream)), "cascade_stage_plan")

    def kv_stage(self, deep_pool, deep_blocks, host_pool, host_blocks, block_bytes, src_ids, dst_ids, n_copies_dev,
                 n_copies_max, stream=None):
        _check(_lib.cascade_kv_stage(self._h, _p(deep_pool), deep_blocks, _p(host_pool), host_blocks, block_bytes,
                                     _p(src_ids), _p(dst_ids), _p(n_copies_dev), n_copies_max, _stream(stream)),
               "cascade_kv_stage")

    def dedup(self, args: DedupArgs, n, stream=None):
        _check(_lib.cascade_dedup(self._h, C.byref(args), n, _stream(stream)), "cascade_dedup")

    def status(self, clear: bool = True, stream=None) -> tuple[int, int]:
        st = Status()
        _check(_lib.cascade_status(self._h, C.byref(st), int(clear), _stream(stream)), "cascade_status")
        return int(st.bits), int(st.cuda_error)


def tier_plan_noalloc(params: Params, reqs: Reqs, budget, order, grant, n, D_act, K_act, pools: Pools, plan: Plan,
                      status_dev, stream=None):
    """cascade_tier_plan_noalloc: the tier plan on the library's built-in scratch area, for callers
    that cannot allocate device memory (no context is needed).  ``status_dev`` is a caller-owned
    uint32 device word that receives the CASCADE_ST_* bits.  Raises CascadeError (CASCADE_ETOOBIG)
    when ``n`` exceeds NOALLOC_MAX_REQUESTS."""
    _check(_lib.cascade_tier_plan_noalloc(C.byref(params), C.byref(reqs), _p(budget), _p(order), _p(grant), n,
                                          D_act, K_act, C.byref(pools), C.byref(plan), _p(status_dev),
                                          _stream(stream)), "cascade_tier_plan_noalloc")


def raw():
    """The loaded ctypes library, for tests of the boundary itself."""
    return _lib
