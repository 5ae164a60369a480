"""Device-side state of one serving instance and the five-call iteration over it.

Allocates every tensor the iteration needs (PyTorch as the memory/stream owner), uploads a
``workload.Workload`` and issues the C-ABI calls in stream order:
budget -> schedule -> tier_plan -> kv_evict -> kv_restore.  No host synchronisation happens
between the calls; results are read back only by ``fetch``.
"""
from __future__ import annotations

import numpy as np
import torch

from . import cascade as cs

_REQ_DTYPES = dict(arrival_ns=torch.int64, prompt=torch.int32, pred_out=torch.int32, n0=torch.int32,
                   n1=torch.int32, n2=torch.int32, id=torch.uint32, cls=torch.uint8, flags=torch.uint8)
_NP_DTYPES = dict(arrival_ns=np.int64, prompt=np.int32, pred_out=np.int32, n0=np.int32, n1=np.int32, n2=np.int32,
                  id=np.uint32, cls=np.uint8, flags=np.uint8)


def _to_dev(a: np.ndarray, device, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None and t.dtype != dtype:
        t = t.view(dtype)
    return t.to(device)


class Instance:
    """All device buffers of one scheduler instance.

    ``hbm_pool`` / ``host_pool`` may be passed in (uint8 tensors, device and pinned host); when a
    workload has a layout and none is given they are allocated here, uninitialised."""

    def __init__(self, w, device: str = "cuda:0", max_requests: int | None = None, alloc_pools: bool = True,
                 hbm_pool=None, host_pool=None, ctx: cs.Context | None = None):
        self.device = torch.device(device)
        self.n = w.n
        cap = max_requests or max(w.n, 1)
        self.cap = cap
        dev_index = self.device.index or 0
        self.ctx = ctx or cs.Context(w.params, cap, dev_index)
        if ctx is not None:
            self.ctx.set_params(w.params)
        self.now_ns, self.D_act, self.K_act = w.now_ns, w.D_act, w.K_act
        d = self.device
        # request queue, structure of arrays; a pinned host mirror serves the end-to-end path
        self.reqs = {k: torch.empty(cap, dtype=dt, device=d) for k, dt in _REQ_DTYPES.items()}
        self.reqs_host = {k: torch.empty(cap, dtype=dt, pin_memory=True) for k, dt in _REQ_DTYPES.items()}
        self.reqs_struct = cs.make_reqs(self.reqs)
        self.upload_requests(w.reqs)
        # outputs
        self.budget = torch.empty(cap, dtype=torch.int64, device=d)
        self.key = torch.empty(cap, dtype=torch.uint64, device=d)
        self.order = torch.empty(cap, dtype=torch.uint32, device=d)
        self.grant = torch.empty(cap, dtype=torch.int32, device=d)
        self.sched_counts = torch.zeros(2, dtype=torch.int64, device=d)      # cascade_sched_counts (16 B)
        self.plan_counts = torch.zeros(12, dtype=torch.int32, device=d)      # cascade_plan_counts (48 B)
        self.x1 = torch.empty(cap, dtype=torch.int32, device=d)
        self.x2 = torch.empty(cap, dtype=torch.int32, device=d)
        self.tokens_run = torch.empty(cap, dtype=torch.int32, device=d)
        self.action = torch.empty(cap, dtype=torch.uint8, device=d)
        self.hbm_free_count = torch.tensor([w.hbm_free_count], dtype=torch.int32, device=d)
        self.host_free_count = torch.tensor([w.host_free_count], dtype=torch.int32, device=d)
        self.with_tables = w.hbm_tbl is not None
        self.layout = None
        self.hbm_pool = hbm_pool
        self.host_pool = host_pool
        if self.with_tables:
            self.maxb = w.maxb
            self.hbm_tbl = _to_dev(w.hbm_tbl, d)
            self.host_tbl = _to_dev(w.host_tbl, d)
            self.hbm_free = _to_dev(w.hbm_free, d)
            self.host_free = _to_dev(w.host_free, d)
            self.restore_cap = len(w.hbm_free)
            self.evict_cap = len(w.host_free)
            self.restore_src = torch.full((self.restore_cap,), -1, dtype=torch.int32, device=d)
            self.restore_dst = torch.full((self.restore_cap,), -1, dtype=torch.int32, device=d)
            self.evict_src = torch.full((self.evict_cap,), -1, dtype=torch.int32, device=d)
            self.evict_dst = torch.full((self.evict_cap,), -1, dtype=torch.int32, device=d)
            self.pools_struct = cs.Pools(cs._p(self.hbm_tbl), cs._p(self.host_tbl), self.maxb, cs._p(self.hbm_free),
                                         cs._p(self.hbm_free_count), len(w.hbm_free), cs._p(self.host_free),
                                         cs._p(self.host_free_count), len(w.host_free))
            self.plan_struct = cs.Plan(cs._p(self.x1), cs._p(self.x2), cs._p(self.tokens_run), cs._p(self.action),
                                       cs._p(self.restore_src), cs._p(self.restore_dst), self.restore_cap,
                                       cs._p(self.evict_src), cs._p(self.evict_dst), self.evict_cap,
                                       cs._p(self.plan_counts))
            self.layout_dict = w.layout
            self.layout = cs.make_layout(w.layout)
            self.host_blocks = w.host_blocks
            self.block_bytes = w.block_bytes
            if alloc_pools:
                if self.hbm_pool is None:
                    self.hbm_pool = torch.empty(w.layout["n_blocks"] * self.block_bytes, dtype=torch.uint8, device=d)
                if self.host_pool is None:
                    self.host_pool = torch.empty(w.host_blocks * self.block_bytes, dtype=torch.uint8, pin_memory=True)
        else:
            self.pools_struct = cs.Pools(None, None, 0, None, cs._p(self.hbm_free_count), 0, None,
                                         cs._p(self.host_free_count), 0)
            self.plan_struct = cs.Plan(cs._p(self.x1), cs._p(self.x2), cs._p(self.tokens_run), cs._p(self.action),
                                       None, None, 0, None, None, 0, cs._p(self.plan_counts))

    # -- inputs ---------------------------------------------------------------------------------
    def upload_requests(self, reqs: dict, n: int | None = None, stream=None):
        """Host -> device copy of the whole request queue through the pinned mirror."""
        n = len(reqs["prompt"]) if n is None else n
        self.n = n
        for k, dt in _NP_DTYPES.items():
            src = np.ascontiguousarray(reqs[k], dtype=dt)
            self.reqs_host[k][:n].numpy()[...] = src if dt != np.uint32 else src
            self.reqs[k][:n].copy_(self.reqs_host[k][:n], non_blocking=True)

    def stage_slot_update(self, reqs: dict, slots: np.ndarray) -> int:
        """Write the new values of ``slots`` (taken from the full arrays ``reqs``) into the pinned staging
        arrays; host work only.  Returns the number of bytes the device will read."""
        m = len(slots)
        if not hasattr(self, "upd_host"):
            self.upd_host = {k: torch.empty(self.cap, dtype=dt, pin_memory=True) for k, dt in _REQ_DTYPES.items()}
            self.upd_slots = torch.empty(self.cap, dtype=torch.int32, pin_memory=True)
            self.upd_struct = cs.make_reqs(self.upd_host)
        for k, dt in _NP_DTYPES.items():
            self.upd_host[k][:m].numpy()[...] = np.ascontiguousarray(reqs[k], dtype=dt)[slots]
        self.upd_slots[:m].numpy()[...] = slots
        self.upd_m = m
        return m * (sum(self.reqs[k].element_size() for k in self.reqs) + 4)

    def run_slot_update(self, stream=None):
        """Scatter the staged slots into the device queue (the kernel reads the pinned staging arrays in place)."""
        self.ctx.reqs_update(self.reqs_struct, self.cap, self.upd_struct, self.upd_slots, self.upd_m, stream)

    def request_bytes(self) -> int:
        return sum(self.reqs[k].element_size() for k in self.reqs) * self.n

    def set_clock(self, now_ns: int, D_act: int, K_act: int):
        self.now_ns, self.D_act, self.K_act = now_ns, D_act, K_act

    # -- the path -------------------------------------------------------------------------------
    def run_schedule(self, stream=None):
        """budget -> schedule -> tier plan (three C-ABI calls, stream ordered)."""
        c = self.ctx
        c.budget(self.reqs_struct, self.n, self.now_ns, self.D_act, self.K_act, self.budget, self.key, stream)
        c.schedule(self.reqs_struct, self.key, self.n, self.D_act, self.order, self.grant, self.sched_counts, stream)
        c.tier_plan(self.reqs_struct, self.budget, self.order, self.grant, self.n, self.D_act, self.K_act,
                    self.pools_struct, self.plan_struct, stream)

    def step_args(self, with_update: bool = False, with_move: bool = False) -> cs.StepArgs:
        """The arguments of one whole iteration for cascade_step; the structure points at this instance's buffers
        and is kept alive by it (only clock, load and the update count change from iteration to iteration)."""
        import ctypes as C
        a = cs.StepArgs()
        a.reqs = C.pointer(self.reqs_struct)
        a.n, a.D_act, a.K_act, a.now_ns = self.n, self.D_act, self.K_act, self.now_ns
        if with_update:
            a.upd_src = C.pointer(self.upd_struct)
            a.upd_slots, a.upd_m, a.upd_cap = cs._p(self.upd_slots), self.upd_m, self.cap
        a.budget, a.key, a.order, a.grant = (cs._p(t) for t in (self.budget, self.key, self.order, self.grant))
        a.sched_counts = cs._p(self.sched_counts)
        a.pools, a.plan = C.pointer(self.pools_struct), C.pointer(self.plan_struct)
        if with_move:
            if not hasattr(self, "move_scratch"):
                self.move_scratch = torch.empty(cs.kv_move_scratch_len(self.evict_cap, self.restore_cap),
                                                dtype=torch.int32, device=self.device)
            self._layout_keep = self.layout
            a.layout = C.addressof(self.layout)
            a.hbm_pool, a.host_pool, a.host_blocks = cs._p(self.hbm_pool), cs._p(self.host_pool), self.host_blocks
            a.move_scratch = cs._p(self.move_scratch)
        return a

    def run_step(self, args: cs.StepArgs, stream=None):
        """One cascade_step call with the current clock and load."""
        args.n, args.D_act, args.K_act, args.now_ns = self.n, self.D_act, self.K_act, self.now_ns
        if args.upd_slots:
            args.upd_m = self.upd_m
        self.ctx.step(args, stream)

    def run_prefetch(self, link_budget_ns: int, hbm_reserve: int = 0, stream=None):
        """Budget-bounded prefetch for the requests that stay queued (after run_schedule, before run_copies)."""
        if not hasattr(self, "pf"):
            self.pf = torch.empty(self.cap, dtype=torch.int32, device=self.device)
            self.prefetch_counts = torch.zeros(6, dtype=torch.int32, device=self.device)   # 24-byte struct
        self.ctx.prefetch_plan(self.reqs_struct, self.budget, self.order, self.grant, self.action, self.n, self.D_act,
                               self.K_act, link_budget_ns, hbm_reserve, self.pools_struct, self.plan_struct, self.pf,
                               self.prefetch_counts, stream)

    def fetch_prefetch(self) -> dict:
        torch.cuda.synchronize(self.device)
        c = self.prefetch_counts.cpu().numpy()
        return dict(pf=self.pf[: self.n].cpu().numpy(),
                    counts=dict(n_prefetch=int(c[0]), n_requests=int(c[1]), hbm_free_after=int(c[2]),
                                n_restore_total=int(c[3]), link_ns_left=int(c[4:6].view(np.int64)[0])))

    def run_copies(self, stream=None, record_pool=None, record_is_device: bool = False):
        """evict then restore, with the counts the plan left in device memory."""
        c = self.ctx
        rec = self.host_pool if record_pool is None else record_pool
        n_evict = self.plan_counts[1:2]
        n_restore = self.plan_counts[0:1]
        c.kv_evict(self.layout, self.hbm_pool, rec, self.host_blocks, record_is_device, self.evict_src,
                   self.evict_dst, n_evict, self.evict_cap, stream)
        c.kv_restore(self.layout, self.hbm_pool, rec, self.host_blocks, record_is_device, self.restore_src,
                     self.restore_dst, n_restore, self.restore_cap, stream)

    def run_move(self, stream=None):
        """evict + restore as one call that uses both directions of the host link at once."""
        if not hasattr(self, "move_scratch"):
            self.move_scratch = torch.empty(cs.kv_move_scratch_len(self.evict_cap, self.restore_cap),
                                            dtype=torch.int32, device=self.device)
        self.ctx.kv_move(self.layout, self.hbm_pool, self.host_pool, self.host_blocks, self.evict_src, self.evict_dst,
                         self.plan_counts[1:2], self.evict_cap, self.restore_src, self.restore_dst,
                         self.plan_counts[0:1], self.restore_cap, self.move_scratch, stream)

    def run_move_staged(self, staging, stream=None):
        """evict + restore through the copy engines (one host synchronisation inside the call); ``staging`` is a
        device uint8 tensor of a whole number of blocks."""
        if not hasattr(self, "mailbox"):
            self.mailbox = torch.empty(cs.kv_mailbox_len(self.evict_cap, self.restore_cap), dtype=torch.int32,
                                       pin_memory=True)
        self.ctx.kv_move_staged(self.layout, self.hbm_pool, self.host_pool, self.host_blocks, self.evict_src,
                                self.evict_dst, self.plan_counts[1:2], self.evict_cap, self.restore_src,
                                self.restore_dst, self.plan_counts[0:1], self.restore_cap, staging,
                                staging.numel() // self.block_bytes, self.mailbox, stream)

    # -- deep tier and shared blocks -------------------------------------------------------------
    def enable_deep(self, w, deep_pool=None, alloc_pool: bool = True):
        """Upload the deep-tier table of ``w`` and allocate what the stage plan and the one-copy-per-source
        pass need: the stage list, the merged lists, share counts and the pass's scratch."""
        d = self.device
        self.deep_blocks = w.deep_blocks
        self.deep_tbl = _to_dev(w.deep_tbl, d)
        self.stage_cap = self.evict_cap
        self.stage_src = torch.full((self.stage_cap,), -1, dtype=torch.int32, device=d)
        self.stage_dst = torch.full((self.stage_cap,), -1, dtype=torch.int32, device=d)
        self.staged = torch.zeros(self.cap, dtype=torch.int32, device=d)
        self.stage_counts = torch.zeros(6, dtype=torch.int32, device=d)           # cascade_stage_counts (24 B)
        self.stage_struct = cs.Stage(cs._p(self.deep_tbl), cs._p(self.stage_src), cs._p(self.stage_dst),
                                     self.stage_cap, cs._p(self.staged), cs._p(self.stage_counts))
        self.restore_src_m = torch.full((self.restore_cap,), -1, dtype=torch.int32, device=d)
        self.restore_dst_m = torch.full((self.restore_cap,), -1, dtype=torch.int32, device=d)
        self.stage_src_m = torch.full((self.stage_cap,), -1, dtype=torch.int32, device=d)
        self.stage_dst_m = torch.full((self.stage_cap,), -1, dtype=torch.int32, device=d)
        n_hbm = self.layout_dict["n_blocks"]
        self.hbm_ref = torch.zeros(n_hbm, dtype=torch.int32, device=d)
        self.host_ref = torch.zeros(self.host_blocks, dtype=torch.int32, device=d)
        self.shared_restore = torch.zeros(self.cap, dtype=torch.uint8, device=d)
        self.shared_stage = torch.zeros(self.cap, dtype=torch.uint8, device=d)
        self.dedup_counts_restore = torch.zeros(6, dtype=torch.int32, device=d)
        self.dedup_counts_stage = torch.zeros(6, dtype=torch.int32, device=d)
        len_r = cs.dedup_scratch_len(self.host_blocks, self.restore_cap)
        len_s = cs.dedup_scratch_len(self.deep_blocks, self.stage_cap)
        self.dedup_scratch = torch.empty(max(len_r, len_s), dtype=torch.int32, device=d)
        self.dedup_restore_args = lambda: cs.make_dedup_args(
            lo_a=self.reqs["n0"], lo_b=None, len_a=self.x1, len_b=getattr(self, "pf", None), src_tbl=self.host_tbl,
            dst_tbl=self.hbm_tbl, maxb=self.maxb, list_src=self.restore_src, list_dst=self.restore_dst,
            list_count=self.plan_counts[0:1], list_cap=self.restore_cap, out_src=self.restore_src_m,
            out_dst=self.restore_dst_m, n_src_ids=self.host_blocks, n_dst_ids=n_hbm, free_list=self.hbm_free,
            free_count=self.hbm_free_count, free_cap=len(self.hbm_free), ref=self.hbm_ref, shared=self.shared_restore,
            scratch=self.dedup_scratch, scratch_len=self.dedup_scratch.numel(), counts=self.dedup_counts_restore)
        self.dedup_stage_args = lambda: cs.make_dedup_args(
            lo_a=self.reqs["n0"], lo_b=self.reqs["n1"], len_a=self.staged, len_b=None, src_tbl=self.deep_tbl,
            dst_tbl=self.host_tbl, maxb=self.maxb, list_src=self.stage_src, list_dst=self.stage_dst,
            list_count=self.stage_counts[0:1], list_cap=self.stage_cap, out_src=self.stage_src_m,
            out_dst=self.stage_dst_m, n_src_ids=self.deep_blocks, n_dst_ids=self.host_blocks,
            free_list=self.host_free, free_count=self.host_free_count, free_cap=len(self.host_free),
            ref=self.host_ref, shared=self.shared_stage, scratch=self.dedup_scratch,
            scratch_len=self.dedup_scratch.numel(), counts=self.dedup_counts_stage)
        self.deep_pool = deep_pool
        if deep_pool is None and alloc_pool:
            self.deep_pool = torch.empty(w.deep_blocks * self.block_bytes, dtype=torch.uint8, pin_memory=True)

    def run_stage_plan(self, link_budget_ns: int, host_reserve: int = 0, stream=None):
        """First hop of the deep-tier path for this iteration (after run_schedule)."""
        self.ctx.stage_plan(self.reqs_struct, self.budget, self.order, self.action, self.n, self.D_act, self.K_act,
                            link_budget_ns, host_reserve, self.pools_struct, self.stage_struct, stream)

    def run_dedup_restore(self, stream=None):
        """One copy per shared host block of the restore list (after the plan and the prefetch plan)."""
        self.ctx.dedup(self.dedup_restore_args(), self.n, stream)

    def run_dedup_stage(self, stream=None):
        """One copy per shared deep-tier block of the stage list (after run_stage_plan)."""
        self.ctx.dedup(self.dedup_stage_args(), self.n, stream)

    def run_move_merged(self, stream=None):
        """evict + restore over the merged restore list."""
        if not hasattr(self, "move_scratch"):
            self.move_scratch = torch.empty(cs.kv_move_scratch_len(self.evict_cap, self.restore_cap),
                                            dtype=torch.int32, device=self.device)
        self.ctx.kv_move(self.layout, self.hbm_pool, self.host_pool, self.host_blocks, self.evict_src, self.evict_dst,
                         self.plan_counts[1:2], self.evict_cap, self.restore_src_m, self.restore_dst_m,
                         self.dedup_counts_restore[1:2], self.restore_cap, self.move_scratch, stream)

    def run_stage_copy(self, merged: bool = True, stream=None):
        """deep-tier records -> host records over the (merged) stage list."""
        src, dst = (self.stage_src_m, self.stage_dst_m) if merged else (self.stage_src, self.stage_dst)
        cnt = self.dedup_counts_stage[1:2] if merged else self.stage_counts[0:1]
        self.ctx.kv_stage(self.deep_pool, self.deep_blocks, self.host_pool, self.host_blocks, self.block_bytes, src, dst,
                          cnt, self.stage_cap, stream)

    def run_iteration_deep(self, link_budget_ns: int, host_reserve: int = 0, stream=None):
        """budget -> schedule -> tier plan -> merge the restore list -> stage plan -> merge the stage list ->
        evict + restore -> stage copy.  (The stage copy writes host records that this iteration's restore list
        never reads and its evict list never writes: both came off the free list after them.)"""
        self.run_schedule(stream)
        self.run_dedup_restore(stream)
        self.run_stage_plan(link_budget_ns, host_reserve, stream)
        self.run_dedup_stage(stream)
        self.run_move_merged(stream)
        self.run_stage_copy(True, stream)

    def fetch_deep(self) -> dict:
        torch.cuda.synchronize(self.device)
        n = self.n
        sc = self.stage_counts.cpu().numpy()
        names = ("n_in", "n_unique", "n_surplus", "n_shared_requests", "max_share", "free_after")
        dr = {k: int(v) for k, v in zip(names, self.dedup_counts_restore.cpu().numpy())}
        ds = {k: int(v) for k, v in zip(names, self.dedup_counts_stage.cpu().numpy())}
        ns = min(int(sc[0]), self.stage_cap)
        return dict(staged=self.staged[:n].cpu().numpy(), stage_src=self.stage_src[:ns].cpu().numpy(),
                    stage_dst=self.stage_dst[:ns].cpu().numpy(),
                    stage_counts=dict(n_stage=int(sc[0]), n_requests=int(sc[1]), n_short=int(sc[2]),
                                      host_free_after=int(sc[3]), link_ns_left=int(sc[4:6].view(np.int64)[0])),
                    dedup_restore=dr, dedup_stage=ds,
                    restore_src_m=self.restore_src_m[: dr["n_unique"]].cpu().numpy(),
                    restore_dst_m=self.restore_dst_m[: dr["n_unique"]].cpu().numpy(),
                    stage_src_m=self.stage_src_m[: ds["n_unique"]].cpu().numpy(),
                    stage_dst_m=self.stage_dst_m[: ds["n_unique"]].cpu().numpy(),
                    hbm_ref=self.hbm_ref.cpu().numpy(), host_ref=self.host_ref.cpu().numpy(),
                    shared_restore=self.shared_restore[:n].cpu().numpy(),
                    shared_stage=self.shared_stage[:n].cpu().numpy())

    def run_iteration(self, stream=None, fused_move: bool = False):
        self.run_schedule(stream)
        if self.with_tables and self.hbm_pool is not None:
            if fused_move:
                self.run_move(stream)
            else:
                self.run_copies(stream)

    # -- outputs --------------------------------------------------------------------------------
    def fetch(self) -> dict:
        """Synchronise and bring every result to the host as numpy."""
        torch.cuda.synchronize(self.device)
        n = self.n
        sc = self.sched_counts.cpu().numpy()
        pc = self.plan_counts.cpu().numpy()
        names = ("n_restore", "n_evict", "n_drop_blocks", "n_victims", "n_unadmitted", "n_admitted", "hbm_need",
                 "deficit", "hbm_free_after", "host_free_after")
        plan_counts = {k: int(pc[i]) for i, k in enumerate(names)}
        plan_counts["tokens_run"] = int(pc[10:12].view(np.int64)[0])
        out = dict(
            budget=self.budget[:n].cpu().numpy(), key=self.key[:n].cpu().numpy(),
            order=self.order[:n].cpu().numpy(), grant=self.grant[:n].cpu().numpy(),
            sched_counts=dict(n_tier1=int(sc[0] & 0xFFFFFFFF), n_admitted=int(sc[0] >> 32),
                              tokens_granted=int(sc[1])),
            x1=self.x1[:n].cpu().numpy(), x2=self.x2[:n].cpu().numpy(),
            tokens_run=self.tokens_run[:n].cpu().numpy(), action=self.action[:n].cpu().numpy(),
            plan_counts=plan_counts)
        if self.with_tables:
            nr = min(plan_counts["n_restore"], self.restore_cap)
            ne = min(plan_counts["n_evict"], self.evict_cap)
            out.update(hbm_tbl=self.hbm_tbl.cpu().numpy(), host_tbl=self.host_tbl.cpu().numpy(),
                       hbm_free=self.hbm_free.cpu().numpy(), host_free=self.host_free.cpu().numpy(),
                       hbm_free_count=int(self.hbm_free_count.item()),
                       host_free_count=int(self.host_free_count.item()),
                       restore_src=self.restore_src[:nr].cpu().numpy(), restore_dst=self.restore_dst[:nr].cpu().numpy(),
                       evict_src=self.evict_src[:ne].cpu().numpy(), evict_dst=self.evict_dst[:ne].cpu().numpy())
        out["status"] = self.ctx.status(clear=True)[0]
        return out


def host_memory_available() -> int | None:
    """MemAvailable of the box in bytes (None where /proc/meminfo cannot be read)."""
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return None


def alloc_pinned_pool(nbytes: int, floor: int = 1 << 28, share_of_available: float = 0.7):
    """Pinned, device-mapped host pool of ``nbytes``.  The request is first cut to ``share_of_available`` of
    the box's available memory (page-locking more than the box can spare takes the box down instead of
    failing), then halved until the allocation succeeds.  Returns (uint8 tensor, bytes obtained)."""
    avail = host_memory_available()
    if avail is not None and nbytes > avail * share_of_available:
        nbytes = int(avail * share_of_available) // (1 << 21) * (1 << 21)
    while nbytes >= floor:
        try:
            return torch.empty(nbytes, dtype=torch.uint8, pin_memory=True), nbytes
        except RuntimeError:
            nbytes //= 2
    raise RuntimeError("could not pin a host pool")


def fill_pools(hbm_pool, host_pool):
    """Deterministic, position-dependent byte patterns for both pools, produced on the device in
    256 MiB pieces (the host pool is filled by device-to-host copies)."""
    piece = 1 << 28
    words = torch.arange(piece // 8, dtype=torch.int64, device=hbm_pool.device)
    for base in range(0, hbm_pool.numel(), piece):
        n = min(piece, hbm_pool.numel() - base)
        chunk = words[: n // 8] * -0x61C8864680B583EB + (base * 31 + 1)
        hbm_pool[base:base + (n // 8) * 8].view(torch.int64).copy_(chunk)
    for base in range(0, host_pool.numel(), piece):
        n = min(piece, host_pool.numel() - base)
        chunk = words[: n // 8] * -0x6B2FB644ECCEEE15 + (base * 17 + 2)
        host_pool[base:base + (n // 8) * 8].view(torch.int64).copy_(chunk, non_blocking=True)
    torch.cuda.synchronize()
