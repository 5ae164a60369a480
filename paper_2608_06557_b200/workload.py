"""Seeded synthetic workloads for the Cascade scheduling + KV-tier step.

This module only DRAWS inputs (numpy, ``default_rng(seed)``): request arrays, class tables,
block tables, free lists, copy lists and pool byte patterns.  It holds none of the method's
arithmetic and is the one module shared by the CUDA tests/bench and the CPU oracle's tests.

The paper evaluates on production traces that are not available here; these inputs stand in
for them with the same kind of structure: heterogeneous (lognormal) prompt and output
lengths, mixed SLO classes, partial prefix reuse split between HBM and host DRAM.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

Q20 = 1 << 20
FLAG_HBM_PRIVATE, FLAG_RUNNING = 1, 2
MS = 1_000_000
S = 1_000_000_000


def default_params(**over) -> dict:
    """Cost-model and policy parameters (synthetic; the paper prints no coefficients)."""
    d = dict(
        bt=16, chunk_shift=9, max_batch=128, max_ctx_avg=2048, gamma_q16=81920,
        token_budget=2048, tier2_reserve=256,
        c_tok_q20=50_000 * Q20, c_attn_q20=Q20 // 2, c_iter_q20=2_000_000 * Q20,
        c_dseq_q20=10_000 * Q20, c_dkv_q20=20 * Q20,
        delta_ns=[0, 10_000, 110_000], blk_ns=[0, 40_000, 340_000],
        ttft_ns=[1 * S], tpot_ns=[50 * MS],
    )
    d.update(over)
    return d


def kv_layout(n_blocks: int, n_chunks: int, chunk_bytes: int) -> dict:
    """Layer-major paged HBM pool: chunk c of block b at c*chunk_stride + b*block_stride."""
    return dict(n_blocks=n_blocks, n_chunks=n_chunks, chunk_bytes=chunk_bytes,
                chunk_stride=n_blocks * chunk_bytes, block_stride=chunk_bytes)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Counter-based 64-bit mixer used for pool byte patterns (uint64 in, uint64 out)."""
    x = (x + np.uint64(0x9E3779B97F4A7C15)).astype(np.uint64)
    x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return x ^ (x >> np.uint64(31))


def pool_bytes(tag: int, n_bytes: int) -> np.ndarray:
    """Deterministic byte pattern of a pool: word i = splitmix64(tag * 2^40 + i)."""
    assert n_bytes % 8 == 0
    with np.errstate(over="ignore"):
        w = splitmix64(np.arange(n_bytes // 8, dtype=np.uint64) + (np.uint64(tag) << np.uint64(40)))
    return w.view(np.uint8)


@dataclass
class Workload:
    """One iteration's inputs.  Arrays are host numpy; the caller moves them where needed."""
    name: str
    params: dict
    reqs: dict                    # arrival_ns i64, prompt/pred_out/n0/n1/n2 i32, id u32, cls/flags u8
    now_ns: int
    D_act: int
    K_act: int
    layout: dict | None = None    # HBM pool layout
    host_blocks: int = 0
    maxb: int = 0
    hbm_tbl: np.ndarray | None = None
    host_tbl: np.ndarray | None = None
    hbm_free: np.ndarray | None = None   # stack storage sized to the pool; top = [count-1]
    hbm_free_count: int = 0
    host_free: np.ndarray | None = None
    host_free_count: int = 0
    notes: dict = field(default_factory=dict)
    deep_tbl: np.ndarray | None = None   # int32 [n, maxb]: deep-tier record of table positions n0+n1 .. n0+n1+n2
    deep_blocks: int = 0

    @property
    def n(self) -> int:
        return len(self.reqs["prompt"])

    @property
    def block_bytes(self) -> int:
        return self.layout["n_chunks"] * self.layout["chunk_bytes"]


def _lognormal_int(rng, median, sigma, lo, hi, n):
    v = np.exp(rng.normal(np.log(median), sigma, n))
    return np.clip(np.rint(v), lo, hi).astype(np.int32)


def draw_requests(rng, n, class_mix, ttft_ns, prompt_median, prompt_clip, out_median_by_class, out_clip,
                  now_ns, elapsed_scale, hit_draw, hbm_share, bt, id0=0):
    """Request fields of the SoA arrays.  ``hit_draw(rng, n)`` gives the reused fraction in [0,1];
    ``hbm_share`` of the reused blocks sit in HBM (the head of the prefix), the rest on host."""
    cls = rng.choice(len(class_mix), size=n, p=np.asarray(class_mix, float)).astype(np.uint8)
    prompt = _lognormal_int(rng, prompt_median, 1.0, prompt_clip[0], prompt_clip[1], n)
    med = np.asarray(out_median_by_class, float)[cls]
    pred_out = np.clip(np.rint(np.exp(rng.normal(np.log(med), 1.0))), out_clip[0], out_clip[1]).astype(np.int32)
    if elapsed_scale is None:          # C1: uniform in [0, 2 s]
        elapsed = rng.uniform(0, 2 * S, n)
    else:                              # uniform in [0, elapsed_scale * TTFT_c]
        elapsed = rng.uniform(0, 1, n) * elapsed_scale * np.asarray(ttft_ns, float)[cls]
    arrival = (now_ns - np.rint(elapsed)).astype(np.int64)
    frac = hit_draw(rng, n)
    max_hit = (prompt - 1) // bt       # at least one prompt token is always computed
    hit = np.minimum(np.floor(frac * (prompt // bt)).astype(np.int64), max_hit).astype(np.int32)
    n0 = np.ceil(hit * hbm_share).astype(np.int32)
    n0 = np.minimum(n0, hit)
    n1 = (hit - n0).astype(np.int32)
    n2 = np.zeros(n, np.int32)
    ids = (np.arange(n, dtype=np.uint32) + np.uint32(id0))
    flags = np.zeros(n, np.uint8)
    return dict(arrival_ns=arrival, prompt=prompt, pred_out=pred_out, n0=n0, n1=n1, n2=n2, id=ids, cls=cls,
                flags=flags)


def place_blocks(rng, reqs, n_hbm, n_host, maxb, occupancy, hbm_free_target, private_prob):
    """Give every hit block an id, request by request, until a pool reaches ``occupancy``; later hits
    in that tier are truncated.  Then other tenants' blocks are taken out of the HBM free list until
    ``hbm_free_target`` ids are left.  Returns tables and free-list stacks."""
    n = len(reqs["prompt"])
    hbm_ids = rng.permutation(n_hbm).astype(np.int32)
    host_ids = rng.permutation(n_host).astype(np.int32)
    hbm_lim, host_lim = int(n_hbm * occupancy), int(n_host * occupancy)
    hbm_used = host_used = 0
    hbm_tbl = np.full((n, maxb), -1, np.int32)
    host_tbl = np.full((n, maxb), -1, np.int32)
    n0, n1 = reqs["n0"], reqs["n1"]
    for r in range(n):
        a = min(int(n0[r]), hbm_lim - hbm_used)
        if a < n0[r]:                  # HBM prefix cut short: the host part would not be contiguous
            n0[r], n1[r] = a, 0
        hbm_tbl[r, :a] = hbm_ids[hbm_used:hbm_used + a]
        hbm_used += a
        b = min(int(n1[r]), host_lim - host_used)
        n1[r] = b
        host_tbl[r, a:a + b] = host_ids[host_used:host_used + b]
        host_used += b
    has = n0 > 0
    private = has & (rng.uniform(0, 1, n) < private_prob)
    reqs["flags"][private] |= FLAG_HBM_PRIVATE | FLAG_RUNNING
    hbm_free_count = min(n_hbm - hbm_used, hbm_free_target)
    hbm_free = np.full(n_hbm, -1, np.int32)
    hbm_free[:hbm_free_count] = hbm_ids[n_hbm - hbm_free_count:]
    host_free_count = n_host - host_used
    host_free = np.full(n_host, -1, np.int32)
    host_free[:host_free_count] = host_ids[host_used:]
    return hbm_tbl, host_tbl, hbm_free, hbm_free_count, host_free, host_free_count


def config_tiny(seed: int = 0, hbm_free_target: int = 32) -> Workload:
    """64 requests, two SLO classes, 16 KiB blocks, 512+512 block pools, one iteration."""
    rng = np.random.default_rng(seed)
    ttft = [S // 2, 5 * S]
    params = default_params(ttft_ns=ttft, tpot_ns=[50 * MS, 50 * MS], token_budget=2048, tier2_reserve=256,
                            max_batch=128)
    bb = 16384  # 2 layers x (K,V) x 2 KV heads x 64 dim x 2 B (bf16) x 16 tokens = 16 KiB
    n_chunks, chunk_bytes = 4, bb // 4
    params["blk_ns"] = [0, -(-bb * 1_000_000_000 // 50_000_000_000), 340_000]
    now = 10 * S
    reqs = draw_requests(rng, 64, [0.5, 0.5], ttft, 256, (16, 2048), [128, 128], (1, 4096), now, None,
                         lambda g, n: g.uniform(0, 1, n), 0.5, params["bt"])
    maxb = 128
    tbl = place_blocks(rng, reqs, 512, 512, maxb, 1.0, hbm_free_target, 0.5)
    return Workload("tiny", params, reqs, now, 8, 8 * 512, kv_layout(512, n_chunks, chunk_bytes), 512, maxb, *tbl)


def config_deep_shared(seed: int = 0, n: int = 256, n_hbm: int = 4096, n_host: int = 4096, n_deep: int = 8192,
                       group_frac: float = 0.4, hbm_free_target: int = 2048, host_free_target: int = 1 << 30,
                       n_chunks: int = 4, chunk_bytes: int = 4096) -> Workload:
    """Matched prefixes that reach into the deep tier, with shared prefixes.

    Every request reuses a uniform fraction of its prompt, split 30 % HBM / 35 % host / 35 % deep tier (head
    to tail).  ``group_frac`` of the requests form prefix groups of 2 to 6: a group's members hold nothing in
    HBM, and their host and deep table cells hold the SAME record ids as the group leader's over the length
    they share with it (a member's match may stop anywhere inside the leader's)."""
    rng = np.random.default_rng(seed)
    ttft = [2 * S, 20 * S]
    params = default_params(ttft_ns=ttft, tpot_ns=[50 * MS, 50 * MS], token_budget=4096, tier2_reserve=512,
                            max_batch=128)
    bb = n_chunks * chunk_bytes
    host_blk = -(-bb * 1_000_000_000 // 50_000_000_000)
    params["blk_ns"] = [0, host_blk, host_blk + 20_000]
    params["delta_ns"] = [0, 10_000, 110_000]
    bt = params["bt"]
    now = 50 * S
    reqs = draw_requests(rng, n, [0.5, 0.5], ttft, 512, (32, 4096), [128, 128], (1, 4096), now, 0.5,
                         lambda g, m: g.uniform(0, 1, m), 0.3, bt)
    hit = reqs["n0"] + reqs["n1"]
    n0 = np.ceil(hit * 0.3).astype(np.int32)
    n1 = np.ceil((hit - n0) * 0.5).astype(np.int32)
    n2 = (hit - n0 - n1).astype(np.int32)
    prompt = reqs["prompt"]
    maxb = 4096 // bt + 8
    hbm_ids = rng.permutation(n_hbm).astype(np.int32)
    host_ids = rng.permutation(n_host).astype(np.int32)
    deep_ids = rng.permutation(n_deep).astype(np.int32)
    hbm_tbl = np.full((n, maxb), -1, np.int32)
    host_tbl = np.full((n, maxb), -1, np.int32)
    deep_tbl = np.full((n, maxb), -1, np.int32)
    # prefix groups: consecutive runs of a random permutation
    perm = rng.permutation(n)
    grouped = perm[: int(n * group_frac)]
    leader = np.full(n, -1, np.int64)
    i = 0
    while i < len(grouped):
        size = int(rng.integers(2, 7))
        members = grouped[i:i + size]
        i += size
        if len(members) < 2:
            break
        lead = members[np.argmax(prompt[members])]      # the longest prompt leads: its match covers the others'
        leader[members] = lead
    hbm_used = host_used = deep_used = 0
    order = np.argsort(np.where(leader == np.arange(n), 0, 1), kind="stable")   # leaders first
    for r in order:
        ld = leader[r]
        if ld >= 0:
            n0[r] = 0
        if ld >= 0 and ld != r:
            # match a prefix of the leader's blocks: m blocks, first its host part, then its deep part
            m = int(min(rng.integers(1, n1[ld] + n2[ld] + 1) if n1[ld] + n2[ld] > 0 else 0, (prompt[r] - 1) // bt))
            n1[r] = min(m, n1[ld])
            n2[r] = m - n1[r]
            if n2[r] > 0 and n1[r] < n1[ld]:
                n2[r] = 0
            host_tbl[r, : n1[r]] = host_tbl[ld, : n1[r]]
            deep_tbl[r, n1[r]: n1[r] + n2[r]] = deep_tbl[ld, n1[ld]: n1[ld] + n2[r]]
            continue
        a, b, c = int(n0[r]), int(n1[r]), int(n2[r])
        if hbm_used + a > n_hbm or host_used + b > n_host or deep_used + c > n_deep:
            n0[r] = n1[r] = n2[r] = 0
            continue
        hbm_tbl[r, :a] = hbm_ids[hbm_used:hbm_used + a]
        host_tbl[r, a:a + b] = host_ids[host_used:host_used + b]
        deep_tbl[r, a + b:a + b + c] = deep_ids[deep_used:deep_used + c]
        hbm_used, host_used, deep_used = hbm_used + a, host_used + b, deep_used + c
    reqs["n0"], reqs["n1"], reqs["n2"] = n0, n1, n2
    private = (n0 > 0) & (rng.uniform(0, 1, n) < 0.5)
    reqs["flags"][private] |= FLAG_HBM_PRIVATE | FLAG_RUNNING
    hbm_free_count = min(n_hbm - hbm_used, hbm_free_target)
    hbm_free = np.full(n_hbm, -1, np.int32)
    hbm_free[:hbm_free_count] = hbm_ids[n_hbm - hbm_free_count:]
    host_free_count = min(n_host - host_used, host_free_target)
    host_free = np.full(n_host, -1, np.int32)
    host_free[:host_free_count] = host_ids[n_host - host_free_count:]
    w = Workload("deep_shared", params, reqs, now, 8, 8 * 512, kv_layout(n_hbm, n_chunks, chunk_bytes), n_host, maxb,
                 hbm_tbl, host_tbl, hbm_free, hbm_free_count, host_free, host_free_count)
    w.deep_tbl, w.deep_blocks = deep_tbl, n_deep
    w.notes["leader"] = leader
    return w


LLAMA8B_CLASSES = dict(mix=[0.6, 0.3, 0.1], ttft=[1 * S, 3 * S, 30 * S], out_median=[256, 256, 4096])


def config_llama8b(seed: int = 0, n: int = 1024, hbm_bytes: int = 60 * 10**9, host_bytes: int = 40 * 10**9,
                   hbm_free_target: int = 256, elapsed_scale: float = 1.5, hbm_share: float = 0.5) -> Workload:
    """Llama-3-8B-shaped KV (2 MiB blocks: 64 chunks of 32 KiB), three SLO classes, beta(2,2) reuse.
    Waiting times are uniform in [0, elapsed_scale * TTFT of the class]; ``hbm_share`` of every reused
    prefix sits in HBM, the rest in the host pool."""
    rng = np.random.default_rng(seed)
    c = LLAMA8B_CLASSES
    n_chunks, chunk_bytes = 64, 32 * 1024
    bb = n_chunks * chunk_bytes
    params = default_params(ttft_ns=c["ttft"], tpot_ns=[50 * MS] * 3, token_budget=8192, tier2_reserve=1024,
                            max_batch=128)
    params["blk_ns"] = [0, -(-bb * 1_000_000_000 // 50_000_000_000), 10 * -(-bb * 1_000_000_000 // 50_000_000_000)]
    now = 100 * S
    reqs = draw_requests(rng, n, c["mix"], c["ttft"], 1024, (32, 32768), c["out_median"], (1, 65536), now,
                         elapsed_scale, lambda g, m: g.beta(2, 2, m), hbm_share, params["bt"])
    n_hbm, n_host = hbm_bytes // bb, host_bytes // bb
    maxb = 2048
    tbl = place_blocks(rng, reqs, n_hbm, n_host, maxb, 0.9, hbm_free_target, 0.5)
    return Workload("llama8b", params, reqs, now, 64, 64 * 2048, kv_layout(n_hbm, n_chunks, chunk_bytes), n_host,
                    maxb, *tbl)


class SchedulerSweep:
    """Scheduler-scale sweep: budget + order + admission + plan only (no tables, no copies).

    ``n`` live requests drawn as in the Llama-3-8B-shaped configuration; the load comes from 256
    in-flight decode sequences.  Every iteration the clock advances 25 ms, a seeded 5 % of the
    slots are replaced by fresh arrivals and 5 % of the decode contexts are replaced; the rest of
    the contexts grow by one token."""

    def __init__(self, n: int, seed: int = 0):
        self.rng = np.random.default_rng(seed)
        c = LLAMA8B_CLASSES
        self.n = n
        bb = 64 * 32 * 1024
        self.params = default_params(ttft_ns=c["ttft"], tpot_ns=[50 * MS] * 3, token_budget=8192,
                                     tier2_reserve=1024, max_batch=512)
        self.params["blk_ns"] = [0, -(-bb * 1_000_000_000 // 50_000_000_000), 420_000]
        self.now = 100 * S
        self.reqs = self._draw(n, 0)
        self.next_id = n
        self.ctx = self._draw_ctx(256)
        self.hbm_free_count = 1 << 30
        self.host_free_count = 1 << 30

    def _draw(self, m, id0, fresh=False):
        c = LLAMA8B_CLASSES
        r = draw_requests(self.rng, m, c["mix"], c["ttft"], 1024, (32, 32768), c["out_median"], (1, 65536),
                          self.now, 0.0 if fresh else 1.5, lambda g, k: g.beta(2, 2, k), 0.5, self.params["bt"], id0)
        has = r["n0"] > 0
        r["flags"][has & (self.rng.uniform(0, 1, m) < 0.5)] |= FLAG_HBM_PRIVATE | FLAG_RUNNING
        return r

    def _draw_ctx(self, m):
        c = LLAMA8B_CLASSES
        r = draw_requests(self.rng, m, c["mix"], c["ttft"], 1024, (32, 32768), c["out_median"], (1, 65536),
                          self.now, 1.5, lambda g, k: g.beta(2, 2, k), 0.5, self.params["bt"])
        return r["prompt"].astype(np.int64) + np.floor(self.rng.uniform(0, 1, m) * r["pred_out"]).astype(np.int64)

    @property
    def D_act(self) -> int:
        return len(self.ctx)

    @property
    def K_act(self) -> int:
        return int(self.ctx.sum())

    def step(self):
        """Advance one iteration.  Returns the slot indices that were rewritten."""
        self.now += 25 * MS
        m = max(1, self.n // 20)
        slots = self.rng.choice(self.n, size=m, replace=False)
        fresh = self._draw(m, self.next_id & 0xFFFFFFFF, fresh=True)
        self.next_id += m
        for k, v in fresh.items():
            self.reqs[k][slots] = v
        self.ctx += 1
        k = max(1, len(self.ctx) // 20)
        which = self.rng.choice(len(self.ctx), size=k, replace=False)
        self.ctx[which] = self._draw_ctx(k)
        return np.sort(slots)

    def workload(self) -> Workload:
        w = Workload(f"sweep{self.n}", self.params, self.reqs, self.now, self.D_act, self.K_act)
        w.hbm_free_count = self.hbm_free_count
        w.host_free_count = self.host_free_count
        return w


def copy_lists(seed: int, n_copies: int, n_src_blocks: int, n_dst_blocks: int):
    """Two independent samples without replacement: scattered, non-contiguous source and destination ids."""
    rng = np.random.default_rng(seed)
    src = rng.choice(n_src_blocks, size=n_copies, replace=False).astype(np.int32)
    dst = rng.choice(n_dst_blocks, size=n_copies, replace=False).astype(np.int32)
    return src, dst


LLAMA70B_CLASSES = dict(mix=[0.3, 0.2, 0.1, 0.4], ttft=[1 * S, 3 * S, 30 * S, 1 * S], out_median=[256, 256, 4096, 128])


@dataclass
class Trace:
    """A whole arrival trace for the closed-loop replay (Llama-3-70B-shaped KV, 5 MiB blocks)."""
    params: dict
    arrival_ns: np.ndarray     # int64 [n], ascending
    prompt: np.ndarray         # int32
    pred_out: np.ndarray       # int32
    cls: np.ndarray            # uint8
    n0: np.ndarray             # int32: matched blocks resident in HBM at arrival
    n1: np.ndarray             # int32: matched blocks on host at arrival
    shared: np.ndarray         # bool: the HBM part is the shared system prefix (never preempted)
    hbm_tbl: np.ndarray        # int32 [n, maxb]
    host_tbl: np.ndarray       # int32 [n, maxb]
    hbm_free: np.ndarray
    hbm_free_count: int
    host_free: np.ndarray
    host_free_count: int
    layout: dict
    host_blocks: int
    maxb: int
    shared_ids: np.ndarray     # HBM ids of the shared prefix


def config_llama70b_trace(seed: int = 0, n: int = 4096, rate_per_s: float = 20.0, hbm_bytes: int = 60 * 10**9,
                          host_bytes: int = 40 * 10**9, shared_prefix_tokens: int = 8192,
                          hbm_occupancy: float = 0.5) -> Trace:
    """4096 requests with exponential inter-arrival times (20 requests/s), four SLO classes (chat, code,
    reasoning, agentic).  Agentic requests hit a shared system prefix held in HBM with probability 0.7 (the
    same block ids in every hitting request's table); other requests reuse a Beta(2,2) fraction of their
    prompt, 40 % of it in HBM and 60 % on host.  5 MiB blocks (160 chunks of 32 KiB).  Cached prefixes of
    requests that have not arrived yet occupy at most ``hbm_occupancy`` of the HBM pool."""
    rng = np.random.default_rng(seed)
    c = LLAMA70B_CLASSES
    n_chunks, chunk_bytes = 160, 32 * 1024
    bb = n_chunks * chunk_bytes
    blk = -(-bb * 1_000_000_000 // 50_000_000_000)
    params = default_params(ttft_ns=c["ttft"], tpot_ns=[100 * MS] * 4, token_budget=16384, tier2_reserve=2048,
                            max_batch=128, blk_ns=[0, blk, 10 * blk])
    bt = params["bt"]
    arrival = np.cumsum(rng.exponential(1e9 / rate_per_s, n)).astype(np.int64)
    cls = rng.choice(4, size=n, p=c["mix"]).astype(np.uint8)
    prompt = _lognormal_int(rng, 1024, 1.0, 32, 32768, n)
    agentic_hit = (cls == 3) & (rng.uniform(0, 1, n) < 0.7)
    prompt[agentic_hit] = np.maximum(prompt[agentic_hit], shared_prefix_tokens + 64)  # prefix + own suffix
    med = np.asarray(c["out_median"], float)[cls]
    pred_out = np.clip(np.rint(np.exp(rng.normal(np.log(med), 1.0))), 1, 65536).astype(np.int32)
    n_hbm, n_host = hbm_bytes // bb, host_bytes // bb
    maxb = 2048
    shared_blocks = shared_prefix_tokens // bt
    hbm_ids = rng.permutation(n_hbm).astype(np.int32)
    host_ids = rng.permutation(n_host).astype(np.int32)
    shared_ids = hbm_ids[:shared_blocks].copy()
    hbm_used, host_used = shared_blocks, 0
    hbm_lim, host_lim = int(n_hbm * hbm_occupancy), int(n_host * 0.9)
    frac = rng.beta(2, 2, n)
    n0 = np.zeros(n, np.int32)
    n1 = np.zeros(n, np.int32)
    hbm_tbl = np.full((n, maxb), -1, np.int32)
    host_tbl = np.full((n, maxb), -1, np.int32)
    for r in range(n):
        if agentic_hit[r]:
            n0[r] = shared_blocks
            hbm_tbl[r, :shared_blocks] = shared_ids
            continue
        hit = min(int(frac[r] * (prompt[r] // bt)), (prompt[r] - 1) // bt)
        a = int(np.ceil(hit * 0.4))
        a = min(a, hbm_lim - hbm_used)
        b = hit - int(np.ceil(hit * 0.4)) if a == int(np.ceil(hit * 0.4)) else 0
        b = min(b, host_lim - host_used)
        n0[r], n1[r] = a, b
        hbm_tbl[r, :a] = hbm_ids[hbm_used:hbm_used + a]
        hbm_used += a
        host_tbl[r, a:a + b] = host_ids[host_used:host_used + b]
        host_used += b
    hbm_free = np.full(n_hbm, -1, np.int32)
    hbm_free_count = n_hbm - hbm_used
    hbm_free[:hbm_free_count] = hbm_ids[hbm_used:]
    host_free = np.full(n_host, -1, np.int32)
    host_free_count = n_host - host_used
    host_free[:host_free_count] = host_ids[host_used:]
    return Trace(params, arrival, prompt, pred_out, cls, n0, n1, agentic_hit, hbm_tbl, host_tbl, hbm_free,
                 hbm_free_count, host_free, host_free_count, kv_layout(n_hbm, n_chunks, chunk_bytes), n_host, maxb,
                 shared_ids)


def fuzz_params(rng) -> dict:
    """Random parameters anywhere inside the library's validated bounds, extremes included."""
    nc = int(rng.integers(1, 5))
    bt = int(rng.choice([1, 4, 16, 16, 16, 32, 128]))
    d = dict(bt=bt, chunk_shift=int(rng.integers(0, 13)), max_batch=int(rng.choice([1, 4, 64, 128, 512, 4096])),
             max_ctx_avg=int(rng.choice([0, 512, 2048, 1 << 15])), gamma_q16=int(rng.choice([0, 65536, 81920, 1 << 17])),
             token_budget=int(rng.choice([0, 64, 2048, 8192, 1 << 20])), tier2_reserve=int(rng.choice([0, 64, 1024, 1 << 21])),
             c_tok_q20=int(rng.choice([0, 1000, 50_000, 1 << 19])) * Q20, c_attn_q20=int(rng.choice([0, 1, Q20 // 2, Q20])),
             c_iter_q20=int(rng.choice([0, 2_000_000, 1 << 29])) * Q20, c_dseq_q20=int(rng.choice([0, 10_000, 1 << 19])) * Q20,
             c_dkv_q20=int(rng.choice([0, 20, 255])) * Q20,
             delta_ns=[0, int(rng.choice([0, 10_000, 1 << 30])), int(rng.choice([0, 110_000, 5000]))],
             blk_ns=[0, int(rng.choice([1, 328, 40_000, 1 << 27])), int(rng.choice([1, 20_000, 340_000]))],
             ttft_ns=[int(rng.choice([0, 10**8, 10**9, 3 * 10**10, 1 << 40])) for _ in range(nc)],
             tpot_ns=[int(rng.choice([0, 10**6, 5 * 10**7])) for _ in range(nc)],
             policy=int(rng.choice([0, 0, 0, 1, 2, 3])), plan_first=int(rng.integers(0, 2)))
    if (d["max_batch"] - 1) * d["max_ctx_avg"] > (1 << 32):
        d["max_ctx_avg"] = 512
    return d


def fuzz_workload(rng, d: dict, sizes=(1, 2, 33, 200, 1000, 1025, 3000)) -> Workload:
    """A random queue with tables, free lists and a deep tier for the parameters ``d``: sizes from 1 to 3000
    (or one of ``sizes``), hit profiles of every shape, a few requests outside the input bounds, rows too short for
    their prompt, shared host / deep record ids, free lists from empty to ample, loads from idle to the maximum."""
    n = int(rng.choice(list(sizes)))
    bt = d["bt"]
    nc = len(d["ttft_ns"])
    maxb = int(rng.choice([8, 64, 200]))
    prompt = rng.integers(1, maxb * bt + 1, n).astype(np.int32)
    if rng.uniform() < 0.3:
        prompt[rng.integers(0, n, max(1, n // 50))] = maxb * bt + int(rng.integers(1, 100))   # row too short: invalid with tables
    hit = np.floor(rng.uniform(0, 1, n) * ((prompt - 1) // bt)).astype(np.int64)
    a = rng.uniform(0, 1, n); b = rng.uniform(0, 1, n)
    n0 = np.floor(hit * a).astype(np.int32)
    n1 = np.floor((hit - n0) * b).astype(np.int32)
    n2 = (hit - n0 - n1).astype(np.int32)
    z = rng.uniform(0, 1, n)
    n1[z < 0.2] += n2[z < 0.2]; n2[z < 0.2] = 0
    now = int(rng.choice([0, 10**10, 1 << 45]))
    elapsed = rng.integers(0, 4 * 10**10, n) if rng.uniform() < 0.8 else rng.integers(-10**6, 1 << 49, n)
    reqs = dict(arrival_ns=(now - elapsed).astype(np.int64), prompt=prompt,
                pred_out=rng.integers(0, 1 << 16, n).astype(np.int32), n0=n0, n1=n1, n2=n2,
                id=rng.permutation(1 << 23)[:n].astype(np.uint32) if rng.uniform() < 0.7 else rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32),
                cls=rng.integers(0, nc, n).astype(np.uint8), flags=rng.integers(0, 4, n).astype(np.uint8))
    # some broken requests
    if rng.uniform() < 0.3 and n > 3:
        k = rng.integers(0, n, 3)
        reqs["prompt"][k[0]] = 0; reqs["n0"][k[1]] = -1; reqs["cls"][k[2]] = 7
    tot0, tot1, tot2 = int(np.maximum(n0, 0).sum()), int(n1.sum()), int(n2.sum())
    n_hbm = tot0 + int(rng.choice([0, 5, 200, 5000])) + 1
    n_host = tot1 + int(rng.choice([0, 5, 200, 5000])) + 1
    n_deep = tot2 + 8
    hbm_ids, host_ids, deep_ids = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32), rng.permutation(n_deep).astype(np.int32)
    hbm_tbl = np.full((n, maxb + 1), -1, np.int32); host_tbl = hbm_tbl.copy(); deep_tbl = hbm_tbl.copy()
    u0 = u1 = u2 = 0
    share = rng.uniform() < 0.5
    filled = np.zeros(n, bool)
    for r in range(n):
        a0, a1, a2 = max(int(n0[r]), 0), int(n1[r]), int(n2[r])
        if a0 + a1 + a2 > maxb + 1:
            continue
        filled[r] = True
        hbm_tbl[r, :a0] = hbm_ids[u0:u0 + a0]; u0 += a0
        m1 = m2 = 0
        q = int(rng.integers(0, r)) if (share and r > 0 and rng.uniform() < 0.3) else -1
        if q >= 0 and filled[q]:
            q0, q1, q2 = max(int(n0[q]), 0), int(n1[q]), int(n2[q])
            m1 = min(a1, q1)
            host_tbl[r, a0:a0 + m1] = host_tbl[q, q0:q0 + m1]
            m2 = min(a2, q2)
            deep_tbl[r, a0 + a1:a0 + a1 + m2] = deep_tbl[q, q0 + q1:q0 + q1 + m2]
        host_tbl[r, a0 + m1:a0 + a1] = host_ids[u1:u1 + a1 - m1]; u1 += a1 - m1
        deep_tbl[r, a0 + a1 + m2:a0 + a1 + a2] = deep_ids[u2:u2 + a2 - m2]; u2 += a2 - m2
    # -1 cells inside ranges (from sharing with shorter rows) are replaced by fresh ids where possible
    hbm_free = np.full(n_hbm, -1, np.int32); hf = n_hbm - u0
    hbm_free[:hf] = hbm_ids[u0:]
    host_free = np.full(n_host, -1, np.int32); of = n_host - u1
    host_free[:of] = host_ids[u1:]
    hfc = int(rng.choice([hf, hf, min(hf, 3), 0]))
    ofc = int(rng.choice([of, of, min(of, 3), 0]))
    D = int(rng.choice([0, 8, 64, 1 << 16])); K = int(rng.choice([0, 4096, 1 << 20, 1 << 32]))
    lay = kv_layout(n_hbm, 1, 16)
    w = Workload("fuzz", d, reqs, now, D, K, lay, n_host, maxb + 1, hbm_tbl, host_tbl, hbm_free, hfc, host_free, ofc)
    w.deep_tbl, w.deep_blocks = deep_tbl, n_deep
    return w
