"""GPU parity: paged KV restore / evict against the CPU oracle, byte for byte."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def _gpu():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import Instance
    assert torch.cuda.is_available()
    return torch, cs, Instance


class CopyRig:
    """A paged HBM pool, a pinned host pool and a device staging pool with guard bands around each."""

    GUARD = 4096

    def __init__(self, n_hbm, n_host, n_chunks, chunk_bytes, block_major=False):
        torch, cs, _ = _gpu()
        self.torch, self.cs = torch, cs
        if block_major:
            self.lay = dict(n_blocks=n_hbm, n_chunks=n_chunks, chunk_bytes=chunk_bytes, chunk_stride=chunk_bytes,
                            block_stride=n_chunks * chunk_bytes)
        else:
            self.lay = wl.kv_layout(n_hbm, n_chunks, chunk_bytes)
        self.n_hbm, self.n_host = n_hbm, n_host
        self.bb = n_chunks * chunk_bytes
        g = self.GUARD
        self.hbm_np = wl.pool_bytes(1, n_hbm * self.bb).copy()
        self.host_np = wl.pool_bytes(2, n_host * self.bb).copy()
        self.hbm_buf = torch.full((n_hbm * self.bb + 2 * g,), 0xA5, dtype=torch.uint8, device="cuda")
        self.host_buf = torch.full((n_host * self.bb + 2 * g,), 0x5A, dtype=torch.uint8).pin_memory()
        self.stage_buf = torch.full((n_host * self.bb + 2 * g,), 0x3C, dtype=torch.uint8, device="cuda")
        self.hbm = self.hbm_buf[g:-g]
        self.host = self.host_buf[g:-g]
        self.stage = self.stage_buf[g:-g]
        self.hbm.copy_(torch.from_numpy(self.hbm_np))
        self.host.copy_(torch.from_numpy(self.host_np))
        self.stage.copy_(torch.from_numpy(self.host_np))
        self.ctx = cs.Context(wl.default_params(), 16, 0)
        self.layout = cs.make_layout(self.lay)
        torch.cuda.synchronize()

    def ids(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a, np.int32)).cuda()

    def guards_intact(self):
        g = self.GUARD
        t = self.torch
        t.cuda.synchronize()
        return (bool((self.hbm_buf[:g] == 0xA5).all()) and bool((self.hbm_buf[-g:] == 0xA5).all())
                and bool((self.host_buf[:g] == 0x5A).all()) and bool((self.host_buf[-g:] == 0x5A).all())
                and bool((self.stage_buf[:g] == 0x3C).all()) and bool((self.stage_buf[-g:] == 0x3C).all()))


@pytest.mark.parametrize("shape", [(64, 48, 4, 4096, False), (40, 24, 3, 208, False), (33, 20, 5, 48, True),
                                   (24, 16, 64, 32768, False), (20, 12, 2, 16 * 1024 + 16, True)])
@pytest.mark.parametrize("via", ["host", "stage"])
def test_restore_evict_round_trip(shape, via):
    n_hbm, n_host, n_chunks, cb, bm = shape
    rig = CopyRig(n_hbm, n_host, n_chunks, cb, bm)
    torch = rig.torch
    rec = rig.host if via == "host" else rig.stage
    is_dev = via == "stage"
    n = min(n_hbm, n_host) // 2 + 1
    # restore: host records -> HBM blocks
    src, dst = wl.copy_lists(1, n, n_host, n_hbm)
    ref_hbm, ref_host = rig.hbm_np.copy(), rig.host_np.copy()
    assert oracle.kv_restore(ref_hbm, rig.lay, ref_host, n_host, src, dst) == 0
    rig.ctx.kv_restore(rig.layout, rig.hbm, rec, n_host, is_dev, rig.ids(src), rig.ids(dst), None, n)
    torch.cuda.synchronize()
    assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm)
    # evict: other HBM blocks -> other host records, count taken from device memory
    src2, dst2 = wl.copy_lists(2, n, n_hbm, n_host)
    assert oracle.kv_evict(ref_hbm, rig.lay, ref_host, n_host, src2, dst2) == 0
    cap = n + 5
    s2 = rig.ids(np.concatenate([src2, np.full(5, 10**6, np.int32)]))
    d2 = rig.ids(np.concatenate([dst2, np.full(5, 10**6, np.int32)]))
    n_dev = torch.tensor([n], dtype=torch.int32, device="cuda")
    rig.ctx.kv_evict(rig.layout, rig.hbm, rec, n_host, is_dev, s2, d2, n_dev, cap)
    torch.cuda.synchronize()
    assert np.array_equal(rec.cpu().numpy(), ref_host)
    assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm)
    # poison the evicted blocks and bring them back: identity
    view = rig.hbm_np.reshape(-1)
    rig.hbm.fill_(0xEE)
    back = np.random.default_rng(5).permutation(n_hbm)[:n].astype(np.int32)
    rig.ctx.kv_restore(rig.layout, rig.hbm, rec, n_host, is_dev, rig.ids(dst2), rig.ids(back), None, n)
    torch.cuda.synchronize()
    now = rig.hbm.cpu().numpy()
    exp = np.full_like(now, 0xEE)
    assert oracle.kv_restore(exp, rig.lay, ref_host, n_host, dst2, back) == 0
    assert np.array_equal(now, exp)
    assert rig.guards_intact()
    assert rig.ctx.status()[0] == 0


def test_bad_ids_are_skipped_and_flagged():
    rig = CopyRig(16, 16, 4, 256)
    torch = rig.torch
    src = np.array([3, -1, 16, 5, 2], np.int32)
    dst = np.array([0, 1, 2, 99, 7], np.int32)
    ref = rig.hbm_np.copy()
    st = oracle.kv_restore(ref, rig.lay, rig.host_np, 16, src, dst)
    rig.ctx.kv_restore(rig.layout, rig.hbm, rig.host, 16, False, rig.ids(src), rig.ids(dst), None, 5)
    torch.cuda.synchronize()
    assert np.array_equal(rig.hbm.cpu().numpy(), ref)
    assert rig.ctx.status()[0] == st == 1
    assert rig.guards_intact()
    # empty and zero-count calls launch nothing / move nothing
    rig.ctx.kv_restore(rig.layout, rig.hbm, rig.host, 16, False, rig.ids(src), rig.ids(dst), None, 0)
    zero = torch.zeros(1, dtype=torch.int32, device="cuda")
    rig.ctx.kv_evict(rig.layout, rig.hbm, rig.host, 16, False, rig.ids(src), rig.ids(dst), zero, 5)
    torch.cuda.synchronize()
    assert np.array_equal(rig.host.cpu().numpy(), rig.host_np)


def test_bad_ids_in_a_long_list_are_skipped_and_flagged():
    """The same on a call long enough for the ring to hand its pieces out on demand (more than sixteen pieces per CTA),
    over the host link and through the staging buffer, with ids below zero and beyond either pool scattered through
    both lists, and with a device-side count shorter than the list."""
    rig = CopyRig(260, 260, 8, 16384)
    torch = rig.torch
    rng = np.random.default_rng(9)
    n = 250
    src = rng.permutation(260)[:n].astype(np.int32)
    dst = rng.permutation(260)[:n].astype(np.int32)
    for k, v in ((3, -1), (40, 260), (41, 1 << 30), (199, -7)):
        src[k] = v
    for k, v in ((7, -2), (120, 260), (233, 99999)):
        dst[k] = v
    live = 240                                                   # the last ten entries are beyond the device count
    count = torch.tensor([live], dtype=torch.int32, device="cuda")
    for on_device in (False, True):
        rec = rig.stage if on_device else rig.host
        ref = rig.hbm_np.copy()
        st = oracle.kv_restore(ref, rig.lay, rig.host_np, 260, src[:live], dst[:live])
        rig.hbm.copy_(torch.from_numpy(rig.hbm_np))
        rig.ctx.kv_restore(rig.layout, rig.hbm, rec, 260, on_device, rig.ids(src), rig.ids(dst), count, n)
        torch.cuda.synchronize()
        assert np.array_equal(rig.hbm.cpu().numpy(), ref), on_device
        assert rig.ctx.status(clear=True)[0] == st == 1
        ref_rec = rig.host_np.copy()
        st = oracle.kv_evict(rig.hbm_np, rig.lay, ref_rec, 260, dst[:live], src[:live])
        rig.hbm.copy_(torch.from_numpy(rig.hbm_np))
        rec.copy_(torch.from_numpy(rig.host_np))
        rig.ctx.kv_evict(rig.layout, rig.hbm, rec, 260, on_device, rig.ids(dst), rig.ids(src), count, n)
        torch.cuda.synchronize()
        assert np.array_equal(rec.cpu().numpy(), ref_rec), on_device
        assert rig.ctx.status(clear=True)[0] == st == 1
    assert rig.guards_intact()


def test_layout_validation_on_the_host():
    rig = CopyRig(8, 8, 2, 64)
    cs = rig.cs
    ids = rig.ids([0])
    bad = cs.make_layout(dict(rig.lay, chunk_bytes=40))
    with pytest.raises(cs.CascadeError):
        rig.ctx.kv_restore(bad, rig.hbm, rig.host, 8, False, ids, ids, None, 1)
    with pytest.raises(cs.CascadeError):
        rig.ctx.kv_restore(rig.layout, rig.hbm[8:], rig.host, 8, False, ids, ids, None, 1)
    with pytest.raises(cs.CascadeError):
        rig.ctx.kv_restore(rig.layout, rig.hbm, rig.host, 8, False, None, ids, None, 1)


@pytest.mark.parametrize("seed,ttft_scale", [(0, 1), (1, 1), (2, 1), (0, 20), (3, 20)])
def test_full_iteration_tiny_with_copies(seed, ttft_scale):
    """All five calls on the tiny configuration; pools compared byte for byte with the oracle's mirrors.
    With the published class targets most queued requests are already past their TTFT target and get no
    restore (Eq. 7 with a negative remaining budget); the looser targets exercise the restore list."""
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(seed)
    w.params["ttft_ns"] = [t * ttft_scale for t in w.params["ttft_ns"]]
    ref = oracle_iteration(w)
    bb = w.block_bytes
    hbm_np = wl.pool_bytes(3, w.layout["n_blocks"] * bb).copy()
    host_np = wl.pool_bytes(4, w.host_blocks * bb).copy()
    inst = Instance(w)
    inst.hbm_pool.copy_(torch.from_numpy(hbm_np))
    inst.host_pool.copy_(torch.from_numpy(host_np))
    inst.run_iteration()
    got = inst.fetch()
    plan = ref["plan"]
    assert oracle.kv_evict(hbm_np, w.layout, host_np, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
    assert oracle.kv_restore(hbm_np, w.layout, host_np, w.host_blocks, plan["restore_src"], plan["restore_dst"]) == 0
    assert got["plan_counts"] == plan["counts"]
    assert np.array_equal(inst.hbm_pool.cpu().numpy(), hbm_np)
    assert np.array_equal(inst.host_pool.cpu().numpy(), host_np)
    if ttft_scale > 1:
        assert plan["counts"]["n_restore"] > 0


@pytest.mark.parametrize("shape", [(64, 48, 4, 4096), (40, 40, 3, 208), (48, 48, 64, 32768), (30, 30, 2, 32 * 1024 + 64)])
def test_fused_move_equals_evict_then_restore(shape):
    """One call, both directions at once; half of the restores land in blocks the same call evicts."""
    n_hbm, n_host, n_chunks, cb = shape
    rig = CopyRig(n_hbm, n_host, n_chunks, cb)
    torch = rig.torch
    rng = np.random.default_rng(n_hbm)
    ne, nr = n_hbm // 3, n_host // 3
    hperm, operm = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32)
    evict_src, evict_dst = hperm[:ne], operm[:ne]
    restore_src = operm[ne:ne + nr]
    # restore destinations: the blocks evicted LAST (as the plan's stack hands them out), then untouched blocks
    reuse = evict_src[::-1][: nr // 2]
    restore_dst = np.concatenate([reuse, hperm[ne:ne + nr - len(reuse)]]).astype(np.int32)
    ref_hbm, ref_host = rig.hbm_np.copy(), rig.host_np.copy()
    assert oracle.kv_evict(ref_hbm, rig.lay, ref_host, n_host, evict_src, evict_dst) == 0
    assert oracle.kv_restore(ref_hbm, rig.lay, ref_host, n_host, restore_src, restore_dst) == 0
    cap_e, cap_r = ne + 3, nr + 2
    pad = lambda a, cap: rig.ids(np.concatenate([a, np.full(cap - len(a), 10**6, np.int32)]))
    counts = torch.tensor([nr, ne], dtype=torch.int32, device="cuda")
    scratch = torch.empty(rig.cs.kv_move_scratch_len(cap_e, cap_r), dtype=torch.int32, device="cuda")
    for rep in range(2):                              # twice: the scratch is reused as it was left
        rig.hbm.copy_(torch.from_numpy(rig.hbm_np))
        rig.host.copy_(torch.from_numpy(rig.host_np))
        rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, pad(evict_src, cap_e), pad(evict_dst, cap_e),
                        counts[1:2], cap_e, pad(restore_src, cap_r), pad(restore_dst, cap_r), counts[0:1], cap_r,
                        scratch)
        torch.cuda.synchronize()
        assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm), rep
        assert np.array_equal(rig.host.cpu().numpy(), ref_host), rep
    assert rig.guards_intact() and rig.ctx.status()[0] == 0
    # one list empty, and a bad id on each side
    rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, None, None, None, 0, pad(restore_src, cap_r),
                    pad(restore_dst, cap_r), counts[0:1], cap_r, scratch)
    bad_e = evict_src.copy()
    bad_e[0] = -5
    rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, pad(bad_e, cap_e), pad(evict_dst, cap_e), counts[1:2],
                    cap_e, None, None, None, 0, scratch)
    torch.cuda.synchronize()
    assert rig.ctx.status()[0] == 1 and rig.guards_intact()


@pytest.mark.parametrize("seed", [0, 3, 5])
def test_full_iteration_with_fused_move(seed):
    torch, cs, Instance = _gpu()
    w = wl.config_tiny(seed, hbm_free_target=60)
    w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    ref = oracle_iteration(w)
    bb = w.block_bytes
    hbm_np = wl.pool_bytes(3, w.layout["n_blocks"] * bb).copy()
    host_np = wl.pool_bytes(4, w.host_blocks * bb).copy()
    inst = Instance(w)
    inst.hbm_pool.copy_(torch.from_numpy(hbm_np))
    inst.host_pool.copy_(torch.from_numpy(host_np))
    inst.run_iteration(fused_move=True)
    got = inst.fetch()
    plan = ref["plan"]
    assert oracle.kv_evict(hbm_np, w.layout, host_np, w.host_blocks, plan["evict_src"], plan["evict_dst"]) == 0
    assert oracle.kv_restore(hbm_np, w.layout, host_np, w.host_blocks, plan["restore_src"], plan["restore_dst"]) == 0
    assert got["plan_counts"] == plan["counts"] and got["status"] == ref["status"]
    assert np.array_equal(inst.hbm_pool.cpu().numpy(), hbm_np)
    assert np.array_equal(inst.host_pool.cpu().numpy(), host_np)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable(monkeypatch):
    """The fused move makes a restore wait until the block it lands in has been read out by the evict side.
    With the library's test hook the evict side never reports that, so the wait runs into its clock limit
    (a tenth of a second here): the call returns, CASCADE_ST_ETIMEOUT is set, the evicted bytes are on the
    host, the blocks whose restores gave up are untouched, and the same GPU context goes on working."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    n_chunks, cb = 2, 4096
    bb = n_chunks * cb
    n_hbm, n_host = 16, 16
    lay = wl.kv_layout(n_hbm, n_chunks, cb)
    rng = np.random.default_rng(0)
    hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
    host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
    es, ed = np.array([1, 2], np.int32), np.array([5, 6], np.int32)
    rs, rd = np.array([8, 9], np.int32), np.array([2, 12], np.int32)      # the first restore lands in an evicted block
    t = lambda a: torch.from_numpy(a).cuda()
    monkeypatch.setenv("CASCADE_TEST_MOVE_STALL", "1")
    stalled = cs.Context(wl.default_params(), 16, 0)
    monkeypatch.delenv("CASCADE_TEST_MOVE_STALL")
    hbm, host = torch.from_numpy(hbm_np.copy()).cuda(), torch.from_numpy(host_np.copy()).pin_memory()
    scratch = torch.empty(cs.kv_move_scratch_len(2, 2), dtype=torch.int32, device="cuda")
    stalled.kv_move(cs.make_layout(lay), hbm, host, n_host, t(es), t(ed), None, 2, t(rs), t(rd), None, 2, scratch)
    torch.cuda.synchronize()
    assert stalled.status()[0] == cs.ST_ETIMEOUT
    # the restore that gave up is visible per block: every piece of restore 0 unwritten, restore 1 complete
    assert scratch[:2].cpu().tolist() == [n_chunks, 0]
    want_host = host_np.copy()
    assert oracle.kv_evict(hbm_np.copy(), lay, want_host, n_host, es, ed) == 0
    assert np.array_equal(host.numpy(), want_host)                        # the evictions happened
    want_hbm = hbm_np.copy()
    assert oracle.kv_restore(want_hbm, lay, host_np, n_host, rs[1:], rd[1:]) == 0
    assert np.array_equal(hbm.cpu().numpy(), want_hbm)                    # the independent restore too; block 2 untouched
    # same process, same GPU, ordinary context: the full result
    ctx = cs.Context(wl.default_params(), 16, 0)
    hbm, host = torch.from_numpy(hbm_np.copy()).cuda(), torch.from_numpy(host_np.copy()).pin_memory()
    ctx.kv_move(cs.make_layout(lay), hbm, host, n_host, t(es), t(ed), None, 2, t(rs), t(rd), None, 2, scratch)
    torch.cuda.synchronize()
    ref_h, ref_o = hbm_np.copy(), host_np.copy()
    assert oracle.kv_evict(ref_h, lay, ref_o, n_host, es, ed) == 0 and oracle.kv_restore(ref_h, lay, ref_o, n_host, rs, rd) == 0
    assert ctx.status()[0] == 0 and np.array_equal(hbm.cpu().numpy(), ref_h) and np.array_equal(host.numpy(), ref_o)
    assert scratch[:2].cpu().tolist() == [0, 0]


def test_a_load_that_never_completes_is_reported_and_the_loads_in_flight_are_waited_for(monkeypatch):
    """Second test hook: the first piece of CTA 0 announces 16 bytes more than it loads, so its mbarrier never
    completes and the wait runs into its (lowered) clock limit.  The CTA must record CASCADE_ST_ETIMEOUT, wait
    for the other loads it had in flight, and return; every other CTA finishes its share; the context stays usable."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    n_chunks, cb = 8, 32768
    bb = n_chunks * cb
    n_hbm, n_host, n = 64, 64, 40
    lay = wl.kv_layout(n_hbm, n_chunks, cb)
    rng = np.random.default_rng(1)
    hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
    host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
    src, dst = wl.copy_lists(3, n, n_host, n_hbm)
    t = lambda a: torch.from_numpy(a).cuda()
    monkeypatch.setenv("CASCADE_TEST_MOVE_STALL", "2")
    hooked = cs.Context(wl.default_params(), 16, 0)
    monkeypatch.delenv("CASCADE_TEST_MOVE_STALL")
    hbm, host = torch.from_numpy(hbm_np.copy()).cuda(), torch.from_numpy(host_np.copy()).pin_memory()
    hooked.kv_restore(cs.make_layout(lay), hbm, host, n_host, False, t(src), t(dst), None, n)
    torch.cuda.synchronize()
    assert hooked.status()[0] == cs.ST_ETIMEOUT
    want = hbm_np.copy()
    assert oracle.kv_restore(want, lay, host_np, n_host, src, dst) == 0
    got = hbm.cpu().numpy()
    # only pieces of CTA 0's share may be missing: everything else is in place, nothing else was touched
    diff = np.nonzero(got != want)[0]
    assert len(diff) < len(want) // 4
    untouched = np.ones(n_hbm, bool)
    untouched[dst] = False
    v = lambda a: a.reshape(n_chunks, n_hbm, cb)
    assert np.array_equal(v(got)[:, untouched], v(hbm_np)[:, untouched])
    # same process, same GPU, ordinary context: the full result
    ctx = cs.Context(wl.default_params(), 16, 0)
    ctx.kv_restore(cs.make_layout(lay), hbm, host, n_host, False, t(src), t(dst), None, n)
    torch.cuda.synchronize()
    assert ctx.status()[0] == 0 and np.array_equal(hbm.cpu().numpy(), want)


def test_fused_move_beside_a_kernel_that_holds_most_of_the_gpu(monkeypatch):
    """The paper's premise is that spills and restores overlap the running batch.  A finite filler kernel
    (test-only, clock-bounded) holds the shared memory of all but a few SMs on a second stream while the
    fused move runs with restores that depend on evictions, the wait limit lowered to a tenth of a second.
    The restore grid only starts once every evict CTA is on an SM, so no wait can run out: the result equals
    evict-then-restore bit for bit and the status word stays clear."""
    import torch
    from helpers import load_gpu_filler
    from paper_2608_06557_b200 import cascade as cs
    filler = load_gpu_filler()
    n_chunks, cb = 64, 32768
    bb = n_chunks * cb
    n_hbm, n_host, ne, nr = 80, 80, 32, 32
    lay = wl.kv_layout(n_hbm, n_chunks, cb)
    rng = np.random.default_rng(2)
    hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
    host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
    hp, op = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32)
    es, ed, rs = hp[:ne], op[:ne], op[ne:ne + nr]
    rd = np.concatenate([es[::-1][: nr // 2], hp[ne:ne + nr - nr // 2]]).astype(np.int32)
    ref_h, ref_o = hbm_np.copy(), host_np.copy()
    assert oracle.kv_evict(ref_h, lay, ref_o, n_host, es, ed) == 0 and oracle.kv_restore(ref_h, lay, ref_o, n_host, rs, rd) == 0
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    monkeypatch.setenv("CASCADE_TEST_MOVE_STALL", "3")       # lowers the wait limits, stalls nothing
    ctx = cs.Context(wl.default_params(), 16, 0)
    monkeypatch.delenv("CASCADE_TEST_MOVE_STALL")
    hbm, host = torch.from_numpy(hbm_np.copy()).cuda(), torch.from_numpy(host_np.copy()).pin_memory()
    scratch = torch.empty(cs.kv_move_scratch_len(ne, nr), dtype=torch.int32, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    side, main = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    done_fill, done_move = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start = torch.cuda.Event(enable_timing=True)
    start.record(side)
    # 200 KB of shared memory per CTA: no ring CTA (128 KB) fits beside one; about 30 ms at 1.9 GHz
    assert filler.filler_launch(sms - 6, 200 * 1024, 60_000_000, side.cuda_stream) == 0
    done_fill.record(side)
    ctx.kv_move(cs.make_layout(lay), hbm, host, n_host, t(es), t(ed), None, ne, t(rs), t(rd), None, nr, scratch, main)
    done_move.record(main)
    torch.cuda.synchronize()
    assert ctx.status()[0] == 0
    assert scratch[:nr].cpu().tolist() == [0] * nr
    assert np.array_equal(hbm.cpu().numpy(), ref_h) and np.array_equal(host.numpy(), ref_o)
    assert start.elapsed_time(done_fill) > 5.0            # the filler really held the GPU for a while


@pytest.mark.parametrize("shape,stage_blocks", [((64, 48, 4, 4096), 64), ((64, 48, 4, 4096), 5), ((40, 40, 3, 208), 2),
                                                ((300, 300, 8, 32768), 37), ((30, 30, 2, 32 * 1024 + 64), 30)])
def test_staged_move_through_the_copy_engines_equals_evict_then_restore(shape, stage_blocks):
    """The copy-engine path: lists published to a pinned mailbox, one host wait, per-run cudaMemcpyAsync through a
    device staging buffer, gather / scatter by the ring kernel.  Half of the restores land in blocks the same call
    evicts; staging buffers smaller than the lists make the batches wrap."""
    n_hbm, n_host, n_chunks, cb = shape
    rig = CopyRig(n_hbm, n_host, n_chunks, cb)
    torch, cs = rig.torch, rig.cs
    rng = np.random.default_rng(n_hbm + stage_blocks)
    ne, nr = n_hbm // 3, n_host // 3
    hperm, operm = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32)
    evict_src, evict_dst = hperm[:ne], np.sort(operm[:ne])           # sorted records: runs of consecutive ids occur
    restore_src = np.sort(operm[ne:ne + nr])
    reuse = evict_src[::-1][: nr // 2]
    restore_dst = np.concatenate([reuse, hperm[ne:ne + nr - len(reuse)]]).astype(np.int32)
    ref_hbm, ref_host = rig.hbm_np.copy(), rig.host_np.copy()
    assert oracle.kv_evict(ref_hbm, rig.lay, ref_host, n_host, evict_src, evict_dst) == 0
    assert oracle.kv_restore(ref_hbm, rig.lay, ref_host, n_host, restore_src, restore_dst) == 0
    cap_e, cap_r = ne + 3, nr + 2
    pad = lambda a, cap: rig.ids(np.concatenate([a, np.full(cap - len(a), 10**6, np.int32)]))
    counts = torch.tensor([nr, ne], dtype=torch.int32, device="cuda")
    staging = torch.empty(stage_blocks * rig.bb, dtype=torch.uint8, device="cuda")
    mailbox = torch.empty(cs.kv_mailbox_len(cap_e, cap_r), dtype=torch.int32, pin_memory=True)
    for rep in range(2):
        rig.hbm.copy_(torch.from_numpy(rig.hbm_np))
        rig.host.copy_(torch.from_numpy(rig.host_np))
        rig.ctx.kv_move_staged(rig.layout, rig.hbm, rig.host, n_host, pad(evict_src, cap_e), pad(evict_dst, cap_e),
                               counts[1:2], cap_e, pad(restore_src, cap_r), pad(restore_dst, cap_r), counts[0:1], cap_r,
                               staging, stage_blocks, mailbox)
        torch.cuda.synchronize()
        assert mailbox[:2].tolist() == [ne, nr]
        assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm), rep
        assert np.array_equal(rig.host.cpu().numpy(), ref_host), rep
    assert rig.guards_intact() and rig.ctx.status()[0] == 0


def test_staged_move_orders_a_restore_behind_the_eviction_that_writes_its_record_and_skips_bad_ids():
    rig = CopyRig(32, 32, 4, 4096)
    torch, cs = rig.torch, rig.cs
    # restore 0 reads host record 7, which eviction 1 of the same call writes; ids outside the pools on both lists
    evict_src = np.array([3, 9, 40, 11, 12], np.int32)
    evict_dst = np.array([5, 7, 8, -2, 13], np.int32)
    restore_src = np.array([7, 20, 99, 21], np.int32)
    restore_dst = np.array([9, 1, 2, -1], np.int32)
    ref_hbm, ref_host = rig.hbm_np.copy(), rig.host_np.copy()
    st_e = oracle.kv_evict(ref_hbm, rig.lay, ref_host, 32, evict_src, evict_dst)
    st_r = oracle.kv_restore(ref_hbm, rig.lay, ref_host, 32, restore_src, restore_dst)
    assert st_e == st_r == cs.ST_EBOUNDS
    staging = torch.empty(16 * rig.bb, dtype=torch.uint8, device="cuda")
    mailbox = torch.empty(cs.kv_mailbox_len(5, 4), dtype=torch.int32, pin_memory=True)
    rig.ctx.kv_move_staged(rig.layout, rig.hbm, rig.host, 32, rig.ids(evict_src), rig.ids(evict_dst), None, 5,
                           rig.ids(restore_src), rig.ids(restore_dst), None, 4, staging, 16, mailbox)
    torch.cuda.synchronize()
    assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm) and np.array_equal(rig.host.cpu().numpy(), ref_host)
    assert rig.ctx.status()[0] == cs.ST_EBOUNDS and rig.guards_intact()
    # one list empty, then both empty
    rig.ctx.kv_move_staged(rig.layout, rig.hbm, rig.host, 32, None, None, None, 0, rig.ids(restore_src[1:2]),
                           rig.ids(restore_dst[1:2]), None, 1, staging, 16, mailbox)
    rig.ctx.kv_move_staged(rig.layout, rig.hbm, rig.host, 32, None, None, None, 0, None, None, None, 0, staging, 16, mailbox)
    torch.cuda.synchronize()
    assert np.array_equal(rig.hbm.cpu().numpy(), ref_hbm) and rig.ctx.status()[0] == 0


def test_fused_move_inside_a_cuda_graph():
    """The fused move's two grids are tied together by programmatic launch edges; captured in a CUDA graph together
    with the kernels around it (an evict before, a restore after, as a serving loop would queue them) and replayed
    on fresh data, the result must still be evict-then-restore, bit for bit."""
    rig = CopyRig(96, 96, 8, 32768)
    torch, cs = rig.torch, rig.cs
    rng = np.random.default_rng(11)
    ne, nr = 30, 30
    hp, op = rng.permutation(96).astype(np.int32), rng.permutation(96).astype(np.int32)
    es, ed, rs = hp[:ne], op[:ne], op[ne:ne + nr]
    rd = np.concatenate([es[::-1][: nr // 2], hp[ne:ne + nr - nr // 2]]).astype(np.int32)
    pre_s, pre_d = hp[70:75], op[70:75]                      # an eviction before the move
    post_s, post_d = op[80:84], hp[80:84]                    # a restore after it
    t = [rig.ids(x) for x in (es, ed, rs, rd, pre_s, pre_d, post_s, post_d)]
    scratch = torch.empty(cs.kv_move_scratch_len(ne, nr), dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()

    def chain():
        rig.ctx.kv_evict(rig.layout, rig.hbm, rig.host, 96, False, t[4], t[5], None, 5, st)
        rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, 96, t[0], t[1], None, ne, t[2], t[3], None, nr, scratch, st)
        rig.ctx.kv_restore(rig.layout, rig.hbm, rig.host, 96, False, t[6], t[7], None, 4, st)

    with torch.cuda.stream(st):
        chain()                                               # warm-up outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        chain()
    for rep in range(3):
        hbm_np = rng.integers(0, 256, rig.hbm_np.size, dtype=np.uint8)
        host_np = rng.integers(0, 256, rig.host_np.size, dtype=np.uint8)
        rig.hbm.copy_(torch.from_numpy(hbm_np))
        rig.host.copy_(torch.from_numpy(host_np))
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        ref_h, ref_o = hbm_np.copy(), host_np.copy()
        assert oracle.kv_evict(ref_h, rig.lay, ref_o, 96, pre_s, pre_d) == 0
        assert oracle.kv_evict(ref_h, rig.lay, ref_o, 96, es, ed) == 0
        assert oracle.kv_restore(ref_h, rig.lay, ref_o, 96, rs, rd) == 0
        assert oracle.kv_restore(ref_h, rig.lay, ref_o, 96, post_s, post_d) == 0
        assert np.array_equal(rig.hbm.cpu().numpy(), ref_h), rep
        assert np.array_equal(rig.host.cpu().numpy(), ref_o), rep
    assert rig.ctx.status()[0] == 0 and rig.guards_intact()


def test_fused_move_with_block_ids_that_are_multiples_of_a_power_of_two():
    """The match of restore destinations to evicted blocks goes through a hash table over the block ids; ids that share
    their low bits (every 64th block) must neither break it nor make it crawl."""
    n_hbm, n_host, n_chunks, cb = 64 * 300, 700, 2, 256
    rig = CopyRig(n_hbm, n_host, n_chunks, cb)
    torch, cs = rig.torch, rig.cs
    rng = np.random.default_rng(4)
    ne, nr = 290, 290
    strided = (rng.permutation(300).astype(np.int32) * 64)
    op = rng.permutation(n_host).astype(np.int32)
    es, ed, rs = strided[:ne], op[:ne], op[ne:ne + nr]               # restore sources are not among the evict destinations
    rd = rng.permutation(es)[:nr].astype(np.int32)                    # every restore lands in an evicted block
    ref_h, ref_o = rig.hbm_np.copy(), rig.host_np.copy()
    assert oracle.kv_evict(ref_h, rig.lay, ref_o, n_host, es, ed) == 0 and oracle.kv_restore(ref_h, rig.lay, ref_o, n_host, rs, rd) == 0
    scratch = torch.empty(cs.kv_move_scratch_len(ne, nr), dtype=torch.int32, device="cuda")
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, rig.ids(es), rig.ids(ed), None, ne, rig.ids(rs), rig.ids(rd), None, nr, scratch)
    a.record()
    rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, rig.ids(es), rig.ids(ed), None, ne, rig.ids(rs), rig.ids(rd), None, nr, scratch)
    b.record()
    torch.cuda.synchronize()
    rig.hbm.copy_(torch.from_numpy(rig.hbm_np)); rig.host.copy_(torch.from_numpy(rig.host_np))
    rig.ctx.kv_move(rig.layout, rig.hbm, rig.host, n_host, rig.ids(es), rig.ids(ed), None, ne, rig.ids(rs), rig.ids(rd), None, nr, scratch)
    torch.cuda.synchronize()
    assert np.array_equal(rig.hbm.cpu().numpy(), ref_h) and np.array_equal(rig.host.cpu().numpy(), ref_o)
    assert rig.ctx.status()[0] == 0 and scratch[:nr].cpu().tolist() == [0] * nr
    assert a.elapsed_time(b) < 5.0                                     # milliseconds: 150 KB of payload
