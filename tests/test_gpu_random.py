"""Randomised GPU parity: many small seeded cases of the ordering kernel and of the fused evict+restore
kernel, with sizes and shapes drawn at random (ragged tails, tiny chunks, overlapping block reuse)."""
import numpy as np
import pytest

import oracle
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu


def test_ordering_of_random_keys_and_sizes():
    import torch
    from paper_2608_06557_b200.runner import Instance
    rng = np.random.default_rng(123)
    w = wl.config_llama8b(seed=1, n=65536, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    inst = Instance(w, alloc_pools=False)
    sizes = [1, 2, 33, 255, 256, 257, 1000, 1024, 1025, 2048, 3000, 4096, 4097, 8192, 10000, 16384, 16385, 30000,
             32768, 50000, 65536]
    for trial in range(300):
        n = int(rng.choice(sizes))
        mode = trial % 4
        if mode == 0:
            key = rng.integers(0, 1 << 63, n, dtype=np.int64).astype(np.uint64) * np.uint64(2) \
                + rng.integers(0, 2, n).astype(np.uint64)
        elif mode == 1:     # few distinct values in one digit: most passes are skipped, ties keep slot order
            key = rng.integers(0, 16, n).astype(np.uint64) << np.uint64(int(rng.integers(0, 60)))
        elif mode == 2:     # reverse sorted
            key = np.sort(rng.integers(0, 1 << 62, n, dtype=np.int64)).astype(np.uint64)[::-1].copy()
        else:               # the library's own key shape: 40-bit value, 23-bit id
            key = (rng.integers(0, 1 << 40, n, dtype=np.int64).astype(np.uint64) << np.uint64(23)) \
                | np.arange(n, dtype=np.uint64)
        inst.n = n
        inst.key.view(torch.int64)[:n].copy_(torch.from_numpy(key.view(np.int64)))
        inst.ctx.schedule(inst.reqs_struct, inst.key, n, w.D_act, inst.order, inst.grant, inst.sched_counts)
        torch.cuda.synchronize()
        assert np.array_equal(inst.order[:n].cpu().numpy(), np.argsort(key, kind="stable")), (trial, n, mode)
    assert inst.ctx.status()[0] == 0


def test_fused_move_on_random_shapes():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    rng = np.random.default_rng(7)
    ctx = cs.Context(wl.default_params(), 16, 0)
    done = 0
    while done < 120:
        n_hbm, n_host = int(rng.integers(8, 300)), int(rng.integers(8, 300))
        n_chunks = int(rng.choice([1, 3, 8, 64]))
        cb = int(rng.choice([16, 48, 4096, 32768, 32768 + 16]))
        if n_chunks * cb * (n_hbm + n_host) > 300e6:
            continue
        lay = wl.kv_layout(n_hbm, n_chunks, cb)
        bb = n_chunks * cb
        hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
        host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
        ne = int(rng.integers(0, min(n_hbm, n_host) // 2 + 1))
        nr = int(rng.integers(0, min(n_hbm, n_host) // 2 + 1))
        hp, op = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32)
        es, ed, rs = hp[:ne], op[:ne], op[ne:ne + nr]
        k = int(rng.integers(0, min(ne, nr) + 1))          # restores that land in blocks evicted by the same call
        rd = rng.permutation(np.concatenate([rng.permutation(es)[:k], hp[ne:ne + nr - k]])).astype(np.int32)
        ref_h, ref_o = hbm_np.copy(), host_np.copy()
        assert oracle.kv_evict(ref_h, lay, ref_o, n_host, es, ed) == 0
        assert oracle.kv_restore(ref_h, lay, ref_o, n_host, rs, rd) == 0
        hbm = torch.from_numpy(hbm_np).cuda()
        host = torch.from_numpy(host_np).pin_memory()
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda() if len(a) else \
            torch.zeros(1, dtype=torch.int32, device="cuda")
        scratch = torch.empty(cs.kv_move_scratch_len(ne, nr), dtype=torch.int32, device="cuda")
        ctx.kv_move(cs.make_layout(lay), hbm, host, n_host, t(es), t(ed), None, ne, t(rs), t(rd), None, nr, scratch)
        torch.cuda.synchronize()
        assert np.array_equal(hbm.cpu().numpy(), ref_h), (n_hbm, n_host, n_chunks, cb, ne, nr, k)
        assert np.array_equal(host.numpy(), ref_o), (n_hbm, n_host, n_chunks, cb, ne, nr, k)
        done += 1
    assert ctx.status()[0] == 0


@pytest.mark.parametrize("n,reps", [(1024, 400), (2048, 200), (4096, 200), (16384, 200), (40000, 40), (65536, 40)])
def test_repeated_runs_give_identical_results(n, reps):
    """The cluster kernels exchange data through shared memory of other CTAs; an ordering bug there would show
    as results that change from run to run.  Same inputs, many runs, every output compared with the first."""
    import torch
    from paper_2608_06557_b200.runner import Instance
    sw = wl.SchedulerSweep(n, seed=5)
    inst = Instance(sw.workload(), alloc_pools=False)
    ref = None
    for _ in range(reps):
        for t in (inst.order, inst.grant, inst.x1, inst.tokens_run, inst.action):
            t.fill_(0)
        inst.run_schedule()
        cur = [t[:n].clone() for t in (inst.budget, inst.key.view(torch.int64), inst.order.view(torch.int32), inst.grant,
                                       inst.x1, inst.x2, inst.tokens_run, inst.action)] + [inst.plan_counts.clone(),
                                                                                         inst.sched_counts.clone()]
        if ref is None:
            ref = cur
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, cur))
    assert inst.ctx.status()[0] == 0


def test_staged_move_on_random_shapes():
    """The copy-engine path on random shapes, list lengths and staging sizes (down to one block per direction), with
    restores into blocks the same call evicts, runs of consecutive host records and, now and then, a restore that
    reads a record the same call's evictions write."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    rng = np.random.default_rng(17)
    ctx = cs.Context(wl.default_params(), 16, 0)
    done = 0
    while done < 60:
        n_hbm, n_host = int(rng.integers(8, 200)), int(rng.integers(8, 200))
        n_chunks = int(rng.choice([1, 3, 8, 64]))
        cb = int(rng.choice([16, 48, 4096, 32768, 32768 + 16]))
        if n_chunks * cb * (n_hbm + n_host) > 200e6:
            continue
        lay = wl.kv_layout(n_hbm, n_chunks, cb)
        bb = n_chunks * cb
        hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
        host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
        ne = int(rng.integers(0, min(n_hbm, n_host) // 2 + 1))
        nr = int(rng.integers(0, min(n_hbm, n_host) // 2 + 1))
        hp, op = rng.permutation(n_hbm).astype(np.int32), rng.permutation(n_host).astype(np.int32)
        es, ed, rs = hp[:ne], op[:ne].copy(), op[ne:ne + nr].copy()
        if rng.random() < 0.5:
            ed.sort()
            rs.sort()
        if ne and nr and rng.random() < 0.3:
            rs[0] = ed[-1]                                   # a restore reads what this call's evictions write
        k = int(rng.integers(0, min(ne, nr) + 1))
        rd = rng.permutation(np.concatenate([rng.permutation(es)[:k], hp[ne:ne + nr - k]])).astype(np.int32)
        ref_h, ref_o = hbm_np.copy(), host_np.copy()
        assert oracle.kv_evict(ref_h, lay, ref_o, n_host, es, ed) == 0
        assert oracle.kv_restore(ref_h, lay, ref_o, n_host, rs, rd) == 0
        hbm = torch.from_numpy(hbm_np).cuda()
        host = torch.from_numpy(host_np).pin_memory()
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda() if len(a) else None
        stage_blocks = int(rng.integers(2 if ne and nr else 1, ne + nr + 3))
        staging = torch.empty(stage_blocks * bb, dtype=torch.uint8, device="cuda")
        mailbox = torch.empty(cs.kv_mailbox_len(ne, nr), dtype=torch.int32, pin_memory=True)
        ctx.kv_move_staged(cs.make_layout(lay), hbm, host, n_host, t(es), t(ed), None, ne, t(rs), t(rd), None, nr, staging,
                           stage_blocks, mailbox)
        torch.cuda.synchronize()
        assert np.array_equal(hbm.cpu().numpy(), ref_h), (n_hbm, n_host, n_chunks, cb, ne, nr, k, stage_blocks)
        assert np.array_equal(host.numpy(), ref_o), (n_hbm, n_host, n_chunks, cb, ne, nr, k, stage_blocks)
        done += 1
    assert ctx.status()[0] == 0


def test_ordering_with_random_runs_of_equal_high_bits():
    """Random tie structure for the two-stage ordering (bits 32..63 first, runs of equal values repaired afterwards):
    the high 48 bits are drawn from pools of different sizes, so runs of every length from 2 to far beyond the local
    repair's limit appear at random positions, inside CTAs and astride their boundaries; the low 16 bits are random
    or constant (full-key duplicates keep slot order).  Checked against numpy's stable argsort."""
    import torch
    from paper_2608_06557_b200.runner import Instance
    rng = np.random.default_rng(321)
    w = wl.config_llama8b(seed=2, n=65536, hbm_bytes=2 * 10**9, host_bytes=2 * 10**9)
    w.hbm_tbl = w.host_tbl = w.hbm_free = w.host_free = None
    w.hbm_free_count, w.host_free_count = 1 << 30, 1 << 30
    inst = Instance(w, alloc_pools=False)
    for trial in range(120):
        n = int(rng.integers(4097, 65537)) if trial % 3 else int(rng.choice([4097, 8192, 16384, 16385, 32768, 32769, 65536]))
        pool = int(rng.choice([n // 300 + 1, n // 20 + 1, n // 3 + 1, n, 4 * n]))      # fewer values -> longer runs
        high = rng.integers(0, 1 << 47, pool, dtype=np.int64).astype(np.uint64)[rng.integers(0, pool, n)]
        if trial % 4 == 0:
            high[rng.integers(0, n, n // 10)] = high[0]                                  # one very long run
        low = rng.integers(0, 1 << 16, n).astype(np.uint64) if trial % 5 else np.zeros(n, np.uint64)
        key = (high << np.uint64(16)) | low
        inst.n = n
        inst.key.view(torch.int64)[:n].copy_(torch.from_numpy(key.view(np.int64)))
        inst.ctx.schedule(inst.reqs_struct, inst.key, n, w.D_act, inst.order, inst.grant, inst.sched_counts)
        torch.cuda.synchronize()
        assert np.array_equal(inst.order[:n].cpu().numpy(), np.argsort(key, kind="stable")), (trial, n, pool)
    assert inst.ctx.status()[0] == 0


def test_many_long_copies_in_a_row_on_one_context():
    """Long calls of the copy ring hand their pieces out through a pair of counters that the last CTA leaves at zero;
    the context owns 64 such pairs and gives them to its launches in turn.  150 calls in a row (every pair used more
    than twice), evictions and restores with fresh random lists, each long enough for the on-demand form, no host
    synchronisation in between: the pools must equal the oracle's after the same sequence."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    n_chunks, cb = 8, 16384
    bb = n_chunks * cb
    n_hbm, n_host = 400, 400
    lay = wl.kv_layout(n_hbm, n_chunks, cb)
    rng = np.random.default_rng(77)
    hbm_np = rng.integers(0, 256, n_hbm * bb, dtype=np.uint8)
    host_np = rng.integers(0, 256, n_host * bb, dtype=np.uint8)
    hbm, host = torch.from_numpy(hbm_np.copy()).cuda(), torch.from_numpy(host_np.copy()).pin_memory()
    ctx = cs.Context(wl.default_params(), 16, 0)
    layout = cs.make_layout(lay)
    keep = []
    for call in range(150):
        n = int(rng.integers(140, 200))                     # 1120 .. 1600 pieces: more than sixteen per CTA
        h = rng.permutation(n_hbm)[:n].astype(np.int32)
        o = rng.permutation(n_host)[:n].astype(np.int32)
        th, to = torch.from_numpy(h).cuda(), torch.from_numpy(o).cuda()
        keep.append((th, to))
        if call % 2 == 0:
            ctx.kv_evict(layout, hbm, host, n_host, False, th, to, None, n)
            assert oracle.kv_evict(hbm_np, lay, host_np, n_host, h, o) == 0
        else:
            ctx.kv_restore(layout, hbm, host, n_host, False, to, th, None, n)
            assert oracle.kv_restore(hbm_np, lay, host_np, n_host, o, h) == 0
    torch.cuda.synchronize()
    assert ctx.status()[0] == 0
    assert np.array_equal(hbm.cpu().numpy(), hbm_np) and np.array_equal(host.numpy(), host_np)
