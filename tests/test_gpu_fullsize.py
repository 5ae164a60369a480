"""GPU parity at the benchmark's full sizes: 60 GB paged HBM pool, 40 GB pinned host pool, 2 MiB blocks.

Scheduling outputs are compared in full (1024 requests); the copies are checked on sampled blocks the
oracle computes one by one (compact mirrors of just those blocks) and by properties that hold at any
size: nothing but the named destinations changes."""
import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu

HBM_BYTES, HOST_BYTES = 60 * 10**9, 40 * 10**9
BB = 2 * 1024 * 1024


@pytest.fixture(scope="module")
def pools():
    import torch
    from paper_2608_06557_b200.runner import alloc_pinned_pool, fill_pools
    free, _ = torch.cuda.mem_get_info()
    hbm_bytes = HBM_BYTES if free > HBM_BYTES + 20 * 10**9 else (free // 2 // BB) * BB
    host_pool, host_bytes = alloc_pinned_pool((HOST_BYTES // BB) * BB)
    hbm_pool = torch.empty((hbm_bytes // BB) * BB, dtype=torch.uint8, device="cuda")
    fill_pools(hbm_pool, host_pool)
    yield dict(hbm=hbm_pool, host=host_pool, hbm_bytes=hbm_pool.numel(), host_bytes=(host_bytes // BB) * BB)
    del hbm_pool, host_pool
    torch.cuda.empty_cache()
    torch._C._host_emptyCache()


def hbm_block(torch, pool, lay, ids):
    """[len(ids), block_bytes] uint8: the paged blocks gathered chunk by chunk."""
    v = pool.view(lay["n_chunks"], lay["n_blocks"], lay["chunk_bytes"])
    return v[:, ids.long(), :].permute(1, 0, 2).reshape(len(ids), -1)


def host_record(pool, ids, bb):
    return pool.view(-1, bb)[ids.long().cpu()]


def block_sums(torch, pool, n_rows, row_bytes):
    return pool.view(torch.int64).view(n_rows, row_bytes // 8).sum(dim=1)


@pytest.mark.parametrize("seed", [0, 14, 25])
def test_bench_step_at_full_size(pools, seed):
    import torch
    from paper_2608_06557_b200.runner import Instance
    w = wl.config_llama8b(seed=seed, n=1024, hbm_bytes=pools["hbm_bytes"], host_bytes=pools["host_bytes"],
                          hbm_free_target=256, elapsed_scale=0.3, hbm_share=0.5 if seed == 0 else 0.4)
    lay = w.layout
    ref = oracle_iteration(w)
    plan = ref["plan"]
    inst = Instance(w, hbm_pool=pools["hbm"], host_pool=pools["host"][: w.host_blocks * BB], alloc_pools=False)
    rng = np.random.default_rng(seed)
    pick = lambda a, k: np.sort(rng.choice(len(a), size=min(k, len(a)), replace=False)) if len(a) else np.zeros(0, int)
    ie, ir = pick(plan["evict_src"], 48), pick(plan["restore_src"], 48)
    es, ed = plan["evict_src"][ie], plan["evict_dst"][ie]
    rs, rd = plan["restore_src"][ir], plan["restore_dst"][ir]
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    # sources as they are before the step
    src_hbm = hbm_block(torch, inst.hbm_pool, lay, t(es)).cpu().numpy() if len(es) else None
    src_host = host_record(inst.host_pool, t(rs), BB).numpy().copy() if len(rs) else None
    # checksums of every chunk row / record, to prove nothing else moves
    n_rows = lay["n_chunks"] * lay["n_blocks"]
    hbm_before = block_sums(torch, inst.hbm_pool, n_rows, lay["chunk_bytes"]).cpu().numpy()
    probe = np.sort(rng.choice(w.host_blocks, size=512, replace=False))
    host_before = host_record(inst.host_pool, t(probe), BB).view(torch.int64).sum(dim=1).numpy()

    if seed == 14:
        inst.run_step(inst.step_args(with_move=True))     # as bench.py times it: one call, evict + restore as the fused move
    elif seed == 25:
        # the copy-engine path, with a staging buffer smaller than the lists (batches reuse their regions)
        inst.run_step(inst.step_args())
        staging = torch.empty(96 * BB, dtype=torch.uint8, device="cuda")
        inst.run_move_staged(staging)
        torch.cuda.synchronize()
        del staging
    else:
        inst.run_iteration()                              # the five calls, evict then restore
    got = inst.fetch()

    # scheduling and plan outputs in full
    for k in ("budget", "key", "order", "grant"):
        assert np.array_equal(got[k], ref[k]), k
    for k in ("x1", "x2", "tokens_run", "action", "restore_src", "restore_dst", "evict_src", "evict_dst"):
        assert np.array_equal(got[k], plan[k]), k
    assert got["plan_counts"] == plan["counts"] and got["status"] == ref["status"]
    assert np.array_equal(got["hbm_tbl"], ref["pools"].hbm_tbl) and np.array_equal(got["host_tbl"], ref["pools"].host_tbl)
    assert plan["counts"]["n_evict"] > 0

    # sampled copies: the oracle computes these blocks on compact mirrors, one slot per sampled block
    if len(es):
        mlay = wl.kv_layout(len(es), lay["n_chunks"], lay["chunk_bytes"])
        m_hbm = np.ascontiguousarray(src_hbm.reshape(len(es), lay["n_chunks"], -1).transpose(1, 0, 2)).reshape(-1)
        m_host = np.zeros(len(es) * BB, np.uint8)
        assert oracle.kv_evict(m_hbm, mlay, m_host, len(es), np.arange(len(es), dtype=np.int32),
                               np.arange(len(es), dtype=np.int32)) == 0
        assert np.array_equal(host_record(inst.host_pool, t(ed), BB).numpy().reshape(-1), m_host)
    if len(rs):
        mlay = wl.kv_layout(len(rs), lay["n_chunks"], lay["chunk_bytes"])
        m_hbm = np.zeros(len(rs) * BB, np.uint8)
        assert oracle.kv_restore(m_hbm, mlay, src_host.reshape(-1), len(rs), np.arange(len(rs), dtype=np.int32),
                                 np.arange(len(rs), dtype=np.int32)) == 0
        dev = hbm_block(torch, inst.hbm_pool, lay, t(rd)).cpu().numpy()
        exp = m_hbm.reshape(lay["n_chunks"], len(rs), -1).transpose(1, 0, 2).reshape(len(rs), -1)
        assert np.array_equal(dev, exp)

    # nothing but the restore destinations changed in HBM; sampled host records change only if evict destinations
    hbm_after = block_sums(torch, inst.hbm_pool, n_rows, lay["chunk_bytes"]).cpu().numpy()
    changed = np.unique(np.nonzero(hbm_before != hbm_after)[0] % lay["n_blocks"])
    assert set(changed.tolist()) <= set(plan["restore_dst"].tolist())
    host_after = host_record(inst.host_pool, t(probe), BB).view(torch.int64).sum(dim=1).numpy()
    moved = probe[host_before != host_after]
    assert set(moved.tolist()) <= set(plan["evict_dst"].tolist())


@pytest.mark.parametrize("n", [1, 16, 256, 4096])
def test_evict_restore_round_trip_sweep(pools, n):
    """Evict n scattered blocks to the host pool, poison them in HBM, restore them: bytes come back."""
    import torch
    from paper_2608_06557_b200 import cascade as cs
    n_hbm, n_host = pools["hbm_bytes"] // BB, pools["host_bytes"] // BB
    lay = wl.kv_layout(n_hbm, 64, 32 * 1024)
    layout = cs.make_layout(lay)
    ctx = cs.Context(wl.default_params(), 16, 0)
    hbm_ids, host_ids = wl.copy_lists(40 + n, n, n_hbm, n_host)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    h, o = t(hbm_ids), t(host_ids)
    original = hbm_block(torch, pools["hbm"], lay, h).clone()
    ctx.kv_evict(layout, pools["hbm"], pools["host"], n_host, False, h, o, None, n)
    torch.cuda.synchronize()
    step = max(1, n // 64)
    assert torch.equal(host_record(pools["host"], o[::step], BB), original[::step].cpu())
    pools["hbm"].view(64, n_hbm, 32 * 1024)[:, h.long(), :] = 0xEE
    ctx.kv_restore(layout, pools["hbm"], pools["host"], n_host, False, o, h, None, n)
    torch.cuda.synchronize()
    assert torch.equal(hbm_block(torch, pools["hbm"], lay, h), original)
    assert ctx.status()[0] == 0
