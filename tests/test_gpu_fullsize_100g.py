"""The evict / restore bandwidth sweep's host pool at its stated size: 100 * 10^9 bytes of pinned host memory.

The pool is requested once at that size; a box that cannot page-lock so much gets the largest pool it grants
(the request is cut to 70 % of the available memory, then halved until it succeeds) and the size obtained is
printed.  Round trips of 1, 16, 256 and 4096 scattered blocks use records over the WHOLE pool, the last record
included; bytes must come back as they were."""
import numpy as np
import pytest

from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu

BB = 2 * 1024 * 1024
STATED = 100 * 10**9


def test_round_trips_over_the_100_gb_pinned_pool():
    import torch
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200.runner import alloc_pinned_pool
    torch.cuda.empty_cache()
    torch._C._host_emptyCache()
    host, got = alloc_pinned_pool(STATED // BB * BB)
    n_host = got // BB
    print(f"pinned host pool: asked {STATED} bytes, got {got} bytes ({n_host} records)")
    assert got >= 8 * 10**9
    n_hbm = 8192                                          # 16 GiB paged pool: the link and the record side are under test
    hbm = torch.empty(n_hbm * BB, dtype=torch.uint8, device="cuda")
    words = torch.arange(BB // 8, dtype=torch.int64, device="cuda")
    v = hbm.view(torch.int64).view(64, n_hbm, 32768 // 8)
    for c in range(64):
        v[c] = (torch.arange(n_hbm, dtype=torch.int64, device="cuda")[:, None] * 0x9E3779B97F4A7C15 % (1 << 62)
                + words[None, c * 4096:(c + 1) * 4096] * 31 + c)
    lay = wl.kv_layout(n_hbm, 64, 32 * 1024)
    layout = cs.make_layout(lay)
    ctx = cs.Context(wl.default_params(), 16, 0)
    rng = np.random.default_rng(5)
    for n in (1, 16, 256, 4096):
        hbm_ids = rng.choice(n_hbm, size=n, replace=False).astype(np.int32)
        host_ids = rng.choice(n_host - 1, size=n, replace=False).astype(np.int32)
        host_ids[0] = n_host - 1                           # the very last record of the pool
        h, o = torch.from_numpy(hbm_ids).cuda(), torch.from_numpy(host_ids).cuda()
        blocks = lambda: hbm.view(64, n_hbm, 32 * 1024)[:, h.long(), :].permute(1, 0, 2).reshape(n, -1)
        original = blocks().clone()
        ctx.kv_evict(layout, hbm, host, n_host, False, h, o, None, n)
        torch.cuda.synchronize()
        step = max(1, n // 32)
        assert torch.equal(host.view(-1, BB)[o[::step].long().cpu()], original[::step].cpu())
        hbm.view(64, n_hbm, 32 * 1024)[:, h.long(), :] = 0xEE
        ctx.kv_restore(layout, hbm, host, n_host, False, o, h, None, n)
        torch.cuda.synchronize()
        assert torch.equal(blocks(), original)
    assert ctx.status()[0] == 0
    del host, hbm
    torch.cuda.empty_cache()
    torch._C._host_emptyCache()
