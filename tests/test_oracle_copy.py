"""Pins for the oracle's paged copies: byte identity, evict -> restore identity, nothing else touched."""
import numpy as np

import oracle
from paper_2608_06557_b200 import workload as wl


def pools(n_hbm=40, n_host=24, n_chunks=4, chunk_bytes=64):
    lay = wl.kv_layout(n_hbm, n_chunks, chunk_bytes)
    hbm = wl.pool_bytes(1, n_hbm * n_chunks * chunk_bytes).copy()
    host = wl.pool_bytes(2, n_host * n_chunks * chunk_bytes).copy()
    return lay, hbm, host


def test_restore_matches_plain_indexing():
    lay, hbm, host = pools()
    src, dst = wl.copy_lists(0, 9, 24, 40)
    ref = hbm.copy().reshape(lay["n_chunks"], lay["n_blocks"], lay["chunk_bytes"])
    hview = host.reshape(24, lay["n_chunks"], lay["chunk_bytes"])
    for s, d in zip(src, dst):
        ref[:, d, :] = hview[s]
    assert oracle.kv_restore(hbm, lay, host, 24, src, dst) == 0
    assert np.array_equal(hbm, ref.reshape(-1))
    assert np.array_equal(host, wl.pool_bytes(2, host.size))          # source untouched


def test_evict_matches_plain_indexing_and_round_trip_is_identity():
    lay, hbm, host = pools()
    hbm0, host0 = hbm.copy(), host.copy()
    src, dst = wl.copy_lists(1, 11, 40, 24)
    assert oracle.kv_evict(hbm, lay, host, 24, src, dst) == 0
    ref = host0.copy().reshape(24, lay["n_chunks"], lay["chunk_bytes"])
    hv = hbm0.reshape(lay["n_chunks"], lay["n_blocks"], lay["chunk_bytes"])
    for s, d in zip(src, dst):
        ref[d] = hv[:, s, :]
    assert np.array_equal(host, ref.reshape(-1)) and np.array_equal(hbm, hbm0)
    # poison the evicted HBM blocks, restore to other blocks: bytes come back
    hbm.reshape(lay["n_chunks"], lay["n_blocks"], lay["chunk_bytes"])[:, src, :] = 0xEE
    back = np.random.default_rng(3).permutation(40)[:11].astype(np.int32)
    assert oracle.kv_restore(hbm, lay, host, 24, dst, back) == 0
    now = hbm.reshape(lay["n_chunks"], lay["n_blocks"], lay["chunk_bytes"])
    for s, b in zip(src, back):
        assert np.array_equal(now[:, b, :], hv[:, s, :])


def test_block_major_strides_and_bad_ids():
    n_hbm, n_chunks, cb = 10, 3, 32
    lay = dict(n_blocks=n_hbm, n_chunks=n_chunks, chunk_bytes=cb, chunk_stride=cb, block_stride=n_chunks * cb)
    hbm = np.zeros(n_hbm * n_chunks * cb, np.uint8)
    host = wl.pool_bytes(7, 5 * n_chunks * cb).copy()
    st = oracle.kv_restore(hbm, lay, host, 5, np.array([4, 9, -1, 2], np.int32), np.array([0, 1, 2, 10], np.int32))
    assert st == oracle.ST_EBOUNDS
    assert np.array_equal(hbm[: n_chunks * cb], host[4 * n_chunks * cb:])   # block-major: records are contiguous
    assert not hbm[n_chunks * cb:].any()                                   # bad pairs were skipped
    assert oracle.kv_restore(hbm, lay, host, 5, np.zeros(0, np.int32), np.zeros(0, np.int32)) == 0
