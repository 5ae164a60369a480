"""The library used from plain C: tests/c_abi_driver.c is compiled with gcc against the header and the CUDA
runtime, runs one whole iteration without Python or PyTorch in the process (as the five calls, as one cascade_step call, or
with the copy-engine move), and its outputs are compared with the oracle's."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle
from helpers import oracle_iteration
from paper_2608_06557_b200 import build as cbuild
from paper_2608_06557_b200 import cascade as cs
from paper_2608_06557_b200 import workload as wl

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _compile(tmp_path):
    lib = cbuild.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = tmp_path / "c_abi_driver"
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(cuda, "include"), os.path.join(ROOT, "tests", "c_abi_driver.c"),
                           "-o", str(exe), lib, "-L", os.path.join(cuda, "lib64"), "-lcudart",
                           f"-Wl,-rpath,{os.path.dirname(lib)}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"])
    return exe


@pytest.mark.parametrize("seed,mode", [(0, "calls"), (3, "calls"), (0, "step"), (3, "staged")])
def test_one_iteration_from_plain_c(tmp_path, seed, mode):
    w = wl.config_tiny(seed, hbm_free_target=60)
    w.params["ttft_ns"] = [20 * t for t in w.params["ttft_ns"]]
    lay, bb = w.layout, w.block_bytes
    n_hbm, n_host = lay["n_blocks"], w.host_blocks
    hbm = wl.pool_bytes(1, n_hbm * bb).copy()
    host = wl.pool_bytes(2, n_host * bb).copy()
    params = cs.make_params(w.params)
    header = np.zeros(16, np.int64)
    header[:12] = [w.n, w.maxb, n_hbm, n_host, lay["n_chunks"], lay["chunk_bytes"], w.hbm_free_count, w.host_free_count,
                   w.now_ns, w.D_act, w.K_act, ctypes.sizeof(params)]
    r = w.reqs
    with open(tmp_path / "in.bin", "wb") as f:
        f.write(header.tobytes())
        f.write(bytes(params))
        for k, dt in (("arrival_ns", np.int64), ("prompt", np.int32), ("pred_out", np.int32), ("n0", np.int32),
                      ("n1", np.int32), ("n2", np.int32), ("id", np.uint32), ("cls", np.uint8), ("flags", np.uint8)):
            f.write(np.ascontiguousarray(r[k], dtype=dt).tobytes())
        for a in (w.hbm_tbl, w.host_tbl, w.hbm_free, w.host_free, hbm, host):
            f.write(np.ascontiguousarray(a).tobytes())
    exe = _compile(tmp_path)
    subprocess.check_call([str(exe), str(tmp_path / "in.bin"), str(tmp_path / "out.bin")] +
                          ([] if mode == "calls" else [mode]))

    ref = oracle_iteration(w)
    plan, pools = ref["plan"], ref["pools"]
    ref_hbm, ref_host = hbm.copy(), host.copy()
    assert oracle.kv_evict(ref_hbm, lay, ref_host, n_host, plan["evict_src"], plan["evict_dst"]) == 0
    assert oracle.kv_restore(ref_hbm, lay, ref_host, n_host, plan["restore_src"], plan["restore_dst"]) == 0
    assert plan["counts"]["n_restore"] > 0 and plan["counts"]["n_evict"] > 0

    buf = open(tmp_path / "out.bin", "rb").read()
    pos = 0

    def take(dtype, count):
        nonlocal pos
        a = np.frombuffer(buf, dtype=dtype, count=count, offset=pos)
        pos += a.nbytes
        return a

    oh = take(np.int64, 4)
    assert oh[0] == ref["status"] and oh[1] == 0 and oh[2] >= 100
    n = w.n
    assert np.array_equal(take(np.int64, n), ref["budget"]) and np.array_equal(take(np.uint64, n), ref["key"])
    assert np.array_equal(take(np.uint32, n), ref["order"]) and np.array_equal(take(np.int32, n), ref["grant"])
    sc = take(np.int32, 4)
    assert sc[0] == ref["sched_counts"]["n_tier1"] and sc[1] == ref["sched_counts"]["n_admitted"]
    assert int(sc[2:4].view(np.int64)[0]) == ref["sched_counts"]["tokens_granted"]
    for k in ("x1", "x2", "tokens_run"):
        assert np.array_equal(take(np.int32, n), plan[k]), k
    assert np.array_equal(take(np.uint8, n), plan["action"])
    pc = take(np.int32, 12)
    names = ("n_restore", "n_evict", "n_drop_blocks", "n_victims", "n_unadmitted", "n_admitted", "hbm_need", "deficit",
             "hbm_free_after", "host_free_after")
    assert {k: int(v) for k, v in zip(names, pc[:10])} == {k: plan["counts"][k] for k in names}
    assert int(pc[10:12].view(np.int64)[0]) == plan["counts"]["tokens_run"]
    nr, ne = plan["counts"]["n_restore"], plan["counts"]["n_evict"]
    assert np.array_equal(take(np.int32, n_hbm)[:nr], plan["restore_src"])
    assert np.array_equal(take(np.int32, n_hbm)[:nr], plan["restore_dst"])
    assert np.array_equal(take(np.int32, n_host)[:ne], plan["evict_src"])
    assert np.array_equal(take(np.int32, n_host)[:ne], plan["evict_dst"])
    assert np.array_equal(take(np.int32, n * w.maxb).reshape(n, w.maxb), pools.hbm_tbl)
    assert np.array_equal(take(np.int32, n * w.maxb).reshape(n, w.maxb), pools.host_tbl)
    assert take(np.int32, 1)[0] == pools.hbm_free_count and take(np.int32, 1)[0] == pools.host_free_count
    assert np.array_equal(take(np.uint8, n_hbm * bb), ref_hbm)
    assert np.array_equal(take(np.uint8, n_host * bb), ref_host)
    assert pos == len(buf)
