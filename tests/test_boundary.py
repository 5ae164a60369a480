"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2608_06557_b200 import build as cbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cascade.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cascade_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(cbuild.build())
    names = declared_symbols()
    assert {"cascade_budget", "cascade_schedule", "cascade_tier_plan", "cascade_kv_restore",
            "cascade_kv_evict"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    lib.cascade_version.restype = ctypes.c_int
    assert lib.cascade_version() >= 100


def test_binding_lists_the_same_symbols_and_struct_sizes():
    from paper_2608_06557_b200 import cascade as cs
    declared = set(declared_symbols())
    assert declared == set(cs.EXPORTS)
    assert ctypes.sizeof(cs.Params) == 8 * 4 + 5 * 8 + 6 * 8 + 16 * 8 + 8
    assert ctypes.sizeof(cs.SchedCounts) == 16 and ctypes.sizeof(cs.PlanCounts) == 48
    assert ctypes.sizeof(cs.KvLayout) == 40 and ctypes.sizeof(cs.Reqs) == 72


def test_host_validation_without_a_device():
    """Errors the library finds before touching CUDA are reachable with no GPU at all."""
    from paper_2608_06557_b200 import cascade as cs
    from paper_2608_06557_b200 import workload as wl
    lib = cs.raw()
    h = ctypes.c_void_p()
    p = cs.make_params(wl.default_params())
    assert lib.cascade_create(None, ctypes.byref(p), 16, 0) == cs.EINVAL
    assert lib.cascade_create(ctypes.byref(h), None, 16, 0) == cs.EINVAL
    assert lib.cascade_create(ctypes.byref(h), ctypes.byref(p), 0, 0) == cs.EINVAL
    assert lib.cascade_create(ctypes.byref(h), ctypes.byref(p), cs.MAX_REQUESTS + 1, 0) == cs.EINVAL
    for bad in (dict(bt=0), dict(gamma_q16=1 << 18), dict(blk_ns=[0, 0, 1]), dict(c_attn_q20=(1 << 20) + 1),
                dict(ttft_ns=[1 << 41]), dict(max_batch=0), dict(delta_ns=[0, -1, 0])):
        q = cs.make_params(wl.default_params(**bad))
        assert lib.cascade_create(ctypes.byref(h), ctypes.byref(q), 16, 0) == cs.ERANGE, bad
    assert lib.cascade_budget(None, None, 0, 0, 0, 0, None, None, None) == cs.EINVAL
    assert lib.cascade_status(None, None, 0, None) == cs.EINVAL
    assert lib.cascade_step(None, None, None) == cs.EINVAL
    assert lib.cascade_kv_move(None, None, None, None, 0, None, None, None, 1, None, None, None, 1, None, None) == cs.EINVAL
    assert lib.cascade_kv_move_staged(None, None, None, None, 0, None, None, None, 1, None, None, None, 1, None, 4, None,
                                      None) == cs.EINVAL


def test_scratch_and_mailbox_sizes_are_plain_host_arithmetic():
    """The two size helpers need no device: restore results + restore matches + evict counters + a hash table of at
    most half-full power-of-two size for the move; two counts + four lists for the mailbox."""
    from paper_2608_06557_b200 import cascade as cs
    assert cs.kv_move_scratch_len(0, 0) == 2 * 64
    assert cs.kv_move_scratch_len(10, 7) == 2 * 7 + 10 + 2 * 64
    assert cs.kv_move_scratch_len(33, 0) == 33 + 2 * 128            # 66 slots needed -> 128
    assert cs.kv_move_scratch_len(19073, 28610) == 2 * 28610 + 19073 + 2 * 65536
    assert cs.kv_move_scratch_len(-1, 0) == -1 and cs.kv_mailbox_len(0, -5) == -1
    assert cs.kv_mailbox_len(0, 0) == 2 and cs.kv_mailbox_len(5, 9) == 2 + 10 + 18
    prev = 0
    for ne in range(0, 3000, 37):
        cur = cs.kv_move_scratch_len(ne, 11)
        assert cur >= prev and cur >= 2 * 11 + ne + 4 * ne           # room for a table no more than half full
        prev = cur


def test_header_is_plain_c_and_the_binding_mirrors_its_struct_layouts(tmp_path):
    """The header must compile as C99 on its own, and every ctypes mirror must have the size and the field
    offsets the C compiler gives the struct (a silent mismatch would shift every pointer behind it)."""
    import subprocess
    from paper_2608_06557_b200 import cascade as cs
    pairs = [("cascade_params", cs.Params), ("cascade_reqs", cs.Reqs), ("cascade_sched_counts", cs.SchedCounts),
             ("cascade_plan_counts", cs.PlanCounts), ("cascade_pools", cs.Pools), ("cascade_plan", cs.Plan),
             ("cascade_kv_layout", cs.KvLayout), ("cascade_status_t", cs.Status),
             ("cascade_stage_counts", cs.StageCounts), ("cascade_stage", cs.Stage),
             ("cascade_dedup_counts", cs.DedupCounts), ("cascade_dedup_args", cs.DedupArgs),
             ("cascade_step_args", cs.StepArgs)]
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "cascade.h"', 'int main(void) {']
    for cname, ct in pairs:
        lines.append(f'  printf("{cname} %zu", sizeof({cname}));')
        for fname, _ in ct._fields_:
            lines.append(f'  printf(" %zu", offsetof({cname}, {fname}));')
        lines.append('  printf("\\n");')
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                           "-o", str(exe), str(src)])
    out = subprocess.check_output([str(exe)], text=True).splitlines()
    for (cname, ct), line in zip(pairs, out):
        got = [int(x) for x in line.split()[1:]]
        want = [ctypes.sizeof(ct)] + [getattr(ct, f).offset for f, _ in ct._fields_]
        assert got == want, (cname, got, want)
    # prefetch counts have no ctypes mirror (the runner reads them as six int32): pin their size here
    src2 = tmp_path / "pf.c"
    src2.write_text('#include <stdio.h>\n#include "cascade.h"\nint main(void){printf("%zu", sizeof(cascade_prefetch_counts));return 0;}')
    subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), "-o", str(tmp_path / "pf"), str(src2)])
    assert subprocess.check_output([str(tmp_path / "pf")], text=True) == "24"
