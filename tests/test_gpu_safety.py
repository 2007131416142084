"""What output parity cannot show: that no kernel touches memory outside its tiles, and that the bounded
waits of the bulk-copy kernels fail safely.

* Checked build: the library compiled with ``-DREDIST_BOUNDS`` tests every global access against the
  tiles of the launch and every dynamic shared-memory access against the launch's shared-memory size,
  skips what fails and counts it.  The parity problems run on it in a fresh process (the binding loads
  one library per process) and must report zero failures -- and a positive control, in which the checks
  are told that every tile is 16 bytes shorter than it is, must report some.
* Bounded wait: a test-only tuning value makes every block announce 16 bytes more than its copies
  deliver, so that every copy lands but no wait completes, and a second one shortens the poll limit.
  The blocks must count themselves, store nothing, and leave the context usable.  Nothing here faults,
  traps or hangs: the waits simply run out.

Runs in fresh processes, so the counters of the main test process stay at zero.
"""
import os
import subprocess
import sys

import pytest

from paper_2112_01075_b200 import api

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
BOUNDS_LIB = os.path.join(ROOT, "paper_2112_01075_b200", "libredist_b200_bounds.so")


def run_fresh(code, env=None, timeout=1500):
    code = "import sys; sys.path[:0] = [%r, %r]\n" % (HERE, ROOT) + code
    res = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, **(env or {})), capture_output=True,
                         text=True, timeout=timeout)
    assert res.returncode == 0, (res.stdout[-1500:] + "\n" + res.stderr[-2500:])
    return res.stdout


CHECKED_RUN = r"""
import numpy as np, torch
import oracle
from paper_2112_01075_b200 import api, workloads as wl
import test_gpu_parity as T
import test_planner as TP
from _plancheck import types_of

assert api.LIB_PATH.endswith("_bounds.so")
assert api.debug_bounds_report()[0] == 0
variants = set()
variants |= T.random_problems_small_and_odd(600)
with api.tuning(bulk=0, gather=0):
    variants |= T.random_problems_small_and_odd(200)
with api.tuning(gather=2, zip=0, box=0):
    variants |= T.random_problems_small_and_odd(200)
with api.tuning(box=2):
    variants |= T.random_problems_small_and_odd(400)
with api.tuning(box=0):
    variants |= T.random_problems_small_and_odd(200)
for case in T.BOXES:
    T.test_super_box_kernels(*case)
for width in (0, 1, 4, 16):
    T.test_super_box_kernels_at_every_lane_group_width(width)
for values in ({"zip_walks": 0}, {"zip_walks": 2, "zip_by_range_slots": 1}, {"zip_walks": 4}):
    with api.tuning(**values):
        variants |= T.random_problems_small_and_odd(200)
for case in T.INTERLEAVED:
    T.test_gather_walk_and_zip_kernels(*case)
for case in T.SMALL_UNITS:
    T.test_short_run_kernels_on_one_and_two_byte_units(*case)
T.test_structured_probes_at_reduced_size()
for mesh, gshape, a1, a2, e, v in TP.KERNEL_CHOICE:
    if int(np.prod(gshape)) * e > (8 << 20):
        gshape = tuple(max(8, s // 8) if k else s for k, s in enumerate(gshape))
    G = np.random.default_rng(3).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    for mode in T.MODES:
        _, got = T.run_gpu(mesh, (gshape, a1), (gshape, a2), e, oracle.reslice(mesh, (gshape, a1), G), mode)
        T.assert_same(got, oracle.reslice(mesh, (gshape, a2), G), "kernel choice")
for w in wl.adversarial_problems():          # P1-P4 with every dimension reduced
    shape = [max(8, s // 4) // 8 * 8 for s in w.src.global_shape]
    ws = w.scaled(shape)
    src, dst, tiles, want = T.make_case(ws)
    for mode in (api.FUSE_ADJACENT, api.FUSE_NONE):
        _, got = T.run_gpu(ws.mesh_shape, src, dst, ws.elem_bytes, tiles, mode)
        T.assert_same(got, want, ws.name)
for w in T.MEDIUM:
    src, dst, tiles, want = T.make_case(w)
    for mode in T.MODES:
        _, got = T.run_gpu(w.mesh_shape, src, dst, w.elem_bytes, tiles, mode)
        T.assert_same(got, want, w.name)
torch.cuda.synchronize()
assert variants >= {0, 1, 2, 3, 4, 5, 6, 7, 8}, variants
rep = api.debug_bounds_report()
assert rep[0] == 0, "out-of-range access skipped: count %d, line %d, block %d, side %d, distance %d" % rep
assert api.redist_bulk_timeouts() == 0

# positive control: the checks are told that every tile ends 16 bytes early; the last accesses of every
# tile must then fail their test, be skipped (those target bytes keep their fill) and be counted
hits = 0
for mesh, gshape, a1, a2, e, v in TP.KERNEL_CHOICE[1:]:
    G = np.random.default_rng(4).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    with api.tuning(test_shrink_tiles=16):
        plan = api.Plan(mesh, (gshape, a1), (gshape, a2), e)
    tiles = oracle.reslice(mesh, (gshape, a1), G)
    mem = T.Carved(torch, tiles, plan.n_devices, plan.local_elems(1) * e, plan.scratch_bytes)
    plan.execute(mem.src, mem.dst, mem.scratch)
    mem.check("positive control")
    rep = api.debug_bounds_report()
    assert rep[0] > 0 and rep[3] in (1, 2), (v, rep)
    want = oracle.reslice(mesh, (gshape, a2), G)
    # what was skipped is missing from the result
    assert any(not np.array_equal(got, want[d].reshape(-1)) for d, got in enumerate(mem.results())), v
    hits += 1
assert hits == len(TP.KERNEL_CHOICE) - 1
print("checked build ok", sorted(variants))
"""


def test_checked_build_finds_no_access_outside_the_tiles():
    assert os.path.exists(BOUNDS_LIB), "build the checked library with python -m paper_2112_01075_b200.build"
    out = run_fresh(CHECKED_RUN, {"REDIST_LIB": BOUNDS_LIB})
    assert "checked build ok" in out


# variant -> (mesh, global shape, source axes, target axes, element bytes): small problems of at most 16 blocks
TIMEOUT_CASES = {
    4: ((2,), (64, 2048), ((0,), ()), ((), (0,)), 2),          # aligned 2 KiB runs: plain bulk copies, 16 blocks
    6: ((2,), (16, 2050), ((), (0,)), ((), ()), 4),            # ragged 4100-byte runs: bulk-loaded chunk walk, 8 blocks
    7: ((2,), (1024, 24), ((), (0,)), ((), ()), 4),            # 48-byte runs zipped through shared memory, 7 blocks
    8: ((2, 2), (8, 8, 24, 12), ((), (), (0,), (1,)), ((), (0,), (), ()), 4),    # super-boxes, 16 blocks
}

TIMEOUT_RUN = r"""
import numpy as np, torch
import oracle
from paper_2112_01075_b200 import api
import test_gpu_parity as T
from test_gpu_safety import TIMEOUT_CASES

for variant, (mesh, gshape, a1, a2, e) in sorted(TIMEOUT_CASES.items()):
    src, dst = (gshape, a1), (gshape, a2)
    G = np.random.default_rng(variant).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    tiles, want = oracle.reslice(mesh, src, G), oracle.reslice(mesh, dst, G)
    with api.tuning(test_extra_tx=16, wait_polls=4096, box=2 if variant == 8 else 0):
        broken = api.Plan(mesh, src, dst, e)
    li = broken.launch_info(0)
    assert broken.num_launches == 1 and li.variant == variant and 1 <= li.n_items <= 16, (variant, li.variant, li.n_items)
    before = api.redist_bulk_timeouts()
    mem = T.Carved(torch, tiles, broken.n_devices, broken.local_elems(1) * e, 0)
    broken.execute(mem.src, mem.dst)
    torch.cuda.synchronize()                                   # the kernel returned: no hang, no error
    assert api.redist_bulk_timeouts() == before + li.n_items   # every block counted itself once
    mem.check("wait ran out")
    for got in mem.results():
        assert np.all(got == 0xEE)                             # nothing was stored
    # the context is still usable and a normal run is exact and counts nothing
    _, got = T.run_gpu(mesh, src, dst, e, tiles)
    T.assert_same(got, want, "after a timed-out launch")
    assert api.redist_bulk_timeouts() == before + li.n_items
print("timeouts ok")
"""


def test_bounded_wait_runs_out_without_hanging_or_storing():
    out = run_fresh(TIMEOUT_RUN)
    assert "timeouts ok" in out
