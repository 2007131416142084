"""The entry point for callers that cannot allocate device memory (``redist_execute_static``).

A plug-in that receives its tiles from a host framework but may not call cudaMalloc -- because the
process gave all device memory to a pool at start-up, or because an allocation on its path could
fail or stall -- still has to run unfused plans, whose intermediates need scratch.  The library
serves those from a fixed array inside its own image.  Checked here through the C boundary: two
calls in a row must give exactly the bytes the ordinary entry point gives with a scratch buffer
the test allocates (the second call finds the first call's leftovers in the array), and a plan
that needs more than the array holds must be refused.

Collected last on purpose, so a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest

import oracle
from paper_2112_01075_b200 import api, workloads as wl

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def tiles_for(w, seed):
    src = (w.src.global_shape, w.src.axes)
    G = wl.global_array_bytes(w.src.global_shape, w.elem_bytes, "random_bits", seed)
    return oracle.reslice(w.mesh_shape, src, G)


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    # two alltoalls, unfused: one intermediate per virtual device lives in scratch
    w = wl.config2().scaled((8, 128, 512))
    plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, api.FUSE_NONE)
    assert plan.num_launches == 2 and 0 < plan.scratch_bytes <= api.STATIC_SCRATCH_BYTES
    nb = plan.local_elems(1) * w.elem_bytes
    for seed in (1, 2):                                   # second call: other data, dirty array
        d_src = [torch.from_numpy(t).cuda() for t in tiles_for(w, seed)]
        ref = [torch.full((nb,), 0xEE, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
        got = [torch.full((nb,), 0x11, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
        plan.execute(d_src, ref, plan.alloc_scratch())    # existing entry point, scratch from torch
        plan.execute_static(d_src, got)                   # new entry point, nothing allocated
        torch.cuda.synchronize()
        for d in range(plan.n_devices):
            assert torch.equal(got[d], ref[d]), f"call with seed {seed}: device {d} differs"


def test_static_scratch_three_step_plan_uses_both_slots():
    mesh = (2, 3, 2)
    src = ((12, 12, 8), ((0,), (1,), ()))
    dst = ((12, 12, 8), ((1,), (), (0,)))
    plan = api.Plan(mesh, src, dst, 4, api.FUSE_NONE)         # dynslice, alltoall, allpermute, allgather
    assert plan.num_launches >= 3 and plan.scratch_bytes_per_device == 2 * 512
    G = np.random.default_rng(7).integers(0, 256, size=(12, 12, 8, 4), dtype=np.uint8)
    want = oracle.reslice(mesh, dst, G)
    d_src = [torch.from_numpy(t).cuda() for t in oracle.reslice(mesh, src, G)]
    nb = plan.local_elems(1) * 4
    for _ in range(2):
        got = [torch.zeros(nb, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
        plan.execute_static(d_src, got)
        torch.cuda.synchronize()
        for d in range(plan.n_devices):
            assert np.array_equal(got[d].cpu().numpy(), want[d].reshape(-1))


def test_plans_beyond_the_built_in_array_are_refused():
    w = wl.config2()                                      # unfused: 16 MiB per virtual device
    plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, api.FUSE_NONE)
    assert plan.scratch_bytes > api.STATIC_SCRATCH_BYTES
    nb = plan.local_elems(0) * w.elem_bytes
    src = [torch.empty(nb, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
    dst = [torch.full((nb,), 0xEE, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
    with pytest.raises(api.RedistError) as e:
        plan.execute_static(src, dst)
    assert e.value.status == 5                            # refused ...
    torch.cuda.synchronize()
    assert all(bool((t == 0xEE).all()) for t in dst)      # ... before anything ran


STATIC_CASES = [   # mesh, global shape, source axes, target axes, element bytes: small plans that need scratch when unfused
    ((4, 2), (8, 256, 512), ((0,), (), (1,)), ((), (0, 1), ()), 2),       # two alltoalls, aligned 512-byte runs (bulk copies)
    ((2, 3, 2), (12, 12, 8), ((0,), (1,), ()), ((1,), (), (0,)), 4),      # four steps, both scratch slots, short runs
    ((2, 2, 2), (8, 6, 60), ((0,), (), (1, 2)), ((2,), (0,), ()), 4),     # interleaving short runs (zip / gather / units)
    ((2, 2), (6, 70, 6), ((0,), (), ()), ((), (1,), ()), 4),              # ragged runs of a few hundred bytes
    ((2, 2), (16, 6, 4), ((), (0,), ()), ((1,), (), (0,)), 8),            # 8-byte pieces
]


@pytest.mark.parametrize("mesh,gshape,a1,a2,e", STATIC_CASES)
def test_static_scratch_stays_inside_the_callers_tiles(mesh, gshape, a1, a2, e):
    """The built-in array replaces the scratch buffer and nothing else: with the caller's tiles carved out
    of one canary-filled buffer (16-byte alignment and no better, guard bands around every destination
    tile) the result is the oracle's, every guard byte survives, and no bounded wait ran out."""
    from _buffers import Carved
    src, dst = (gshape, a1), (gshape, a2)
    G = np.random.default_rng(len(gshape) + e).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    want = oracle.reslice(mesh, dst, G)
    tiles = oracle.reslice(mesh, src, G)
    seen = set()
    for flags in (api.FUSE_NONE, api.FUSE_ADJACENT):
        plan = api.Plan(mesh, src, dst, e, flags)
        assert plan.scratch_bytes <= api.STATIC_SCRATCH_BYTES
        seen.add(plan.scratch_bytes > 0)
        mem = Carved(torch, tiles, plan.n_devices, plan.local_elems(1) * e, 0)
        plan.execute_static(mem.src, mem.dst)
        mem.check(f"static scratch {mesh} {src} -> {dst}")
        for d, got in enumerate(mem.results()):
            assert np.array_equal(got, want[d].reshape(-1)), f"device {d} differs"
    assert True in seen                                   # the unfused plan did use the built-in array
    assert api.redist_bulk_timeouts() == 0


def test_static_entry_point_checks_its_tiles_before_the_foreign_call():
    """Wrong count, wrong size and non-contiguous tiles are refused in the binding: the C entry point
    cannot know how large the caller's buffers are."""
    w = wl.config2().scaled((8, 128, 512))
    plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, api.FUSE_NONE)
    n, sb, db = plan.n_devices, plan.local_elems(0) * w.elem_bytes, plan.local_elems(1) * w.elem_bytes
    good_s = [torch.zeros(sb, dtype=torch.uint8, device="cuda") for _ in range(n)]
    good_d = [torch.zeros(db, dtype=torch.uint8, device="cuda") for _ in range(n)]
    for bad_s, bad_d in ((good_s[:-1], good_d), (good_s, good_d + good_d[:1]),
                         (good_s, [torch.zeros(db - 16, dtype=torch.uint8, device="cuda")] + good_d[1:]),
                         ([torch.zeros(2 * sb, dtype=torch.uint8, device="cuda")[::2]] + good_s[1:], good_d),
                         ([t.cpu() for t in good_s], good_d)):
        with pytest.raises(api.RedistError) as e:
            plan.execute_static(bad_s, bad_d)
        assert e.value.status == 1
    plan.execute_static(good_s, good_d)
    torch.cuda.synchronize()
