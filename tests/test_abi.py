"""The C-ABI library loads without a GPU and exports every symbol include/redist.h declares."""
import ctypes
import os
import re

from paper_2112_01075_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "redist.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(redist_[a-z_]+)\s*\(", text))
    return names


def test_header_and_binding_agree():
    assert declared_functions() == set(api.EXPORTS)


def test_library_exports_every_declared_symbol():
    lib = api.load()
    for name in declared_functions():
        assert getattr(lib, name) is not None, name


def test_host_only_entry_points_work_without_a_gpu():
    p = api.Plan((2, 2), ((8, 8), ((0,), (1,))), ((8, 8), ((1,), (0,))), 4)
    assert p.n_devices == 4 and p.num_steps == 1 and p.scratch_bytes == 0
    assert api._status_string(4).startswith("source and target")
    info = p.step_info(0)
    assert api.STEP_KINDS[info.kind] == "allpermute" and info.cost == 16
    assert list(info.local_after)[:2] == [4, 4]
    li = p.launch_info(0)
    assert li.bytes_read == li.bytes_written == 8 * 8 * 4
    d = p.describe()
    assert d["n_devices"] == 4 and len(d["launches"]) == 1
    assert api.load().redist_last_cuda_error() == 0
    # null handles are tolerated by the queries
    lib = api.load()
    assert lib.redist_plan_num_devices(None) == 0
    lib.redist_plan_destroy(None)
    assert lib.redist_plan_step_info(None, 0, ctypes.byref(api.StepInfo())) == 1


def test_execute_rejects_bad_buffers_before_touching_the_gpu():
    p = api.Plan((2,), ((8, 8), ((0,), ())), ((8, 8), ((), (0,))), 4, api.FUSE_NONE)
    import pytest
    with pytest.raises(api.RedistError) as e:
        p.execute_ptrs([0, 0], [0, 0])
    assert e.value.status == 1                      # null tile pointers
    with pytest.raises(api.RedistError) as e:
        p.execute_ptrs([4096, 8192], [4096 + 8, 12288])
    assert e.value.status in (6, 7)                 # misaligned / overlapping
    with pytest.raises(api.RedistError) as e:
        p.execute_ptrs([4096, 8192], [4096 + 64, 12288])
    assert e.value.status == 6                      # a destination overlaps a source
    with pytest.raises(api.RedistError) as e:
        p.execute_ptrs([4096, 4096], [12288, 12288 + 64])
    assert e.value.status == 6                      # two destinations overlap
    q = api.Plan((2, 2), ((8, 8), ((0,), (1,))), ((8, 8), ((), (0, 1))), 4, api.FUSE_NONE)
    if q.scratch_bytes:
        with pytest.raises(api.RedistError) as e:
            q.execute_ptrs([4096 * (i + 1) for i in range(4)], [65536 + 4096 * i for i in range(4)])
        assert e.value.status == 5                  # scratch missing


def test_every_tensor_entry_point_checks_its_tiles_before_the_foreign_call():
    """execute, execute_static and execute_host share one check: a wrong number of tiles, a tile of the
    wrong size, a non-contiguous tile or a tile in the wrong memory is refused with EINVAL before the
    library sees a pointer (the C entry points cannot know how large the caller's buffers are)."""
    import pytest
    torch = pytest.importorskip("torch")
    p = api.Plan((2,), ((8, 8), ((0,), ())), ((8, 8), ((), (0,))), 4, api.FUSE_NONE)
    good = [torch.zeros(128, dtype=torch.uint8) for _ in range(2)]
    short = [torch.zeros(112, dtype=torch.uint8), good[1]]
    strided = [torch.zeros(256, dtype=torch.uint8)[::2], good[1]]
    for call in (p.execute, p.execute_static):
        for s, d in ((good[:1], good), (good, good + good), (short, good), (good, short), (strided, good), (good, good)):
            with pytest.raises(api.RedistError) as e:
                call(s, d)                      # the last pair is well-shaped but lives in host memory
            assert e.value.status == 1
    for s, d in ((good[:1], good), (short, good), (good, strided)):
        with pytest.raises(api.RedistError) as e:
            p.execute_host(s, d, None, None)
        assert e.value.status == 1
    with pytest.raises(api.RedistError) as e:
        p.bind([4096], [8192, 12288])
    assert e.value.status == 1


def test_pretty_prints_the_sequence_in_the_papers_notation():
    p = api.Plan((4, 2), ((8, 2048, 4096), ((0,), (), (1,))), ((8, 2048, 4096), ((), (0, 1), ())), 2)
    text = p.pretty(("x", "y"))
    lines = text.splitlines()
    assert lines[0] == "[2{x.0,x.1}8, 2048, 2048{y}4096]"
    assert lines[2].endswith("[8, 256{x.0,x.1,y}2048, 4096]") and "alltoall" in lines[1] and "alltoall" in lines[2]
    assert "launch fused: steps 0..1, src -> dst" in text and "scratch per device 0 B" in text
