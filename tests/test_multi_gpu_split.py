"""Byte accounting for virtual devices spread over several GPUs (``redist_plan_gpu_split``), host only.

The paper's setting is one device per accelerator (Section 8) and its Discussion (Section 9) raises
device-to-device transfers derived from the base offset maps.  The library only *accounts* for that
setting: per launch, the matrix of bytes by reading GPU and receiving GPU.  Checked here against a brute
force over every element of every target tile, written with the oracle's base offsets."""
import numpy as np
import pytest

import oracle
from paper_2112_01075_b200 import api, workloads as wl
from test_planner import random_problem


def brute_matrix(mesh, src, dst, e, n_gpus):
    """Every element of every target tile: which GPU holds the source tile it comes from (a replica on the
    receiving GPU if there is one, else the lowest-numbered holder), which GPU receives it."""
    n = int(np.prod(mesh))
    per = n // n_gpus
    tile_s, off_s = oracle.base_offsets(mesh, src)
    tile_d, off_d = oracle.base_offsets(mesh, dst)
    gshape = src[0]
    holders = {}
    for d in range(n):
        holders.setdefault(tuple(int(o) for o in off_s[d]), []).append(d)
    m = np.zeros((n_gpus, n_gpus), dtype=np.int64)
    for d in range(n):
        gd = d // per
        for idx in np.ndindex(*tile_d):
            g = [int(o) + i for o, i in zip(off_d[d], idx)]
            key = tuple(x // c * c for x, c in zip(g, tile_s))
            hs = holders[key]
            local = [h for h in hs if h // per == gd]
            gs = gd if local else hs[0] // per
            m[gs, gd] += e
    return m.tolist()


@pytest.mark.parametrize("mesh,gpus", [((2, 2), (1, 2, 4)), ((4, 3), (1, 2, 4, 12)), ((2, 2, 2), (1, 2, 4, 8)), ((6, 2), (2, 3, 6))])
def test_split_matches_brute_force(mesh, gpus):
    rng = np.random.default_rng(sum(mesh))
    for _ in range(12):
        src, dst = random_problem(rng, mesh, max_rank=3, mult=2)
        e = int(rng.choice([1, 2, 4]))
        plan = api.Plan(mesh, src, dst, e, api.FUSE_ALL)
        assert plan.num_launches == 1
        li = plan.launch_info(0)
        for g in gpus:
            m = plan.gpu_split(g, 0)
            assert m == brute_matrix(mesh, src, dst, e, g), (mesh, src, dst, g)
            assert sum(map(sum, m)) == li.bytes_written
        assert plan.gpu_split(1, 0) == [[li.bytes_written]]          # one GPU: today's launch


def test_every_launch_of_an_unfused_plan_accounts_for_all_its_bytes():
    for w in wl.config4(30, (16, 32, 64, 128)):
        plan = api.Plan(w.mesh_shape, w.src, w.dst, 4, api.FUSE_NONE)
        for q in range(plan.num_launches):
            li = plan.launch_info(q)
            for g in (1, 2, 8, 16):                                   # prefixes of the mesh (2, 4, 2)
                m = plan.gpu_split(g, q)
                assert sum(map(sum, m)) == li.bytes_written
                if li.kernel == 0:                                    # dynslice is purely local (Appendix B)
                    assert all(m[s][t] == 0 for s in range(g) for t in range(g) if s != t)


def test_benchmark_configurations_on_eight_gpus():
    """What would cross NVLink if the 64 virtual devices of config 5 sat on 8 GPUs (mesh axis x and half of
    y choose the GPU): the permutation of 5a and the fused alltoall + permutation of 5b move 3/4 and 7/8
    of the array between GPUs; config 3c's allgather to replicas sends every GPU the other seven's parts."""
    b = wl.bench_workloads()
    w = b["c5a"]
    m = api.Plan(w.mesh_shape, w.src, w.dst, 2).gpu_split(8, 0)
    total = sum(map(sum, m))
    assert total == 2 * 2**30 and sum(m[g][g] for g in range(8)) * 4 == total
    w = b["c5b"]
    m = api.Plan(w.mesh_shape, w.src, w.dst, 2).gpu_split(8, 0)
    assert sum(map(sum, m)) == 2 * 2**30 and sum(m[g][g] for g in range(8)) * 8 == 2 * 2**30
    w = b["c3c"]
    m = api.Plan(w.mesh_shape, w.src, w.dst, 2).gpu_split(8, 0)
    assert all(m[s][t] == 64 * 2**20 for s in range(8) for t in range(8))


def test_only_prefixes_of_the_mesh_are_accepted():
    plan = api.Plan((4, 3), ((24, 12), ((0,), (1,))), ((24, 12), ((1,), (0,))), 4)
    for g in (3, 5, 6, 8, 24):
        with pytest.raises(api.RedistError) as e:
            plan.gpu_split(g, 0)
        assert e.value.status == 1
    with pytest.raises(api.RedistError):
        plan.gpu_split(2, 7)
