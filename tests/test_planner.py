"""Planner (host) tests through the C boundary: typed sequences are replayed with the paper's rules
on real data and compared with the oracle after every step; launch descriptors are interpreted in
numpy; costs are compared with the paper's examples and with a brute-force optimum."""
import heapq
import itertools

import os

import numpy as np
import pytest

from oracle import collectives as C
from paper_2112_01075_b200 import api, workloads as wl
from _plancheck import check_plan, types_of

MODES = [api.FUSE_ADJACENT, api.FUSE_NONE, api.FUSE_ALL, api.NAIVE]


def small(w, shape):
    return w.scaled(shape)


SCALED = [
    small(wl.config1(), (8, 8)),
    small(wl.config1().reversed(), (8, 8)),
    small(wl.config2(), (8, 32, 16)),
    small(wl.config2().reversed(), (8, 32, 16)),
    small(wl.config3("a"), (16, 32)),
    small(wl.config3("b"), (16, 32)),
    small(wl.config3("c"), (16, 32)),
    small(wl.config5("a"), (64, 32)),
    small(wl.config5("b"), (64, 64)),
]


@pytest.mark.parametrize("w", SCALED, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", MODES)
def test_benchmark_shapes_scaled_down(w, mode):
    src, dst = types_of(w)
    check_plan(w.mesh_shape, src, dst, w.elem_bytes, mode)


def test_expected_sequences_for_the_benchmark_configurations():
    exp = {"c1": ["allpermute"], "c2": ["alltoall", "alltoall"], "c2_back": ["alltoall", "alltoall"],
           "c3a": ["alltoall"], "c3b": ["dynslice"], "c3c": ["allgather"], "c5a": ["allpermute"],
           "c5b": ["alltoall", "allpermute"]}
    for name, kinds in exp.items():
        w = wl.bench_workloads()[name]
        p = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes)
        assert p.step_kinds() == kinds, name
        assert p.num_launches == 1 and p.scratch_bytes == 0
        assert p.height <= max(p.local_elems(0), p.local_elems(1))
        rd, wr = p.bytes_moved()
        assert rd == w.global_elems * w.elem_bytes
        assert wr == p.n_devices * p.local_elems(1) * w.elem_bytes
        un = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, api.FUSE_NONE)
        assert un.num_launches == len(kinds)
        assert un.scratch_bytes_per_device <= 2 * (max(p.local_elems(0), p.local_elems(1)) * w.elem_bytes + 255)


def random_problem(rng, mesh, max_rank=3, mult=2):
    rank = int(rng.integers(1, max_rank + 1))

    def draw():
        per = [[] for _ in range(rank)]
        for a in range(len(mesh)):
            c = int(rng.integers(0, rank + 1))
            if c < rank:
                per[c].append(a)
        return tuple(tuple(ax[i] for i in rng.permutation(len(ax))) if ax else () for ax in per)

    a1, a2 = draw(), draw()
    gshape = []
    for k in range(rank):
        f1 = int(np.prod([mesh[a] for a in a1[k]], dtype=np.int64))
        f2 = int(np.prod([mesh[a] for a in a2[k]], dtype=np.int64))
        gshape.append(int(np.lcm(f1, f2)) * int(rng.integers(1, mult + 1)))
    return (tuple(gshape), a1), (tuple(gshape), a2)


@pytest.mark.parametrize("mesh", [(2, 2), (4,), (2, 3), (4, 6), (2, 4, 2), (3, 3), (6, 2), (8,), (2, 2, 2, 2)])
def test_random_problems_every_step_checked(mesh):
    rng = np.random.default_rng(sum(mesh) * 31 + len(mesh))
    for t in range(24):
        src, dst = random_problem(rng, mesh)
        e = int(rng.choice([1, 2, 4, 8, 16]))
        mode = MODES[t % 4]
        check_plan(mesh, src, dst, e, mode, seed=t)


def test_random_problems_element_sized_runs():
    """Last dimension fully sharded: runs of a single element, vector width = element size."""
    rng = np.random.default_rng(99)
    for t in range(20):
        mesh = (2, 3, 2)
        src, dst = random_problem(rng, mesh, max_rank=2, mult=1)
        check_plan(mesh, src, dst, int(rng.choice([1, 2, 4])), MODES[t % 3], seed=t)


def test_identity_is_a_copy():
    mesh = (2, 2)
    t = ((8, 8), ((0,), (1,)))
    d = check_plan(mesh, t, t, 4)
    assert d["steps"] == [] and len(d["launches"]) == 1 and d["launches"][0]["kernel"] == "copy"


def test_size_one_axes_and_empty_mesh():
    check_plan((1, 2, 1), ((4, 4), ((0, 1), (2,))), ((4, 4), ((), (1,))), 2)
    check_plan((), ((3, 5), ((), ())), ((3, 5), ((), ())), 1)
    check_plan((1,), ((3,), ((0,),)), ((3,), ((),)), 1)


# ------------------------------------------------------------------------- the paper's examples

@pytest.mark.parametrize("w", wl.adversarial_problems(), ids=lambda w: w.name)
def test_adversarial_table_problems(w):
    """P1-P4 as printed (axis sizes inline, 4-byte elements): the printed global sizes follow from the
    shapes, and the synthesized sequences avoid the full allgather the paper says its method never
    issues (they use dynslice / alltoall / allpermute, and for P4 allgathers within the bound)."""
    mib = {"P1": 162, "P2": 113, "P3": 127, "P4": 64}[w.name]
    assert abs(w.global_elems * 4 / 2**20 - mib) <= 0.5          # printed sizes are rounded MiB
    p = api.Plan(w.mesh_shape, w.src, w.dst, 4)
    assert p.height <= max(p.local_elems(0), p.local_elems(1))
    if w.name != "P4":
        assert "allgather" not in p.step_kinds()
    # replay every step on a scaled-down array with the same types (divide every dimension by its gcd
    # with the printed size so that tiles stay integral)
    small = {"P1": (8, 8, 8), "P2": (4, 4, 4, 4), "P3": (8, 4, 4), "P4": (2, 2, 2, 2, 2, 2)}[w.name]
    ws = w.scaled(small)
    src, dst = types_of(ws)
    for mode in MODES:
        check_plan(ws.mesh_shape, src, dst, 4, mode)


def test_merged_alltoall_example():
    """[1{a}8, 8] -> [8, 1{a}8] over {a:8}: one merged alltoall of cost 8, no permutation."""
    d = check_plan((8,), ((8, 8), ((0,), ())), ((8, 8), ((), (0,))), 4)
    assert [s["kind"] for s in d["steps"]] == ["alltoall"]
    assert d["steps"][0]["factor"] == 8 and d["cost"] == 8
    assert [p["size"] for p in d["primes"]] == [2, 2, 2]


def test_factor_decomposition_example():
    """[3{x}12, 2{y}12] -> [2{y}12, 3{x}12] over {x:4, y:6} without gathering everything: the
    paper's sequence uses two alltoalls (cost 2*6) plus permutations; memory stays at 6 elements."""
    d = check_plan((4, 6), ((12, 12), ((0,), (1,))), ((12, 12), ((1,), (0,))), 4)
    kinds = [s["kind"] for s in d["steps"]]
    assert kinds.count("allgather") == 0 and kinds.count("dynslice") == 0
    assert d["height"] == 6
    assert sum(s["cost"] for s in d["steps"] if s["kind"] == "alltoall") == 12
    assert [p["size"] for p in d["primes"]] == [2, 2, 2, 3]


def test_oversharding_example_cost_bounds():
    """Mesh {x:4, y:2, z:4}: the printed sequences cost 512 and 384; the search may not do worse than
    the better one on the weak graph (the search of Section 7.3 gives the final permutation no edge weight)."""
    mesh, gshape = (4, 2, 4), (8, 8, 8, 4)
    src, dst = (gshape, ((1, 0), (), (), ())), (gshape, ((), (1,), (0,), ()))
    d = check_plan(mesh, src, dst, 4)
    weak_cost = sum(s["cost"] for s in d["steps"] if s["kind"] != "allpermute")
    assert weak_cost <= 384
    assert any(s["kind"] == "dynslice" for s in d["steps"])         # over-partitioning happens
    d2 = check_plan(mesh, src, dst, 4, api.FUSE_ADJACENT | api.NO_OVERPARTITION)
    assert not any(s["kind"] == "dynslice" for s in d2["steps"])
    assert sum(s["cost"] for s in d2["steps"] if s["kind"] != "allpermute") == 512


def test_dynslice_picks_the_axis_of_the_target():
    """[16] -> [4{x}16] on {x:4, y:4}: slicing along y would need a permutation afterwards."""
    d = check_plan((4, 4), ((16,), ((),)), ((16,), ((0,),)), 4)
    assert [s["kind"] for s in d["steps"]] == ["dynslice"]
    d = check_plan((4, 4), ((16,), ((),)), ((16,), ((1,),)), 4)
    assert [s["kind"] for s in d["steps"]] == ["dynslice"]


def test_permutation_examples_are_single_permutes():
    mesh = (4, 4)
    for src, dst in [(((1024, 128), ((1, 0), ())), ((1024, 128), ((0, 1), ()))),
                     (((128, 64), ((0,), (1,))), ((128, 64), ((1,), (0,)))),
                     (((128,), ((0,),)), ((128,), ((1,),)))]:
        d = check_plan(mesh, src, dst, 2)
        assert [s["kind"] for s in d["steps"]] == ["allpermute"]


def test_collective_sequence_examples_cost_no_more_than_printed():
    """Figure with six sequences on {x:4, y:4}: the search is at least as cheap as either column."""
    mesh = (4, 4)
    g2, g3 = (512, 128), (128, 512, 128)
    cases = [((g2, ((0, 1), ())), (g2, ((0,), (1,))), 32 * 128 * 2),                 # alltoall + permute
             ((g3, ((0,), (), (1,))), (g3, ((), (1, 0), ())), 2 * 32 * 512 * 32),    # two alltoalls
             ((g3, ((0,), (), (1,))), (g3, ((), (1,), ())), 32 * 512 * 32 + 128 * 128 * 128)]
    for src, dst, printed in cases:
        d = check_plan(mesh, src, dst, 2)
        assert d["cost"] <= printed


def test_permute_is_hoisted_before_trailing_allgathers():
    """Section 7.3: a needed permutation moves in front of the final allgathers (smaller tiles)."""
    rng = np.random.default_rng(4)
    seen = 0
    for t in range(400):
        src, dst = random_problem(rng, (2, 2, 3), max_rank=2)
        p = api.Plan((2, 2, 3), src, dst, 4)
        kinds = p.step_kinds()
        if "allpermute" in kinds and "allgather" in kinds:
            assert kinds.index("allpermute") < kinds.index("allgather")
            i = kinds.index("allpermute")
            assert p.step_info(i).cost <= min(p.local_elems(1), p.step_info(len(kinds) - 1).localsize_after)
            seen += 1
        p.close()
    assert seen > 0


# --------------------------------------------------------------------------------- error paths

def test_error_statuses():
    with pytest.raises(api.RedistError) as e:
        api.Plan((4, 8), ((512, 1024), ((), (0,))), ((1024, 1024), ((), (0,))), 4)
    assert e.value.status == 4                                  # different global arrays
    with pytest.raises(api.RedistError) as e:
        api.Plan((4, 8), ((128, 256), ((0,), (1,))), ((1024, 32), ((0, 1), ())), 4)
    assert e.value.status == 4
    with pytest.raises(api.RedistError) as e:
        api.Plan((4, 8), ((128, 256), ((0,), (0,))), ((128, 256), ((), ())), 4)
    assert e.value.status == 2                                  # axis listed twice
    with pytest.raises(api.RedistError) as e:
        api.Plan((4, 8), ((128, 256), ((5,), ())), ((128, 256), ((), ())), 4)
    assert e.value.status == 2                                  # axis not in the mesh
    with pytest.raises(api.RedistError) as e:
        api.Plan((4, 8), ((6, 256), ((0,), ())), ((6, 256), ((), ())), 4)
    assert e.value.status == 3                                  # 4 does not divide 6
    with pytest.raises(api.RedistError) as e:
        api.Plan((2,), ((4,), ((0,),)), ((4,), ((),)), 3)
    assert e.value.status == 1                                  # element size
    with pytest.raises(api.RedistError) as e:
        api.Plan((2048,), ((4096,), ((0,),)), ((4096,), ((),)), 4)
    assert e.value.status == 10                                 # more virtual devices than supported
    with pytest.raises(api.RedistError) as e:
        api.Plan((2,), ((4,), ((0,),)), ((4,), ((),)), 4, flags=128)
    assert e.value.status == 1


def test_base_offsets_match_the_oracle():
    import oracle
    rng = np.random.default_rng(8)
    for mesh in [(2, 2), (4, 6), (2, 4, 2)]:
        for _ in range(10):
            src, _ = random_problem(rng, mesh)
            tile, off = api.redist_base_offsets(mesh, src)
            otile, ooff = oracle.base_offsets(mesh, src)
            assert tile == otile and np.array_equal(np.array(off), ooff)


# ------------------------------------------------------------- near optimality, brute force

def all_strong_types(mesh, gshape):
    """Every well-formed type over the (prime) mesh: each axis unused or in one dimension, ordered."""
    rank = len(gshape)
    out = set()
    for assign in itertools.product(range(rank + 1), repeat=len(mesh)):
        per = [[a for a in range(len(mesh)) if assign[a] == k] for k in range(rank)]
        for orders in itertools.product(*[list(itertools.permutations(ax)) for ax in per]):
            t = tuple(tuple(o) for o in orders)
            if C.well_formed(mesh, gshape, t):
                out.add(t)
    return out


def brute_force_optimum(mesh, gshape, a1, a2, lat=0, count_permute=True):
    """Dijkstra over strong types with the four typing rules (multi-axes forms included) and
    localsize <= M; returns the minimal cost of a memory-constrained sequence.  `lat` is added to every
    dynslice / alltoall / allgather; with `count_permute` off an allpermute is free (the view of the
    search of Section 7.3, which leaves the permutation out of the edge weights)."""
    M = max(C.localsize(mesh, gshape, a1), C.localsize(mesh, gshape, a2))
    nodes = [t for t in all_strong_types(mesh, gshape) if C.localsize(mesh, gshape, t) <= M]
    by_local = {}
    for t in nodes:
        by_local.setdefault(C.localtype(mesh, gshape, t), []).append(t)
    rank = len(gshape)
    dist = {C.norm_axes(a1): 0}
    pq = [(0, C.norm_axes(a1))]
    goal = C.norm_axes(a2)
    while pq:
        c, t = heapq.heappop(pq)
        if c > dist.get(t, 1 << 62):
            continue
        if t == goal:
            return c
        nxt = []
        L = C.localsize(mesh, gshape, t)
        for u in by_local[C.localtype(mesh, gshape, t)]:
            if u != t:
                nxt.append((u, L if count_permute else 0))
        unused = [a for a in range(len(mesh)) if a not in C.used_axes(t)]
        for i in range(rank):
            for n_ax in range(1, len(t[i]) + 1):
                u = C.t_allgather(mesh, gshape, t, i, n_ax)
                nxt.append((u, C.localsize(mesh, gshape, u) + lat))
                for j in range(rank):
                    if j != i:
                        try:
                            nxt.append((C.t_alltoall(mesh, gshape, t, i, j, n_ax), L + lat))
                        except C.TypeError_:
                            pass
            for k in range(1, len(unused) + 1):
                for seq in itertools.permutations(unused, k):
                    try:
                        nxt.append((C.t_dynslice(mesh, gshape, t, i, seq), lat))
                    except C.TypeError_:
                        pass
        for u, w in nxt:
            if C.localsize(mesh, gshape, u) > M:
                continue
            if c + w < dist.get(u, 1 << 62):
                dist[u] = c + w
                heapq.heappush(pq, (c + w, u))
    raise AssertionError("target unreachable")


@pytest.mark.parametrize("mesh", [(2, 2), (2, 3), (2, 2, 2), (2, 2, 3)])
def test_near_optimality_against_brute_force(mesh):
    """cost(plan) <= optimum over all memory-constrained sequences + localsize(target)."""
    rng = np.random.default_rng(len(mesh) * 7 + mesh[-1])
    for _ in range(10):
        src, dst = random_problem(rng, mesh, max_rank=2, mult=2)
        opt = brute_force_optimum(mesh, src[0], src[1], dst[1])
        p = api.Plan(mesh, src, dst, 4)
        assert p.cost <= opt + p.local_elems(1), (mesh, src, dst, p.cost, opt)
        weak = sum(p.step_info(s).cost for s in range(p.num_steps) if p.step_info(s).kind != 3)
        assert weak <= opt                                        # permutation-free part is optimal
        p.close()


def test_counting_the_permutation_example():
    """Mesh {a:2, b:2, c:3}, [2{c,a}12] -> [4{c}12].  The shortest weak path is a single allgather; lowered, it
    needs a permutation in front and costs 6 in total.  Slicing over the idle axis b first halves the
    tiles the permutation moves: 5 in total, the optimum over all sequences of the four typing rules.  Both plans are checked step by step against the rules and the oracle."""
    mesh, src, dst = (2, 2, 3), ((12,), ((2, 0),)), ((12,), ((2,),))
    d0 = check_plan(mesh, src, dst, 4)
    d1 = check_plan(mesh, src, dst, 4, api.COST_PERMUTE)
    assert (d0["cost"], d1["cost"]) == (6, 5)
    assert brute_force_optimum(mesh, src[0], src[1], dst[1]) == 5
    assert [s["kind"] for s in d1["steps"]] == ["dynslice", "allpermute", "allgather"]


@pytest.mark.parametrize("mesh", [(2, 2), (2, 3), (4, 6), (2, 4, 2), (6, 2), (2, 2, 3), (2, 2, 2, 2)])
def test_counting_the_permutation_never_costs_more(mesh):
    """REDIST_COST_PERMUTE: every plan is still a typed normal-form sequence inside the memory bound
    that ends in the oracle's tiles (check_plan), and its total cost is at most the default plan's."""
    rng = np.random.default_rng(sum(mesh) * 17 + len(mesh))
    for t in range(16):
        src, dst = random_problem(rng, mesh)
        e = int(rng.choice([1, 2, 4, 8, 16]))
        p0 = api.Plan(mesh, src, dst, e)
        d1 = check_plan(mesh, src, dst, e, api.COST_PERMUTE | MODES[t % 4], seed=t)
        assert d1["cost"] <= p0.cost
        p0.close()


def test_counting_the_permutation_on_evaluation_shaped_problems():
    """On problems of the evaluation's shape some plans get cheaper (a permutation avoided or moved to
    smaller tiles), none gets dearer, and the memory bound still holds."""
    better = 0
    for w in wl.evaluation_like_problems(200):
        p0 = api.Plan(w.mesh_shape, w.src, w.dst, 4)
        p1 = api.Plan(w.mesh_shape, w.src, w.dst, 4, api.COST_PERMUTE)
        assert p1.cost <= p0.cost
        assert p1.height <= max(p1.local_elems(0), p1.local_elems(1))
        assert p1.step_kinds().count("allpermute") <= 1
        better += p1.cost < p0.cost
        p0.close()
        p1.close()
    assert better > 0


def test_planner_throughput_on_evaluation_shaped_problems():
    """Section 8 reports synthesis in under a second per problem (unoptimised Python); the host planner
    here must stay far below that on 1000 problems of the same shape (3 mesh axes, up to 6-D), synthesized
    afresh (REDIST_NO_CACHE); asked for again, every one of them comes out of the plan cache."""
    import time
    ws = wl.evaluation_like_problems(1000)
    worst, t0 = 0.0, time.perf_counter()
    costs = []
    for w in ws:
        t1 = time.perf_counter()
        p = api.Plan(w.mesh_shape, w.src, w.dst, 4, api.NO_CACHE)
        worst = max(worst, time.perf_counter() - t1)
        assert p.height <= max(p.local_elems(0), p.local_elems(1))
        assert p.step_kinds().count("allpermute") <= 1
        costs.append(p.cost)
        p.close()
    total = time.perf_counter() - t0
    assert worst < 0.25 and total / len(ws) < 0.05, (worst, total)
    # the cache holds the 256 most recent plans: the last 200 problems, planned twice, hit the second time
    api.plan_cache_clear()
    recent = ws[-200:]
    for w in recent:
        api.Plan(w.mesh_shape, w.src, w.dst, 4).close()
    t0 = time.perf_counter()
    for w, c in zip(recent, costs[-200:]):
        p = api.Plan(w.mesh_shape, w.src, w.dst, 4)
        assert p.cost == c
        p.close()
    again = time.perf_counter() - t0
    hits, misses, entries = api.plan_cache_stats()
    assert (hits, misses, entries) == (200, 200, 200)
    assert again / 200 < total / len(ws)          # a hit costs less than a synthesis


def test_plan_cache_returns_the_same_plan_for_the_same_request():
    api.plan_cache_clear()
    mesh, src, dst = (4, 2), ((8, 64, 64), ((0,), (), (1,))), ((8, 64, 64), ((), (0, 1), ()))
    p1 = api.Plan(mesh, src, dst, 2)
    assert api.plan_cache_stats() == (0, 1, 1)
    p2 = api.Plan(mesh, src, dst, 2)
    assert api.plan_cache_stats() == (1, 1, 1)
    assert p1.describe() == p2.describe()
    p3 = api.Plan(mesh, src, dst, 2, api.NO_CACHE)                  # synthesized afresh, cache untouched
    assert api.plan_cache_stats() == (1, 1, 1) and p3.describe() == p1.describe()
    assert api.Plan(mesh, src, dst, 4).elem_bytes == 4 and api.plan_cache_stats() == (1, 2, 2)   # other element size
    assert api.Plan(mesh, src, dst, 2, api.FUSE_NONE).num_launches == 2 and api.plan_cache_stats() == (1, 3, 3)
    with api.tuning(bulk=0):                                         # other tuning values: another plan
        p4 = api.Plan(mesh, src, dst, 2)
    assert api.plan_cache_stats() == (1, 4, 4)
    assert p4.launch_info(0).variant != p1.launch_info(0).variant
    p1.close()                                                       # a handle is a reference: the others stay valid
    assert p2.step_kinds() == ["alltoall", "alltoall"] and p2.describe()["cost"] == p3.cost
    rng = np.random.default_rng(3)
    for _ in range(300):                                             # more distinct requests than the cache keeps
        g = tuple(int(v) * 4 for v in rng.integers(1, 50, size=2))
        api.Plan((2, 2), (g, ((0,), (1,))), (g, ((1,), (0,))), 4).close()
    assert api.plan_cache_stats()[2] <= 256
    api.plan_cache_clear()
    assert api.plan_cache_stats() == (0, 0, 0)


def test_tuning_values_are_validated_and_copied_into_new_plans_only():
    mesh, src, dst = (2,), ((64, 2048), ((0,), ())), ((64, 2048), ((), (0,)))      # aligned 4 KiB runs
    before = api.Plan(mesh, src, dst, 4, api.NO_CACHE)
    assert api.tuning_get("bulk") == 1
    with pytest.raises(api.RedistError):
        api.tuning_set("no_such_value", 1)
    with pytest.raises(api.RedistError):
        api.tuning_set("gather", 3)
    with api.tuning(bulk=0):
        assert api.tuning_get("bulk") == 0
        inside = api.Plan(mesh, src, dst, 4, api.NO_CACHE)
    assert api.tuning_get("bulk") == 1
    assert before.launch_info(0).variant == 4 and inside.launch_info(0).variant in (0, 1)
    assert api.Plan(mesh, src, dst, 4, api.NO_CACHE).launch_info(0).variant == 4


TUNING_VALUES = {   # name: (default, lowest, highest) as the header states them
    "bulk": (1, 0, 1), "gather": (1, 0, 2), "zip": (2, 0, 2), "box": (1, 0, 2), "box_width": (0, 0, 256),
    "zip_walks": (7, 0, 7), "zip_by_range_slots": (256, 1, 1 << 20), "item_kb": (0, 0, 1024), "l2_hint": (4, 0, 4), "piece": (1, 0, 1),
    "pdl": (1, 0, 1), "nvtx": (0, 0, 1), "step_latency": (0, 0, 1 << 50), "wait_polls": (1 << 18, 1, 1 << 30),
    "test_extra_tx": (0, 0, 1 << 20), "test_shrink_tiles": (0, 0, 1 << 20),
}


def test_every_tuning_value_has_its_documented_default_and_range():
    api.tuning_reset()
    header = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "redist.h")).read()
    for name, (default, lo, hi) in TUNING_VALUES.items():
        assert '"%s"' % name in header, name
        assert api.tuning_get(name) == default, name
        for bad in (lo - 1, hi + 1):
            with pytest.raises(api.RedistError):
                api.tuning_set(name, bad)
        for good in (lo, hi):
            api.tuning_set(name, good)
            assert api.tuning_get(name) == good
        api.tuning_reset()
        assert api.tuning_get(name) == default
    # the lanes per range of the super-box kernels: powers of two are taken, anything else leaves the choice to the library
    mesh, g = (4, 4, 4), (8, 12, 2, 28, 20, 12)
    a1, a2 = ((), (1,), (), (2,), (), ()), ((2,), (), (), (), (0,), (1,))
    def width(**values):
        with api.tuning(box=2, **values):
            geo = api.Plan(mesh, (g, a1), (g, a2), 4, api.NO_CACHE).describe()["launches"][0]["geometry"]
        assert geo["mode"] == 5
        return geo["zip_width"]
    chosen = width()
    assert width(box_width=8) == 8 and width(box_width=64) == 64 and width(box_width=24) == chosen
    # the evict-first policy of the plain bulk-copy kernels: stores only, and only from fan-out 4, unless told otherwise
    def hint(mesh, src, dst, **values):
        with api.tuning(**values):
            return api.Plan(mesh, src, dst, 2, api.NO_CACHE).describe()["launches"][0]["geometry"]["l2_hint"]
    rows, cols, repl = ((4096, 4096), ((0,), ())), ((4096, 4096), ((), (0,))), ((4096, 4096), ((), ()))
    assert hint((8,), rows, cols) == 0 and hint((8,), cols, repl) == 2 and hint((2,), cols, repl) == 0
    assert hint((8,), rows, cols, l2_hint=3) == 3 and hint((8,), cols, repl, l2_hint=0) == 0


@pytest.mark.parametrize("mesh", [(2, 2), (2, 3), (2, 2, 2), (2, 2, 3)])
def test_step_latency_buys_fewer_collectives(mesh):
    """Small transfers are bound by the latency of each collective, not by bytes (Section 8, third research
    question).  With the tuning value step_latency = 0 the plan is the default one; with a latency far
    above any byte cost the searched part of the plan (everything but the final permutation, which the
    search of Section 7.3 never weighs) has the fewest collectives any memory-constrained sequence can
    have, and among those the fewest bytes -- checked against a brute-force search over strong types.
    Every plan is still replayed step by step against the typing rules and the oracle."""
    big = 10 ** 9
    rng = np.random.default_rng(len(mesh) * 11 + mesh[-1])
    fewer = 0
    for _ in range(10):
        src, dst = random_problem(rng, mesh, max_rank=2, mult=2)
        d0 = check_plan(mesh, src, dst, 4)
        with api.tuning(step_latency=0):
            assert check_plan(mesh, src, dst, 4)["steps"] == d0["steps"]
        with api.tuning(step_latency=big):
            d1 = check_plan(mesh, src, dst, 4)
        searched = [s for s in d1["steps"] if s["kind"] != "allpermute"]
        opt = brute_force_optimum(mesh, src[0], src[1], dst[1], lat=big, count_permute=False)
        assert len(searched) == opt // big, (mesh, src, dst)
        assert sum(s["cost"] for s in searched) == opt % big, (mesh, src, dst)
        n0 = len([s for s in d0["steps"] if s["kind"] != "allpermute"])
        assert len(searched) <= n0
        fewer += len(searched) < n0
    return fewer


def test_step_latency_example():
    """The over-partitioning example of Section 7.2 on the mesh {x:4, y:2, z:4}: by bytes the cheapest
    sequence slices over the idle axis first, moves a quarter of the data and gathers at the end (cost
    384, four collectives); when every collective costs a large latency the two plain alltoalls of the
    figure's left column win (cost 512, two collectives)."""
    mesh, g = (4, 2, 4), (8, 8, 8, 4)
    src, dst = (g, ((1, 0), (), (), ())), (g, ((), (1,), (0,), ()))
    d0 = check_plan(mesh, src, dst, 4)
    with api.tuning(step_latency=10 ** 12):
        d1 = check_plan(mesh, src, dst, 4)
    assert ([s["kind"] for s in d0["steps"]], d0["cost"]) == (["dynslice", "alltoall", "allpermute", "allgather"], 384)
    assert ([s["kind"] for s in d1["steps"]], d1["cost"]) == (["alltoall", "alltoall"], 512)


def test_no_overpartition_flag_only_filters_the_axes_it_slices():
    """Regression: the ban on over-partitioning must look only at the primes a dynslice introduces.
    [7, 4{b}4... a dimension sharded 5 ways that has to end sharded 3 ways still needs dynslice(3)."""
    mesh = (3, 2, 5)
    src, dst = ((7, 4, 30), ((), (1,), (2,))), ((7, 4, 30), ((), (1,), (0,)))
    a = check_plan(mesh, src, dst, 4, api.FUSE_ADJACENT)
    b = check_plan(mesh, src, dst, 4, api.FUSE_ADJACENT | api.NO_OVERPARTITION)
    assert [s["kind"] for s in a["steps"]] == [s["kind"] for s in b["steps"]]


def test_random_plans_never_fail_in_any_mode():
    """2000 random problems (odd primes, size-1 axes, rank up to 6) x four flag settings: a plan exists,
    respects the memory bound and has at most one permutation."""
    rng = np.random.default_rng(20211201)
    meshes = [(2,), (6,), (2, 3), (4, 6), (6, 5), (2, 3, 2), (3, 2, 5), (4, 4, 4), (1, 2, 3), (2, 2, 2, 2),
              (2, 3, 5, 7), (12,), (9, 4), (2, 2, 3, 3)]
    for it in range(2000):
        mesh = meshes[it % len(meshes)]
        src, dst = random_problem(rng, mesh, max_rank=6, mult=7)
        for flags in (api.FUSE_ADJACENT, api.FUSE_NONE, api.NAIVE, api.NO_OVERPARTITION):
            p = api.Plan(mesh, src, dst, int(rng.choice([1, 2, 4, 8, 16])), flags)
            assert p.height <= max(p.local_elems(0), p.local_elems(1))
            assert p.step_kinds().count("allpermute") <= 1
            p.close()


KERNEL_CHOICE = [   # mesh, global shape, source axes, target axes, element bytes, expected launch variants
    ((4, 2), (8, 2048, 4096), ((0,), (), (1,)), ((), (0, 1), ()), 2, [4]),             # 4 KiB aligned runs: bulk copies
    ((2,), (64, 24), ((), ()), ((), (0,)), 4, [7]),                                    # 48-byte runs unzipped into 2 tiles
    ((2,), (64, 24), ((), (0,)), ((), ()), 4, [7]),                                    # and zipped back
    ((4, 2), (5, 8, 36), ((), (1,), (0,)), ((), (), ()), 4, [8]),                      # two dimensions interleave: super-boxes
    ((4, 4, 4), (8, 12, 2, 28, 20, 12), ((), (1,), (), (2,), (), ()), ((2,), (), (), (), (0,), (1,)), 4, [8]),   # three
    ((2, 2), (16, 6, 4), ((), (0,), ()), ((), (), (0, 1)), 8, [3]),                    # 8-byte runs scattered: unit walk
    ((2,), (6, 70), ((0,), ()), ((), ()), 4, [6]),                                     # ragged 840-byte runs: bulk-loaded chunk walk
    ((4,), (16, 16), ((0,), ()), ((), (0,)), 4, [0]),                                  # aligned 16-byte runs, too few rows to zip: rows
]


@pytest.mark.parametrize("mesh,gshape,a1,a2,e,variants", KERNEL_CHOICE)
def test_kernel_variant_chosen_for_a_shape(mesh, gshape, a1, a2, e, variants):
    """The host picks the kernel by run length, alignment and how the pieces interleave (no GPU needed)."""
    p = api.Plan(mesh, (gshape, a1), (gshape, a2), e)
    assert [p.launch_info(q).variant for q in range(p.num_launches)] == variants
    p.close()
    check_plan(mesh, (gshape, a1), (gshape, a2), e, api.FUSE_ADJACENT)
