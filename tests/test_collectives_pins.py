"""Pins for the test-side typing rules, cost model and step simulator (oracle/collectives.py):
every sequence the paper prints type-checks, prices as printed, and -- simulated operationally on
real data -- leaves every device with exactly the slice its type prescribes."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import collectives as C
from _notation import load_sequences

FILES = ["fig_permutations.txt", "fig_rename_allgather.txt", "fig_collective_sequences.txt",
         "example_factor_decomposition.txt", "example_extra_permutation.txt", "fig_oversharding.txt"]


def _all_sequences():
    for f in FILES:
        for k, s in enumerate(load_sequences(f)):
            yield pytest.param(s, id=f"{f}:{k}")


def apply_rule(mesh, gshape, axes, step, names):
    kind = step[0]
    if kind == "allgather":
        return C.t_allgather(mesh, gshape, axes, int(step[1]))
    if kind == "dynslice":
        return C.t_dynslice(mesh, gshape, axes, int(step[1]), [names.index(step[2])])
    if kind == "alltoall":
        return C.t_alltoall(mesh, gshape, axes, int(step[1]), int(step[2]))
    raise ValueError(kind)


@pytest.mark.parametrize("seq", list(_all_sequences()))
def test_printed_sequences_type_check_and_price(seq):
    mesh, names = seq["mesh"], seq["names"]
    total = 0
    for k, step in enumerate(seq["steps"]):
        gshape, before, tiles_before = seq["types"][k]
        gshape2, after, tiles_after = seq["types"][k + 1]
        assert gshape == gshape2
        assert C.localtype(mesh, gshape, before) == tiles_before     # printed tile sizes are consistent
        assert C.localtype(mesh, gshape, after) == tiles_after
        if step[0] == "allpermute":
            assert C.t_permute_ok(mesh, gshape, before, after)
        else:
            assert apply_rule(mesh, gshape, before, step, names) == after
        cost = C.step_cost(step[0], mesh, gshape, before, after)
        if k in seq["costs"]:
            assert cost == seq["costs"][k]
        total += cost
    if seq["total"] is not None:
        assert total == seq["total"]


def canonical_coords(mesh):
    return [tuple(c) for c in itertools.product(*[range(k) for k in mesh])]


@pytest.mark.parametrize("seq", list(_all_sequences()))
def test_printed_sequences_simulate_to_the_prescribed_slices(seq):
    mesh, names = seq["mesh"], seq["names"]
    gshape, axes0, _ = seq["types"][0]
    rng = np.random.default_rng(42)
    G = rng.integers(0, 256, size=gshape + (2,), dtype=np.uint8)
    coords = canonical_coords(mesh)
    tiles = oracle.reslice(mesh, (gshape, axes0), G)             # device id = row-major over mesh
    st = C.State(mesh, gshape, C.norm_axes(axes0), coords, tiles)
    st.check_against(G)
    for k, step in enumerate(seq["steps"]):
        _, after, _ = seq["types"][k + 1]
        kind = step[0]
        if kind == "allgather":
            i = int(step[1])
            st = C.sim_allgather(st, i, st.axes[i][:1])
        elif kind == "dynslice":
            st = C.sim_dynslice(st, int(step[1]), [names.index(step[2])])
        elif kind == "alltoall":
            i = int(step[1])
            st = C.sim_alltoall(st, i, int(step[2]), st.axes[i][:1])
        else:
            want = [C.type_offsets(mesh, gshape, after, c) for c in coords]
            have = [st.offsets(d) for d in range(len(coords))]
            pool = {}
            for d, o in enumerate(have):
                pool.setdefault(o, []).append(d)
            src = [pool[o].pop(0) for o in want]                # exists: equal local and global types
            st = C.sim_permute(st, src, coords, after)
        assert st.axes == C.norm_axes(after)
        st.check_against(G)
    final = oracle.reslice(mesh, (gshape, seq["types"][-1][1]), G)
    for d in range(len(final)):
        assert np.array_equal(st.tiles[d], final[d])


def test_merged_alltoall_costs_one_third():
    """Section 7.1: three single-axis alltoalls cost 3*8, the merged multi-axes alltoall costs 8."""
    mesh, gshape = (2, 2, 2), (8, 8)
    t = ((0, 1, 2), ())
    merged = C.t_alltoall(mesh, gshape, t, 0, 1, n_axes=3)
    assert merged == ((), (0, 1, 2))
    assert C.step_cost("alltoall", mesh, gshape, t, merged) == 8
    cost, cur = 0, t
    for _ in range(3):
        nxt = C.t_alltoall(mesh, gshape, cur, 0, 1)
        cost += C.step_cost("alltoall", mesh, gshape, cur, nxt)
        cur = nxt
    assert cost == 24 and C.localtype(mesh, gshape, cur) == (8, 1)


def test_naive_sequence_height_is_the_global_size():
    """Equation (naive redistribution): gathering every dimension reaches localsize = globalsize,
    at least max(localsize tau1, localsize tau2)."""
    mesh, gshape = (4, 4), (128, 512, 128)
    t1, t2 = ((0,), (), (1,)), ((), (1, 0), ())
    seq = [t1, C.t_allgather(mesh, gshape, t1, 0)]
    seq.append(C.t_allgather(mesh, gshape, seq[-1], 2))
    seq.append(C.t_dynslice(mesh, gshape, seq[-1], 1, [1, 0]))
    assert seq[-1] == t2
    assert C.height(mesh, gshape, seq) == 128 * 512 * 128
    assert C.height(mesh, gshape, seq) >= max(C.localsize(mesh, gshape, t1), C.localsize(mesh, gshape, t2))


def test_normal_form_regex():
    assert C.is_normal_form(["dynslice", "dynslice", "alltoall", "allpermute", "allgather"])
    assert C.is_normal_form([])
    assert not C.is_normal_form(["allgather", "dynslice"])
    assert not C.is_normal_form(["alltoall", "dynslice"])
    assert not C.is_normal_form(["allgather", "alltoall"])


def test_rules_reject_what_the_paper_forbids():
    mesh, gshape = (4, 4), (16, 16)
    with pytest.raises(C.TypeError_):
        C.t_dynslice(mesh, gshape, ((0,), ()), 1, [0])          # axis already partitions a dimension
    with pytest.raises(C.TypeError_):
        C.t_alltoall(mesh, (16, 6), ((0,), ()), 0, 1)           # 4 does not divide 6
    with pytest.raises(C.TypeError_):
        C.t_allgather(mesh, gshape, ((), ()), 0)                # nothing to gather


def test_low_level_relabel_moves_no_data():
    """Low-level allgather on a non-minor axis: relabel so that the axis is minor-most, keeping every
    device's base offset, then the plain rule applies (figure on low-level semantics)."""
    mesh, gshape = (2, 3), (12,)
    G = np.arange(12, dtype=np.uint8).reshape(12, 1)
    coords = canonical_coords(mesh)
    st = C.State(mesh, gshape, ((0, 1),), coords, oracle.reslice(mesh, (gshape, ((0, 1),)), G))
    # act on axis 1 (major): beta' lists it first; new coordinates re-digitise the tile index
    new_coords = []
    for c in coords:
        t = c[0] + 2 * c[1]
        new_coords.append((t // 3, t % 3))
    st2 = C.relabel(st, new_coords, ((1, 0),))
    st3 = C.sim_allgather(st2, 0, (1,))
    st3.check_against(G)
    with pytest.raises(AssertionError):
        C.relabel(st, coords, ((1, 0),))                        # same coordinates would move data
