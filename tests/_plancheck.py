"""Check a synthesized plan step by step against the paper's rules and the oracle (CPU only)."""
from __future__ import annotations

import numpy as np

import oracle
from oracle import collectives as C
from paper_2112_01075_b200 import api
from _descsim import run_plan


def types_of(w):
    return (w.src.global_shape, w.src.axes), (w.dst.global_shape, w.dst.axes)


def check_plan(mesh, src, dst, elem_bytes, flags=api.FUSE_ADJACENT, seed=0, simulate_launches=True):
    """Returns the plan description.  Raises AssertionError on any violated property."""
    gshape = tuple(src[0])
    plan = api.Plan(mesh, src, dst, elem_bytes, flags)
    desc = plan.describe()
    rng = np.random.default_rng(seed)
    G = rng.integers(0, 256, size=gshape + (elem_bytes,), dtype=np.uint8)
    src_tiles = oracle.reslice(mesh, src, G)
    want = oracle.redistribute(mesh, src, dst, src_tiles)

    pm = tuple(p["size"] for p in desc["primes"])             # the prime mesh
    n = desc["n_devices"]
    # prime decomposition is equivalent: same base offsets for every device (Principle 1)
    t1, off1 = oracle.base_offsets(mesh, src)
    for d in range(n):
        assert C.type_offsets(pm, gshape, desc["src_axes"], desc["initial_coords"][d]) == tuple(off1[d])
    for p in desc["primes"]:
        assert all(p["size"] % q for q in range(2, p["size"]))  # prime

    st = C.State(pm, gshape, C.norm_axes(desc["src_axes"]), [tuple(c) for c in desc["initial_coords"]], src_tiles)
    st.check_against(G)
    types, kinds, cost = [st.axes], [], 0
    M = max(plan.local_elems(0), plan.local_elems(1))
    for s in desc["steps"]:
        kind, i, j, acting = s["kind"], s["i"], s["j"], s["acting"]
        before_axes = st.axes
        if kind == "allpermute":
            st = C.sim_permute(st, s["source_of"], s["post_coords"], s["post_axes"])
        else:
            # low-level rule: an equivalent assignment with the acting axes minor-most, no data moved
            st = C.relabel(st, s["pre_coords"], s["pre_axes"])
            if kind != "dynslice":
                assert tuple(st.axes[i][:len(acting)]) == tuple(acting)
                assert C.to_front(before_axes, i, acting)[i] == st.axes[i]
            assert _prod(pm[a] for a in acting) == s["factor"]
            if kind == "dynslice":
                st = C.sim_dynslice(st, i, acting)
            elif kind == "alltoall":
                st = C.sim_alltoall(st, i, j, acting)
            elif kind == "allgather":
                st = C.sim_allgather(st, i, acting)
            else:
                raise AssertionError(kind)
            assert [tuple(c) for c in s["post_coords"]] == st.coords
        assert st.axes == C.norm_axes(s["post_axes"])
        st.check_against(G)                       # every intermediate is the slice its type prescribes
        c = C.step_cost(kind, pm, gshape, before_axes, st.axes)
        assert c == s["cost"]
        assert list(C.localtype(pm, gshape, st.axes)) == s["local_after"]
        cost += c
        kinds.append(kind)
        types.append(st.axes)
    for d in range(n):
        assert np.array_equal(st.tiles[d], want[d]), f"device {d} ends with the wrong tile"
    assert C.is_normal_form(kinds), kinds
    assert kinds.count("allpermute") <= 1
    assert cost == plan.cost == desc["cost"]
    h = C.height(pm, gshape, types)
    assert h == plan.height and h <= M          # memory bound of the normal form
    # launches cover the steps in order, without gaps
    if (flags & 3) != api.NAIVE:
        nxt = 0
        for L in desc["launches"]:
            assert L["first_step"] == nxt
            nxt += L["n_steps"]
        assert nxt == len(desc["steps"])
        slots = {L["to"] for L in desc["launches"]} - {"dst"}
        assert plan.scratch_bytes_per_device == len(slots) * desc["slot_bytes"]
        # every intermediate that is materialised fits the bound
        for L in desc["launches"][:-1]:
            assert L["dst_tile_bytes"] <= M * elem_bytes and L["dst_tile_bytes"] <= desc["slot_bytes"]
    if simulate_launches:
        got, counts = run_plan(desc, src_tiles)
        for d in range(n):
            assert np.array_equal(got[d], want[d].reshape(-1)), f"launch descriptors: device {d} differs"
        last = counts[-1]
        for d in range(n):
            assert np.all(last[d] == 1)          # every destination byte written exactly once
    plan.close()
    return desc


def _prod(xs):
    n = 1
    for x in xs:
        n *= int(x)
    return n
