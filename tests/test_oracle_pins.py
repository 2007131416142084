"""Pins for the CPU oracle: the paper's worked example, its lemmas, brute-force ownership written
independently (interval splitting, not the offset recursion), closed forms and round trips."""
import itertools

import numpy as np
import pytest

import oracle
from _notation import load_offset_table
from paper_2112_01075_b200 import workloads as wl


def dev_id(mesh, coord):
    d = 0
    for k, c in zip(mesh, coord):
        d = d * k + c
    return d


def all_coords(mesh):
    return list(itertools.product(*[range(k) for k in mesh]))


def split_interval(mesh, n, ax, coord):
    """Section 2.1 in words: the dimension is split over the last-listed (major) axis first, then
    every piece is split further along the axis listed before it, and so on."""
    lo, hi = 0, n
    for a in reversed(ax):
        size = (hi - lo) // mesh[a]
        lo = lo + coord[a] * size
        hi = lo + size
    return lo, hi


def brute_shards(mesh, gshape, axes, G):
    out = []
    for coord in all_coords(mesh):
        sl = tuple(slice(*split_interval(mesh, s, ax, coord)) for s, ax in zip(gshape, axes))
        out.append(np.ascontiguousarray(G[sl]))
    return out


def linear_global(gshape):
    return wl.global_array_bytes(gshape, 4, "linear_u32", 0)


# ------------------------------------------------------------------------------ worked example

def test_golden_axis_order_offsets():
    names, mesh, (gshape, axes, tiles), rows = load_offset_table("sec2_1_axis_order_offsets.txt")
    tile, off = oracle.base_offsets(mesh, (gshape, axes))
    assert tile == tiles
    for ix, iy, expect in rows:
        assert off[dev_id(mesh, (ix, iy)), 0] == expect


def test_reversed_axis_order_changes_assignment_not_tiles():
    mesh = (2, 2)
    t1, o1 = oracle.base_offsets(mesh, ((32,), ((0, 1),)))
    t2, o2 = oracle.base_offsets(mesh, ((32,), ((1, 0),)))
    assert t1 == t2 == (8,)
    assert sorted(o1[:, 0]) == sorted(o2[:, 0]) == [0, 8, 16, 24]
    assert not np.array_equal(o1, o2)


# -------------------------------------------------------------------------------------- lemmas

MESHES = [(2,), (3,), (2, 2), (2, 3), (4, 6), (2, 4, 2), (3, 2, 2), (4, 4, 4)]


def random_type(rng, mesh, rank, mult=2):
    per_dim = [[] for _ in range(rank)]
    for a in range(len(mesh)):
        c = int(rng.integers(0, rank + 1))
        if c < rank:
            per_dim[c].append(a)
    axes = []
    for ax in per_dim:
        axes.append(tuple(ax[i] for i in rng.permutation(len(ax))) if ax else ())
    gshape = tuple(int(np.prod([mesh[a] for a in ax], dtype=np.int64)) * int(rng.integers(1, mult + 1)) for ax in axes)
    return gshape, tuple(axes)


@pytest.mark.parametrize("mesh", MESHES)
def test_lemma_image_is_all_multiples_of_tile(mesh):
    """Image of D[[c{xs}n]] = all multiples of c below n; every tile is held by N/#tiles devices."""
    rng = np.random.default_rng(7)
    n_dev = int(np.prod(mesh))
    for _ in range(20):
        gshape, axes = random_type(rng, mesh, int(rng.integers(1, 4)), mult=3)
        tile, off = oracle.base_offsets(mesh, (gshape, axes))
        n_tiles = 1
        for k, (s, c) in enumerate(zip(gshape, tile)):
            assert sorted(set(off[:, k])) == list(range(0, s, c))
            n_tiles *= s // c
        uniq, counts = np.unique(off, axis=0, return_counts=True)
        assert len(uniq) == n_tiles and set(counts) == {n_dev // n_tiles}


def test_ill_formed_types_are_rejected():
    mesh = (4, 8)
    with pytest.raises(oracle.OracleError) as e:
        oracle.base_offsets(mesh, ((128, 256), ((0,), (0,))))         # axis used twice
    assert e.value.code == 2
    with pytest.raises(oracle.OracleError) as e:
        oracle.base_offsets(mesh, ((128, 256), ((2,), ())))           # axis not in the mesh
    assert e.value.code == 2
    with pytest.raises(oracle.OracleError) as e:
        oracle.base_offsets(mesh, ((6, 256), ((0,), ())))             # 4 does not divide 6
    assert e.value.code == 3


def test_invalid_casts_have_different_global_types():
    """Section 2.5: [32{xdevs}128, 32{ydevs}256] -> [32{xdevs,ydevs}1024, 32] is not a redistribution
    although tile shapes and tile counts agree."""
    mesh = (4, 8)
    a = ((128, 256), ((0,), (1,)))
    b = ((1024, 32), ((0, 1), ()))
    ta, _ = oracle.base_offsets(mesh, a)
    tb, _ = oracle.base_offsets(mesh, b)
    assert ta == tb == (32, 32)
    shards = [np.zeros((32, 32, 1), np.uint8)] * 32
    with pytest.raises(oracle.OracleError):
        oracle.redistribute(mesh, a, b, shards)


# ------------------------------------------------------------------- brute force on tiny meshes

@pytest.mark.parametrize("mesh", [(2,), (3,), (2, 2), (2, 3), (3, 3), (2, 2, 2), (2, 3, 2), (3, 2, 3)])
def test_brute_force_ownership_and_result(mesh):
    rng = np.random.default_rng(11)
    for _ in range(12):
        rank = int(rng.integers(1, 4))
        g1, a1 = random_type(rng, mesh, rank, 1)
        g2, a2 = random_type(rng, mesh, rank, 1)
        gshape = tuple(int(np.lcm(x, y)) * int(rng.integers(1, 3)) for x, y in zip(g1, g2))
        e = int(rng.choice([1, 2, 4]))
        G = rng.integers(0, 256, size=gshape + (e,), dtype=np.uint8)
        src = brute_shards(mesh, gshape, a1, G)
        want = brute_shards(mesh, gshape, a2, G)
        got = oracle.redistribute(mesh, (gshape, a1), (gshape, a2), src)
        for d in range(len(want)):
            assert got[d].shape == want[d].shape
            assert np.array_equal(got[d], want[d]), (mesh, gshape, a1, a2, d)
            # the one-tile form (used where all tiles do not fit in host memory at once)
            assert np.array_equal(oracle.tile_of(mesh, (gshape, a2), G, d), want[d])
        # ownership: every global element lies in the tile of exactly N/#tiles devices
        tile, off = oracle.base_offsets(mesh, (gshape, a1))
        count = np.zeros(gshape, dtype=np.int64)
        for d in range(len(src)):
            sl = tuple(slice(o, o + c) for o, c in zip(off[d], tile))
            count[sl] += 1
        n_tiles = int(np.prod([s // c for s, c in zip(gshape, tile)]))
        assert np.all(count == len(src) // n_tiles)


# --------------------------------------------------------------------------------- closed forms

@pytest.mark.parametrize("mesh", [(2, 2), (4, 2), (2, 4, 2)])
def test_linear_fill_closed_form(mesh):
    """With G[g] = row-major linear index of g: dst[d][l] = ravel(T[[tau2]](d) + l)."""
    rng = np.random.default_rng(5)
    for _ in range(6):
        rank = int(rng.integers(1, 4))
        g1, a1 = random_type(rng, mesh, rank, 1)
        g2, a2 = random_type(rng, mesh, rank, 1)
        gshape = tuple(int(np.lcm(x, y)) * 2 for x, y in zip(g1, g2))
        G = linear_global(gshape)
        src = oracle.reslice(mesh, (gshape, a1), G)
        got = oracle.redistribute(mesh, (gshape, a1), (gshape, a2), src)
        tile, off = oracle.base_offsets(mesh, (gshape, a2))
        for d, coord in enumerate(all_coords(mesh)):
            lo = [split_interval(mesh, s, ax, coord)[0] for s, ax in zip(gshape, a2)]
            assert list(off[d]) == lo
            idx = np.indices(tile).reshape(rank, -1) + np.array(lo)[:, None]
            lin = np.ravel_multi_index(tuple(idx), gshape).astype("<u4").reshape(tile)
            assert np.array_equal(got[d].view("<u4")[..., 0], lin)


def test_config1_closed_form():
    """256x256 uint32 on (x:2,y:2): swapping the two axes across dimensions exchanges the tiles of
    devices 1 and 2 and leaves 0 and 3 in place."""
    w = wl.config1()
    G = wl.global_array_bytes(w.src.global_shape, 4, w.fill, w.seed)
    src = oracle.reslice(w.mesh_shape, (w.src.global_shape, w.src.axes), G)
    dst = oracle.redistribute(w.mesh_shape, (w.src.global_shape, w.src.axes), (w.dst.global_shape, w.dst.axes), src)
    for d, s in enumerate([0, 2, 1, 3]):
        assert np.array_equal(dst[d], src[s])
    p, q = np.meshgrid(np.arange(128), np.arange(128), indexing="ij")
    assert np.array_equal(dst[1].view("<u4")[..., 0], ((128 + p) * 256 + q).astype("<u4"))


def test_config5a_is_a_device_transpose():
    """{d0:(x,y), d1:z} -> {d0:(y,x), d1:z} on (4,4,4): device (a,b,c) receives the tile of (b,a,c)."""
    w = wl.config5("a").scaled((64, 32))
    rng = np.random.default_rng(3)
    G = rng.integers(0, 256, size=(64, 32, 2), dtype=np.uint8)
    src = oracle.reslice(w.mesh_shape, (w.src.global_shape, w.src.axes), G)
    dst = oracle.redistribute(w.mesh_shape, (w.src.global_shape, w.src.axes), (w.dst.global_shape, w.dst.axes), src)
    for a in range(4):
        for b in range(4):
            for c in range(4):
                assert np.array_equal(dst[16 * a + 4 * b + c], src[16 * b + 4 * a + c])


@pytest.mark.parametrize("n", [2, 4, 8])
def test_one_dimensional_mesh_row_to_column(n):
    """Row-sharded -> column-sharded equals cat(shards, 0)[:, b*w:(b+1)*w] (numpy formulation)."""
    rng = np.random.default_rng(n)
    rows, cols, e = 4 * n, 6 * n, 2
    G = rng.integers(0, 256, size=(rows, cols, e), dtype=np.uint8)
    src = [np.ascontiguousarray(G[d * rows // n:(d + 1) * rows // n]) for d in range(n)]
    got = oracle.redistribute((n,), ((rows, cols), ((0,), ())), ((rows, cols), ((), (0,))), src)
    cat = np.concatenate(src, axis=0)
    w = cols // n
    for b in range(n):
        assert np.array_equal(got[b], cat[:, b * w:(b + 1) * w])
    # and column-sharded -> replicated is the concatenation along dim 1 on every device
    full = oracle.redistribute((n,), ((rows, cols), ((), (0,))), ((rows, cols), ((), ())), got)
    for b in range(n):
        assert np.array_equal(full[b], G)


def test_stack_transpose_formulation_two_axes():
    """For [c{x,y}n] on (x:X, y:Y): stacking tiles as [X, Y, c] and moving y outermost gives G."""
    X, Y, c = 3, 2, 5
    rng = np.random.default_rng(0)
    G = rng.integers(0, 256, size=(X * Y * c, 1), dtype=np.uint8)
    shards = oracle.reslice((X, Y), ((X * Y * c,), ((0, 1),)), G)
    st = np.stack(shards).reshape(X, Y, c)
    assert np.array_equal(st.transpose(1, 0, 2).reshape(-1), G[:, 0])


# ----------------------------------------------------------------------------------- properties

@pytest.mark.parametrize("mesh", [(2, 2), (4, 6), (2, 4, 2)])
def test_round_trip_and_replica_check(mesh):
    rng = np.random.default_rng(13)
    for _ in range(8):
        rank = int(rng.integers(1, 4))
        g1, a1 = random_type(rng, mesh, rank, 1)
        g2, a2 = random_type(rng, mesh, rank, 1)
        gshape = tuple(int(np.lcm(x, y)) for x, y in zip(g1, g2))
        G = rng.integers(0, 256, size=gshape + (2,), dtype=np.uint8)
        A = oracle.reslice(mesh, (gshape, a1), G)
        assert np.array_equal(oracle.materialize(mesh, (gshape, a1), A), G)
        B = oracle.redistribute(mesh, (gshape, a1), (gshape, a2), A)
        A2 = oracle.redistribute(mesh, (gshape, a2), (gshape, a1), B)
        for x, y in zip(A, A2):
            assert np.array_equal(x, y)
        for x, y in zip(B, oracle.reslice(mesh, (gshape, a2), G)):
            assert np.array_equal(x, y)


def test_replica_mismatch_is_detected():
    mesh = (2, 2)
    t = ((8, 4), ((0,), ()))       # axis 1 unused: devices (i,0) and (i,1) are replicas
    G = np.arange(32, dtype=np.uint8).reshape(8, 4, 1)
    shards = [s.copy() for s in oracle.reslice(mesh, t, G)]
    assert np.array_equal(shards[0], shards[1]) and np.array_equal(shards[2], shards[3])
    shards[3][0, 0, 0] ^= 1
    with pytest.raises(oracle.OracleError) as e:
        oracle.materialize(mesh, t, shards, check=True)
    assert e.value.code == 4
    assert np.array_equal(oracle.materialize(mesh, t, shards, check=False), G)   # lowest id wins


def test_threads_do_not_change_the_result():
    mesh = (2, 4, 2)
    rng = np.random.default_rng(1)
    gshape = (16, 8, 8, 16)
    a1, a2 = ((0,), (2, 1), (), ()), ((), (), (1,), (0, 2))
    G = rng.integers(0, 256, size=gshape + (4,), dtype=np.uint8)
    A = oracle.reslice(mesh, (gshape, a1), G)
    oracle.set_threads(1)
    one = oracle.redistribute(mesh, (gshape, a1), (gshape, a2), A)
    oracle.set_threads(max(2, oracle.max_threads()))
    many = oracle.redistribute(mesh, (gshape, a1), (gshape, a2), A)
    oracle.set_threads(1)
    for x, y in zip(one, many):
        assert np.array_equal(x, y)
