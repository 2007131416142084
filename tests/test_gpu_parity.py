"""GPU parity: the CUDA path, called through the C boundary, against the CPU oracle, bit for bit.

Inputs are seeded and synthetic (paper_2112_01075_b200.workloads); source tiles and expected tiles
come from the oracle only.  Comparison is bytewise (the random bf16/f32 patterns include NaNs).
"""
import numpy as np
import pytest

import oracle
from paper_2112_01075_b200 import api, workloads as wl
from _buffers import Carved
from _plancheck import types_of

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MODES = [api.FUSE_ADJACENT, api.FUSE_NONE, api.FUSE_ALL, api.NAIVE]
MODE_NAMES = {0: "adjacent", 1: "unfused", 2: "all", 3: "naive"}


def run_gpu(mesh, src, dst, e, src_tiles, flags=api.FUSE_ADJACENT, stream=None, bound=False):
    """Plan and execute on tiles carved out of one canary-filled buffer (tiles aligned to 16 bytes and no
    better, sources packed, guard bands around every destination tile and the scratch); afterwards every
    guard byte must be intact and the sources unchanged.  `bound`: through redist_bind /
    redist_bound_execute instead of redist_execute."""
    plan = api.Plan(mesh, src, dst, e, flags)
    mem = Carved(torch, src_tiles, plan.n_devices, plan.local_elems(1) * e, plan.scratch_bytes)
    if bound:
        s = stream if stream is not None else torch.cuda.current_stream()
        call = plan.bind([t.data_ptr() for t in mem.src], [t.data_ptr() for t in mem.dst],
                         mem.scratch.data_ptr() if mem.scratch is not None else 0, plan.scratch_bytes)
        call(s.cuda_stream)
    else:
        plan.execute(mem.src, mem.dst, mem.scratch, stream)
    torch.cuda.synchronize()
    mem.check(f"{mesh} {src} -> {dst} e={e} flags={flags}")
    return plan, mem.results()


def assert_same(got, want, what=""):
    assert len(got) == len(want)
    for d, (g, w) in enumerate(zip(got, want)):
        w = np.ascontiguousarray(w).reshape(-1)
        g = np.ascontiguousarray(g).reshape(-1)
        if not np.array_equal(g, w):
            bad = np.flatnonzero(g != w)
            raise AssertionError(f"{what}: device {d}: {bad.size} of {w.size} bytes differ, first at {bad[0]}")


def make_case(w, seed=None):
    src, dst = types_of(w)
    G = wl.global_array_bytes(w.src.global_shape, w.elem_bytes, w.fill, w.seed if seed is None else seed)
    src_tiles = oracle.reslice(w.mesh_shape, src, G)
    want = oracle.redistribute(w.mesh_shape, src, dst, src_tiles)
    return src, dst, src_tiles, want


# ---------------------------------------------------------------- sizes the oracle does in seconds

MEDIUM = [
    wl.config1(), wl.config1().reversed(),
    wl.config2().scaled((8, 512, 1024)), wl.config2().reversed().scaled((8, 512, 1024)),
    wl.config3("a").scaled((2048, 4096)), wl.config3("b").scaled((2048, 4096)), wl.config3("c").scaled((2048, 4096)),
    wl.config5("a").scaled((4096, 2048)), wl.config5("b").scaled((4096, 4096)),
    # ragged: tile rows that do not fill a work item, odd primes, run lengths that are not 16-byte multiples
    wl.config3("a").scaled((8 * 37, 8 * 101)), wl.config3("c").scaled((24, 8 * 3)),
    wl.config2().scaled((8, 8 * 13, 2 * 77)),
]


@pytest.mark.parametrize("w", MEDIUM, ids=lambda w: w.name + "_" + "x".join(map(str, w.src.global_shape)))
@pytest.mark.parametrize("mode", MODES, ids=lambda m: MODE_NAMES[m])
def test_configurations_at_medium_size(w, mode):
    src, dst, src_tiles, want = make_case(w)
    plan, got = run_gpu(w.mesh_shape, src, dst, w.elem_bytes, src_tiles, mode)
    assert_same(got, want, w.name)
    assert plan.height <= max(plan.local_elems(0), plan.local_elems(1))


@pytest.mark.parametrize("mode", MODES, ids=lambda m: MODE_NAMES[m])
def test_random_sweep_reduced_shape(mode):
    """The 100 seeded (source, target) pairs of the random sweep on [16,32,64,128] f32 (16 MiB)."""
    pairs = wl.config4(100, (16, 32, 64, 128))
    G = wl.global_array_bytes((16, 32, 64, 128), 4, "random_bits", wl.CONFIG4_FILL_SEED)
    for w in pairs:
        src, dst = types_of(w)
        src_tiles = oracle.reslice(w.mesh_shape, src, G)
        want = oracle.reslice(w.mesh_shape, dst, G)
        _, got = run_gpu(w.mesh_shape, src, dst, 4, src_tiles, mode)
        assert_same(got, want, w.name + " " + w.src.notation(w.mesh_shape) + "->" + w.dst.notation(w.mesh_shape))


def random_problems_small_and_odd(n_problems, extra_flags=0):
    """Odd primes, all element sizes, element-sized runs, several steps with scratch ping-pong.
    Returns the set of kernel variants that ran."""
    rng = np.random.default_rng(2112)
    meshes = [(2, 3), (4, 6), (3, 3, 2), (2, 2, 2, 2), (6,), (5, 2), (4, 4, 4), (1, 2, 3), (9, 4), (16,)]
    n_multi = 0
    variants = set()
    for t in range(n_problems):
        mesh = meshes[t % len(meshes)]
        rank = int(rng.integers(1, 5))

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
            gshape.append(int(np.lcm(f1, f2)) * int(rng.integers(1, 9)))
        gshape = tuple(gshape)
        e = int(rng.choice([1, 2, 4, 4, 8, 16]))
        if int(np.prod(gshape)) * e > (4 << 20):
            continue
        G = rng.integers(0, 256, size=gshape + (e,), dtype=np.uint8)
        src, dst = (gshape, a1), (gshape, a2)
        src_tiles = oracle.reslice(mesh, src, G)
        want = oracle.redistribute(mesh, src, dst, src_tiles)
        mode = MODES[t % 4] | extra_flags
        plan, got = run_gpu(mesh, src, dst, e, src_tiles, mode, bound=(t // 4) % 2 == 1)
        n_multi += plan.num_launches >= 3
        variants.update(plan.launch_info(q).variant for q in range(plan.num_launches))
        assert_same(got, want, f"{mesh} {src} -> {dst} e={e} mode={mode}")
    assert n_multi > 0          # the two-slot scratch ping-pong was exercised
    return variants


def test_random_problems_small_and_odd():
    variants = random_problems_small_and_odd(600)
    assert variants >= {0, 3, 4, 5, 6, 7, 8}   # rows, units, bulk, gather, ragged bulk, zip and super-box kernels all ran


def test_random_problems_with_the_permutation_counted():
    """Plans chosen with the final permutation in the cost (other sequences than the default ones,
    e.g. an extra leading dynslice) in every execution mode."""
    random_problems_small_and_odd(300, api.COST_PERMUTE)


@pytest.mark.parametrize("hint", [0, 1, 2, 3])
def test_bulk_copies_with_l2_policies(hint):
    """The plain bulk-copy kernels with an L2 evict-first policy on their loads, their stores, both or neither."""
    with api.tuning(l2_hint=hint):
        for w in MEDIUM[:9]:
            src, dst, src_tiles, want = make_case(w)
            plan, got = run_gpu(w.mesh_shape, src, dst, w.elem_bytes, src_tiles)
            assert_same(got, want, f"{w.name} l2_hint={hint}")


def test_register_kernels_behind_the_tuning_values():
    """With the bulk-copy kernels (zip included) and the gather walk switched off the same problems run
    on the plain register kernels."""
    with api.tuning(bulk=0, gather=0):
        v = random_problems_small_and_odd(300)
    assert v == {0, 1, 2, 3}, v


@pytest.mark.parametrize("values", [
    {"zip_walks": 0},                               # flat walk only
    {"zip_walks": 2, "zip_by_range_slots": 1},      # by-range walk, else flat
    {"zip_walks": 4},                               # tabulated places, else flat
], ids=["flat", "by_range", "tabulated"])
def test_zip_kernels_with_each_chunk_map(values):
    """The zip kernels pick one of several ways to map a target chunk to its units; the tuning values
    force the ones that the default choice (periodic walk) seldom leaves work for."""
    with api.tuning(**values):
        v = random_problems_small_and_odd(400)
    assert 7 in v, v


def test_super_box_kernels_wherever_they_apply():
    """box = 2 sends every launch whose inner dimensions allow it through the super-box kernels (by default
    only where the zip, gather and unit walks do badly)."""
    with api.tuning(box=2):
        v = random_problems_small_and_odd(600)
    assert 8 in v, v
    with api.tuning(box=0):
        v = random_problems_small_and_odd(300)
    assert 8 not in v, v


BOXES = [   # mesh, global shape, source axes, target axes, element bytes: several dimensions interleave at run granularity
    ((4, 4, 4), (8, 12, 2, 28, 20, 12), ((), (1,), (), (2,), (), ()), ((2,), (), (), (), (0,), (1,)), 4),   # 12-byte runs, 3 inner dimensions
    ((4, 4, 2), (2, 8, 8, 30, 4, 8), ((), (), (), (), (1,), (0,)), ((), (1,), (0,), (2,), (), ()), 4),      # 8-byte runs from 16 tiles
    ((2, 2, 2), (6, 6, 6, 48, 10, 26), ((), (2,), (), (0,), (), ()), ((), (), (1,), (), (2,), (0,)), 4),   # 52-byte runs, short zipped digit
    ((2, 3), (6, 9, 10, 6), ((), (1,), (0,), ()), ((), (), (), (1,)), 2),                                  # odd primes, 2-byte elements
    ((2, 2, 2), (4, 8, 12, 6), ((0,), (1,), (2,), ()), ((), (2,), (0,), (1,)), 8),                          # every dimension changes, fan-out 1
    ((2, 2, 2), (4, 8, 12, 6), ((0,), (1,), (2,), ()), ((), (), (0,), ()), 4),                              # replicated target: fan-out 4
]


@pytest.mark.parametrize("mesh,gshape,a1,a2,e", BOXES)
def test_super_box_kernels(mesh, gshape, a1, a2, e):
    """Short runs that interleave along several dimensions: the item is widened to a super-box, staged in
    shared memory segment by segment and written out range by range (launch variant 8).  Both directions,
    fused and collective by collective, with the kernels on by default and forced."""
    rng = np.random.default_rng(sum(gshape) + e)
    G = rng.integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    seen = set()
    for src, dst in (((gshape, a1), (gshape, a2)), ((gshape, a2), (gshape, a1))):
        src_tiles = oracle.reslice(mesh, src, G)
        want = oracle.reslice(mesh, dst, G)
        for box in (1, 2):
            with api.tuning(box=box):
                for mode in (api.FUSE_ADJACENT, api.FUSE_NONE):
                    plan, got = run_gpu(mesh, src, dst, e, src_tiles, mode)
                    seen.update(plan.launch_info(q).variant for q in range(plan.num_launches))
                    assert_same(got, want, f"super-box {mesh} {src} -> {dst} box={box} mode={mode}")
    assert 8 in seen


BANKED = [  # a target tile takes one element in 4 or 8 of the last dimension: its units sit 32 bytes apart
    ((4, 2, 2), (2, 17, 16, 28, 9, 8), ((1,), (), (2, 0), (), (), ()), ((), (), (), (1,), (), (0, 2)), 4),
    ((2, 2, 2), (4, 6, 16, 12, 5, 4), ((0,), (), (1, 2), (), (), ()), ((), (), (), (0,), (), (1, 2)), 8),
]


@pytest.mark.parametrize("width", [0, 1, 2, 4, 8, 16, 64])
def test_super_box_kernels_at_every_lane_group_width(width):
    """The lanes that share one target range in the super-box kernels: chosen per launch by default (narrower than
    a warp where one range's units would fall into a few shared-memory banks -- the two BANKED shapes), and every
    width forced over all the super-box shapes."""
    seen, widths = set(), set()
    for mesh, gshape, a1, a2, e in BOXES + BANKED:
        G = np.random.default_rng(sum(gshape) + e + width).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
        for src, dst in (((gshape, a1), (gshape, a2)), ((gshape, a2), (gshape, a1))):
            src_tiles, want = oracle.reslice(mesh, src, G), oracle.reslice(mesh, dst, G)
            with api.tuning(box=2, box_width=width):
                plan, got = run_gpu(mesh, src, dst, e, src_tiles)
            for L in plan.describe()["launches"]:
                if L["geometry"]["mode"] == 5:
                    widths.add(L["geometry"]["zip_width"])
            seen.update(plan.launch_info(q).variant for q in range(plan.num_launches))
            assert_same(got, want, f"super-box {mesh} {src} -> {dst} width={width}")
    assert 8 in seen
    assert widths == {width} if width else min(widths) < 32 <= max(widths), widths


def test_gather_walk_wherever_it_applies():
    """gather = 2 sends every eligible launch through the gather walk, including long source rows that
    are scattered into several target tiles and 16-byte units (not chosen by default)."""
    with api.tuning(gather=2, zip=0, box=0):
        v = random_problems_small_and_odd(600)
    assert 5 in v and 7 not in v, v


def test_round_trip_on_the_gpu():
    w = wl.config2().scaled((8, 256, 512))
    src, dst, src_tiles, want = make_case(w)
    _, mid = run_gpu(w.mesh_shape, src, dst, w.elem_bytes, src_tiles)
    tile_dst, _ = oracle.base_offsets(w.mesh_shape, dst)
    mid_tiles = [m.reshape(tile_dst + (w.elem_bytes,)) for m in mid]
    _, back = run_gpu(w.mesh_shape, dst, src, w.elem_bytes, mid_tiles)
    assert_same(back, src_tiles, "round trip")


def test_identity_and_non_default_stream():
    mesh = (2, 2)
    t = ((64, 48), ((0,), (1,)))
    G = wl.global_array_bytes((64, 48), 2, "random_bits", 5)
    tiles = oracle.reslice(mesh, t, G)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        plan, got = run_gpu(mesh, t, t, 2, tiles, stream=s)
    assert plan.launch_kernels() == ["copy"]
    assert_same(got, tiles, "identity")


def test_replicated_sources_may_alias():
    """Replicas hold identical bytes, so the caller may pass one buffer for all of them."""
    w = wl.config3("b").scaled((512, 256))
    src, dst, src_tiles, want = make_case(w)
    plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes)
    one = torch.from_numpy(src_tiles[0]).cuda()
    dev_dst = [torch.empty(plan.local_elems(1) * w.elem_bytes, dtype=torch.uint8, device="cuda") for _ in range(8)]
    plan.execute([one] * 8, dev_dst)
    torch.cuda.synchronize()
    assert_same([t.cpu().numpy() for t in dev_dst], want, "aliased replicas")


def test_host_buffers_entry_point():
    w = wl.config3("a").scaled((1024, 2048))
    src, dst, src_tiles, want = make_case(w)
    plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes, api.FUSE_NONE)
    n = plan.n_devices
    hs = [torch.from_numpy(np.ascontiguousarray(t)).reshape(-1).pin_memory() for t in src_tiles]
    hd = [torch.zeros(plan.local_elems(1) * w.elem_bytes, dtype=torch.uint8).pin_memory() for _ in range(n)]
    dev_src = torch.empty(plan.staging_bytes(0), dtype=torch.uint8, device="cuda")
    dev_dst = torch.empty(plan.staging_bytes(1), dtype=torch.uint8, device="cuda")
    plan.execute_host(hs, hd, dev_src, dev_dst, plan.alloc_scratch())
    torch.cuda.synchronize()
    assert_same([t.numpy() for t in hd], want, "host entry point")


def test_misuse_is_reported_not_executed():
    w = wl.config3("a").scaled((64, 64))
    src, dst, src_tiles, _ = make_case(w)
    plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes)
    nb = plan.local_elems(1) * w.elem_bytes
    buf = torch.zeros(8 * nb + 64, dtype=torch.uint8, device="cuda")
    dev_src = [torch.from_numpy(t).cuda() for t in src_tiles]
    good = [buf[d * nb:(d + 1) * nb] for d in range(8)]
    with pytest.raises(api.RedistError) as e:
        plan.execute(dev_src, [buf[1 + d * nb:1 + (d + 1) * nb] for d in range(8)])
    assert e.value.status == 7
    with pytest.raises(api.RedistError) as e:
        plan.execute(dev_src, [good[0]] * 8)
    assert e.value.status == 6
    with pytest.raises(api.RedistError) as e:
        plan.execute(good, good)
    assert e.value.status == 6
    plan.execute(dev_src, good)
    torch.cuda.synchronize()


# ------------------------------------------------------------------------------------- full sizes

FULL = ["c2", "c2_back", "c3a", "c3b", "c3c", "c5a", "c5b"]


@pytest.mark.parametrize("name", FULL)
def test_configurations_at_full_size(name):
    """Full benchmark sizes, default mode -- the launch configuration the benchmark times."""
    w = wl.bench_workloads()[name]
    oracle.set_threads(oracle.max_threads())
    try:
        src, dst, src_tiles, want = make_case(w)
    finally:
        oracle.set_threads(1)
    plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes)
    if name == "c3b":
        # eight identical 512 MiB replicas: upload one, alias it (the oracle checked they agree)
        one = torch.from_numpy(src_tiles[0]).cuda()
        dev_src = [one] * plan.n_devices
    else:
        dev_src = [torch.from_numpy(t).cuda() for t in src_tiles]
    nb = plan.local_elems(1) * w.elem_bytes
    dev_dst = [torch.full((nb,), 0xEE, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
    # exactly what the benchmark times: the bound form, launched on the current stream
    run = plan.bind([t.data_ptr() for t in dev_src], [t.data_ptr() for t in dev_dst])
    run(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for d in range(plan.n_devices):
        got = dev_dst[d].cpu().numpy()
        assert np.array_equal(got, want[d].reshape(-1)), f"{name}: device {d} differs"
    assert plan.scratch_bytes == 0 and plan.height <= max(plan.local_elems(0), plan.local_elems(1))


@pytest.mark.parametrize("w", wl.adversarial_problems(), ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [api.FUSE_ADJACENT, api.FUSE_NONE], ids=lambda m: MODE_NAMES[m])
def test_adversarial_table_problems_full_size(w, mode):
    """P1-P4 of the paper's table (rank 3-6, sizes that are not powers of two, 64-162 MB)."""
    oracle.set_threads(oracle.max_threads())
    try:
        src, dst, src_tiles, want = make_case(w)
    finally:
        oracle.set_threads(1)
    _, got = run_gpu(w.mesh_shape, src, dst, w.elem_bytes, src_tiles, mode)
    assert_same(got, want, w.name)


def test_evaluation_like_problems_reduced():
    """Problems shaped like the paper's evaluation sample (up to 6-D, short trailing dimensions),
    every dimension reduced to its sharding factor times a small multiple."""
    rng = np.random.default_rng(77)
    for k, w in enumerate(wl.evaluation_like_problems(60)):
        shape = []
        for d in range(w.src.rank):
            need = 1
            for ax in (w.src.axes[d], w.dst.axes[d]):
                f = 1
                for a in ax:
                    f *= w.mesh_shape[a]
                need = int(np.lcm(need, f))
            shape.append(need * int(rng.integers(1, 5)))
        ws = w.scaled(shape)
        e = int(rng.choice([2, 4, 8]))
        src, dst = types_of(ws)
        G = rng.integers(0, 256, size=tuple(shape) + (e,), dtype=np.uint8)
        src_tiles = oracle.reslice(ws.mesh_shape, src, G)
        want = oracle.reslice(ws.mesh_shape, dst, G)
        _, got = run_gpu(ws.mesh_shape, src, dst, e, src_tiles, MODES[k % 3])
        assert_same(got, want, ws.name)


EVAL_FULL = ["eval0007", "eval0019", "eval0023", "eval0070", "eval0079", "eval0082", "eval0093", "eval0115",
             "eval0134", "eval0175"]


@pytest.mark.parametrize("name", EVAL_FULL)
def test_evaluation_like_problems_full_size(name):
    """Ten problems of the odd-shape sweep at the size the sweep times them (64-800 MB, f32): unit walk,
    gather walk, zip in both directions, ragged bulk and plain bulk kernels; every target tile compared."""
    w = {p.name: p for p in wl.evaluation_like_problems(200)}[name]
    oracle.set_threads(oracle.max_threads())
    try:
        src, dst, src_tiles, want = make_case(w)
    finally:
        oracle.set_threads(1)
    _, got = run_gpu(w.mesh_shape, src, dst, w.elem_bytes, src_tiles)
    assert_same(got, want, w.name)
    del got, src_tiles, want
    torch.cuda.empty_cache()


_C4 = {}


def config4_global():
    """The 4 GiB global array of the random sweep, generated once for the tests that need it."""
    if "G" not in _C4:
        _C4["G"] = wl.global_array_bytes(wl.CONFIG4_SHAPE, 4, "random_bits", wl.CONFIG4_FILL_SEED)
    return _C4["G"]


def launch_class(plan):
    """What decides which kernel code runs on what shape of work: the variant of every launch, the
    largest fan-out, the number of launches and the shortest contiguous run."""
    li = [plan.launch_info(q) for q in range(plan.num_launches)]
    return (tuple(i.variant for i in li), max(i.fanout for i in li), plan.num_launches, min(i.run_bytes for i in li))


def test_random_sweep_full_size_samples():
    """Three multi-step pairs of the sweep at the full [64,128,256,512] f32 shape (4 GiB global), chosen by
    device footprint; every target tile compared with the oracle's."""
    pairs = wl.config4()
    G = config4_global()
    oracle.set_threads(oracle.max_threads())
    done = 0
    try:
        for w in pairs:
            src, dst = types_of(w)
            plan = api.Plan(w.mesh_shape, src, dst, 4)
            foot = (plan.local_elems(0) + plan.local_elems(1)) * 4 * plan.n_devices
            if foot > 12 * 2**30 or plan.num_steps < 2:
                continue
            src_tiles = oracle.reslice(w.mesh_shape, src, G)
            want = oracle.reslice(w.mesh_shape, dst, G)
            _, got = run_gpu(w.mesh_shape, src, dst, 4, src_tiles)
            assert_same(got, want, w.name)
            done += 1
            if done == 3:
                break
    finally:
        oracle.set_threads(1)
    assert done == 3


def test_random_sweep_full_size_every_launch_class():
    """The sweep at full size in the launch configuration the benchmark times, one pair for every class
    of launch (kernel variant, fan-out, launches, shortest run) that occurs among the 100 pairs.  The
    global array goes to the device once; source tiles are cut from it at the oracle's base offsets
    (replicas share one buffer, as in the benchmark); every target tile is compared on the device with
    the block of the global array at the oracle's base offset for that device -- the definition of the
    result -- and the first and last device's tiles also on the host with the oracle's own tile."""
    pairs = wl.config4()
    classes = {}
    for i, w in enumerate(pairs):
        src, dst = types_of(w)
        classes.setdefault(launch_class(api.Plan(w.mesh_shape, src, dst, 4)), i)
    assert len(classes) >= 20
    G = config4_global()
    Gd = torch.from_numpy(G).cuda()

    def cut(off, tile):
        t = Gd
        for k, (o, c) in enumerate(zip(off, tile)):
            t = t.narrow(k, int(o), int(c))
        return t

    ran = set()
    for key, i in sorted(classes.items()):
        w = pairs[i]
        src, dst = types_of(w)
        plan = api.Plan(w.mesh_shape, src, dst, 4)
        n = plan.n_devices
        tile_s, off_s = oracle.base_offsets(w.mesh_shape, src)
        tile_d, off_d = oracle.base_offsets(w.mesh_shape, dst)
        owned, dev_src = {}, []
        for d in range(n):
            k = tuple(int(o) for o in off_s[d])
            if k not in owned:
                owned[k] = cut(k, tile_s).contiguous().reshape(-1)
            dev_src.append(owned[k])
        nb = plan.local_elems(1) * 4
        dev_dst = [torch.full((nb,), 0xEE, dtype=torch.uint8, device="cuda") for _ in range(n)]
        plan.execute(dev_src, dev_dst, plan.alloc_scratch())
        torch.cuda.synchronize()
        assert launch_class(plan) == key
        for d in range(n):
            want = cut(off_d[d], tile_d)
            assert torch.equal(dev_dst[d].view(tuple(tile_d) + (4,)), want), f"{w.name}: device {d} differs"
        for d in (0, n - 1):
            want = oracle.tile_of(w.mesh_shape, dst, G, d)
            assert np.array_equal(dev_dst[d].cpu().numpy().reshape(want.shape), want), f"{w.name}: device {d} (host)"
        ran.add(key)
        del dev_src, dev_dst, owned
        torch.cuda.empty_cache()
    assert ran == set(classes)        # every class present among the 100 pairs ran at full size
    del Gd
    _C4.clear()
    torch.cuda.empty_cache()


def test_execute_can_be_captured_in_a_cuda_graph_and_replayed():
    """redist_execute allocates nothing and copies no table to the device, so a stream capture records
    just its kernel launches; replays on new data must still match the oracle."""
    w = wl.config2().scaled((8, 256, 512))
    src, dst, src_tiles, want = make_case(w, seed=11)
    for flags in (api.FUSE_ADJACENT, api.FUSE_NONE):
        plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes, flags)
        d_src = [torch.zeros_like(torch.from_numpy(t)).cuda() for t in src_tiles]
        nb = plan.local_elems(1) * w.elem_bytes
        d_dst = [torch.zeros(nb, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
        scratch = plan.alloc_scratch()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            plan.execute(d_src, d_dst, scratch, side)          # warm-up outside the capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        bound = plan.bind([t.data_ptr() for t in d_src], [t.data_ptr() for t in d_dst],
                          scratch.data_ptr() if scratch is not None else 0, plan.scratch_bytes)
        with torch.cuda.graph(g, stream=side):
            if flags == api.FUSE_NONE:      # the bound form is launches only: it captures the same way
                bound(torch.cuda.current_stream().cuda_stream)
            else:
                plan.execute(d_src, d_dst, scratch, torch.cuda.current_stream())
        for seed in (11, 12):
            _, _, tiles, expect = make_case(w, seed=seed)
            for t, h in zip(d_src, tiles):
                t.copy_(torch.from_numpy(h))
            for t in d_dst:
                t.fill_(0xEE)
            g.replay()
            torch.cuda.synchronize()
            assert_same([t.cpu().numpy() for t in d_dst], expect, f"graph replay, seed {seed}, flags {flags}")


def test_back_to_back_dependent_launches_are_ordered():
    """Kernels use programmatic dependent launch; a redistribution that reads what the previous one on
    the same stream wrote must still see all of it (A -> B -> A, 20 times, no synchronisation between)."""
    w = wl.config3("a").scaled((1024, 1024))
    src, dst, src_tiles, _ = make_case(w)
    fwd = api.Plan(w.mesh_shape, src, dst, w.elem_bytes)
    back = api.Plan(w.mesh_shape, dst, src, w.elem_bytes)
    a = [torch.from_numpy(t).cuda() for t in src_tiles]
    b = [torch.zeros(fwd.local_elems(1) * w.elem_bytes, dtype=torch.uint8, device="cuda") for _ in range(8)]
    c = [torch.zeros(fwd.local_elems(0) * w.elem_bytes, dtype=torch.uint8, device="cuda") for _ in range(8)]
    for _ in range(20):
        fwd.execute(a, b)
        back.execute(b, c)
        fwd.execute(c, b)
        back.execute(b, a)
    torch.cuda.synchronize()
    assert_same([t.cpu().numpy() for t in a], src_tiles, "A->B->A chain")
    assert_same([t.cpu().numpy() for t in c], src_tiles, "A->B->A chain (intermediate)")


@pytest.mark.parametrize("mesh,src_axes,dst_axes,gshape", [
    ((4, 4, 4, 4), ((0, 1), (2,), (3,)), ((3,), (1, 0), (2,)), (64, 64, 32)),          # 256 virtual devices
    ((1024,), ((0,), ()), ((), (0,)), (2048, 1024)),                                   # 1024: the table limit
    ((2, 3, 5, 7), ((0, 3), (1,), ()), ((2,), (), (3, 1)), (210, 30, 42)),             # 210 devices, odd primes
    ((8, 16), ((), (0,)), ((1, 0), ()), (256, 64)),                                    # 128 devices, replication
])
@pytest.mark.parametrize("mode", [api.FUSE_ADJACENT, api.FUSE_NONE], ids=lambda m: MODE_NAMES[m])
def test_many_virtual_devices_use_the_large_pointer_tables(mesh, src_axes, dst_axes, gshape, mode):
    """More than 64 tiles on a side switches to the 1024-entry kernel-parameter tables."""
    rng = np.random.default_rng(len(mesh))
    e = 2
    G = rng.integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    src, dst = (gshape, src_axes), (gshape, dst_axes)
    src_tiles = oracle.reslice(mesh, src, G)
    want = oracle.reslice(mesh, dst, G)
    plan, got = run_gpu(mesh, src, dst, e, src_tiles, mode)
    assert plan.n_devices > 64
    assert_same(got, want, f"{mesh}")


def test_rank_eight_and_sixteen_byte_elements():
    mesh = (2, 2, 2)
    gshape = (2, 3, 4, 2, 5, 2, 3, 4)
    src = (gshape, ((0,), (), (1,), (), (), (2,), (), ()))
    dst = (gshape, ((), (), (2,), (0,), (), (), (), (1,)))
    rng = np.random.default_rng(8)
    G = rng.integers(0, 256, size=gshape + (16,), dtype=np.uint8)
    src_tiles = oracle.reslice(mesh, src, G)
    want = oracle.reslice(mesh, dst, G)
    for mode in MODES:
        _, got = run_gpu(mesh, src, dst, 16, src_tiles, mode)
        assert_same(got, want, "rank 8, 16-byte elements")


def test_one_plan_executed_from_several_host_threads():
    """A plan is immutable: host threads may execute it at the same time on their own streams and
    buffers (the foreign call releases the interpreter lock)."""
    import threading
    w = wl.config2().scaled((8, 256, 512))
    src, dst, _, _ = make_case(w)
    plan = api.Plan(w.mesh_shape, src, dst, w.elem_bytes, api.FUSE_NONE)
    nb = plan.local_elems(1) * w.elem_bytes
    jobs = []
    for t in range(4):
        _, _, tiles, want = make_case(w, seed=100 + t)
        jobs.append({"src": [torch.from_numpy(x).cuda() for x in tiles], "want": want,
                     "dst": [torch.zeros(nb, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)],
                     "scratch": plan.alloc_scratch(), "stream": torch.cuda.Stream(), "err": None})
    torch.cuda.synchronize()

    def work(j):
        try:
            for _ in range(50):
                plan.execute(j["src"], j["dst"], j["scratch"], j["stream"])
        except Exception as ex:      # surfaced below
            j["err"] = ex

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    for j in jobs:
        assert j["err"] is None, j["err"]
        assert_same([t.cpu().numpy() for t in j["dst"]], j["want"], "threaded execute")


def test_soak_full_size_forward_and_back_without_synchronising():
    """Config 2 at full size, forward and back 100 times on one stream with no host synchronisation:
    kernels overlap their ramp-up with the previous kernel's tail (programmatic dependent launch) and
    every one reads what the previous one wrote.  The data must come back unchanged."""
    w = wl.bench_workloads()["c2"]
    src, dst = types_of(w)
    G = wl.global_array_bytes(w.src.global_shape, w.elem_bytes, w.fill, w.seed)
    tiles = oracle.reslice(w.mesh_shape, src, G)
    fwd = api.Plan(w.mesh_shape, src, dst, w.elem_bytes)
    back = api.Plan(w.mesh_shape, dst, src, w.elem_bytes)
    a = [torch.from_numpy(t).cuda() for t in tiles]
    b = [torch.zeros(fwd.local_elems(1) * w.elem_bytes, dtype=torch.uint8, device="cuda") for _ in range(8)]
    for _ in range(100):
        fwd.execute(a, b)
        back.execute(b, a)
    torch.cuda.synchronize()
    assert_same([t.cpu().numpy() for t in a], tiles, "soak")
    want = oracle.reslice(w.mesh_shape, dst, G)
    assert_same([t.cpu().numpy() for t in b], want, "soak (intermediate)")
    assert api.redist_bulk_timeouts() == 0


INTERLEAVED = [   # mesh, global shape, sharded type, gathered type, element bytes, variant there, variant back
    ((2, 4), (6, 10, 24), ((), (), (1,)), ((), (), ()), 4, 7, 7),
    ((2, 2, 2), (8, 6, 60), ((0,), (), (1, 2)), ((0,), (), (1,)), 4, 7, 7),
    ((4, 2), (5, 8, 36), ((), (1,), (0,)), ((), (), ()), 4, 5, 7),
    ((2, 3, 2), (4, 9, 180), ((0,), (), (1, 2)), ((), (), (2,)), 4, 7, 7),
    ((8,), (33, 88), ((), (0,)), ((), ()), 4, 7, 7),
    ((2, 2), (16, 6, 4), ((), (), (0, 1)), ((), (0,), ()), 8, 5, 3),
    ((2, 2, 2), (6, 5, 56), ((), (), (0, 1, 2)), ((), (), (0,)), 4, 7, 7),
    ((2, 2, 2), (700, 3, 56), ((), (), (0, 1, 2)), ((), (), (0,)), 4, 7, 7),      # many row groups, ragged last one
    ((2, 4, 4), (6, 416), ((), (0, 1, 2)), ((), ()), 4, 7, 7),                      # 32 tiles zipped into one row, 52-byte runs
    ((4, 4, 4), (8, 320), ((), (2, 1, 0)), ((), ()), 4, 5, 7),                      # 64 tiles, 20-byte runs
    ((2, 4, 4), (5, 4, 864), ((), (), (0, 1, 2)), ((), (), ()), 2, 7, 7),           # 32 tiles, 54-byte runs of 2-byte units
]


@pytest.mark.parametrize("mesh,gshape,sharded,gathered,e,v_there,v_back", INTERLEAVED)
def test_gather_walk_and_zip_kernels(mesh, gshape, sharded, gathered, e, v_there, v_back):
    """Short ragged runs interleaved into long target rows go through the zip kernels (launch variant 7;
    source segments staged in shared memory by bulk copies) or the gather walk (variant 5); the way
    back scatters long source rows over several target tiles."""
    rng = np.random.default_rng(sum(gshape))
    G = rng.integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    for src, dst, variant in (((gshape, sharded), (gshape, gathered), v_there),
                              ((gshape, gathered), (gshape, sharded), v_back)):
        src_tiles = oracle.reslice(mesh, src, G)
        want = oracle.reslice(mesh, dst, G)
        with api.tuning(box=0):          # (the super-box kernels would take some of these shapes)
            plan, got = run_gpu(mesh, src, dst, e, src_tiles)
            assert plan.launch_info(0).variant == variant
            assert_same(got, want, f"interleaved {mesh} {src} -> {dst}")
            _, got = run_gpu(mesh, src, dst, e, src_tiles, api.FUSE_NONE)
            assert_same(got, want, f"interleaved, unfused {mesh} {src} -> {dst}")


SMALL_UNITS = [   # mesh, global shape, source axes, target axes, element bytes, unit bytes: odd runs of 8- and 16-bit elements
    ((2, 4), (6, 10, 28), ((), (), (1,)), ((), (), ()), 2, 2),                                              # 14-byte runs
    ((2, 2, 2), (8, 6, 60), ((0,), (), (1, 2)), ((0,), (), (1,)), 1, 1),                                   # 15- and 30-byte runs
    ((8,), (33, 88), ((), (0,)), ((), ()), 2, 2),                                                          # 22-byte runs
    ((4, 4, 4), (8, 12, 2, 28, 20, 12), ((), (1,), (), (2,), (), ()), ((2,), (), (), (), (0,), (1,)), 2, 2),  # 6-byte runs, 3 inner dimensions
    ((4, 4, 4), (8, 12, 2, 28, 20, 12), ((), (1,), (), (2,), (), ()), ((2,), (), (), (), (0,), (1,)), 1, 1),  # 3-byte runs
    ((4, 2, 2), (2, 17, 16, 28, 9, 8), ((1,), (), (2, 0), (), (), ()), ((), (), (), (1,), (), (0, 2)), 2, 2),  # single elements 16 bytes apart
    ((2, 2, 2), (6, 6, 6, 48, 10, 26), ((), (2,), (), (0,), (), ()), ((), (), (1,), (), (2,), (0,)), 1, 1),  # 13-byte runs
    # runs of 64 bytes and more: chunks inside one run are read in one piece
    ((8,), (33, 520), ((), (0,)), ((), ()), 2, 2),                                                          # 130-byte runs
    ((2, 4), (6, 10, 300), ((), (), (1,)), ((), (), ()), 1, 1),                                            # 75-byte runs
    ((2, 2, 2), (6, 6, 6, 48, 10, 74), ((), (2,), (), (0,), (), ()), ((), (), (1,), (), (2,), (0,)), 2, 2),  # 74-byte runs, super-boxes
    ((2, 2, 2), (4, 6, 6, 48, 10, 150), ((), (2,), (), (0,), (), ()), ((), (), (1,), (), (2,), (0,)), 1, 1), # 75-byte runs, super-boxes
]


@pytest.mark.parametrize("mesh,gshape,a1,a2,e,unit", SMALL_UNITS)
def test_short_run_kernels_on_one_and_two_byte_units(mesh, gshape, a1, a2, e, unit):
    """Odd run lengths of 8- and 16-bit elements leave units of 1 or 2 bytes: the zip, super-box and gather kernels
    assemble a 16-byte chunk from 16 or 8 of them (kernels of their own, so that their registers do not weigh on
    the others).  Both directions; the default choice and each family forced."""
    G = np.random.default_rng(sum(gshape) + e).integers(0, 256, size=gshape + (e,), dtype=np.uint8)
    seen = set()
    for src, dst in (((gshape, a1), (gshape, a2)), ((gshape, a2), (gshape, a1))):
        src_tiles, want = oracle.reslice(mesh, src, G), oracle.reslice(mesh, dst, G)
        for values in ({}, {"box": 2}, {"box": 0}, {"gather": 2, "zip": 0, "box": 0}, {"piece": 0}, {"piece": 0, "box": 2},
                       {"box": 0, "zip_walks": 0}, {"box": 0, "zip_walks": 2, "zip_by_range_slots": 1}, {"box": 0, "zip_walks": 4}):
            with api.tuning(**values):
                plan, got = run_gpu(mesh, src, dst, e, src_tiles)
            assert_same(got, want, f"small units {mesh} {src} -> {dst} {values}")
            for q, L in enumerate(plan.describe()["launches"]):
                assert L["geometry"]["unit_bytes"] == unit
                seen.add(plan.launch_info(q).variant)
    assert seen & {7, 8}, seen


def test_structured_probes_at_reduced_size():
    """Every mesh axis on one dimension over 8-64 devices, odd widths of 2- and 4-byte elements: the 92 shapes of
    `bench.py --workload probes` with eight rows per device (the kernel choice depends on the widths, which stay)."""
    seen = set()
    for w in wl.structured_probes():
        n = w.n_devices
        rows = 8 * n if w.name.startswith("t") else 96
        ws = w.scaled((rows, w.src.global_shape[1]))
        src, dst, src_tiles, want = make_case(ws, seed=len(seen) + 7)
        plan, got = run_gpu(ws.mesh_shape, src, dst, ws.elem_bytes, src_tiles)
        assert_same(got, want, ws.name)
        seen.update(plan.launch_info(q).variant for q in range(plan.num_launches))
    assert seen >= {6, 7, 8}, seen


@pytest.mark.parametrize("g,variant", [((32768, 32768), 4), ((44739243, 24), 7)])
def test_four_gib_tiles_need_64_bit_offsets(g, variant):
    """u32 arrays of 4 GiB and a little more (value = global linear index) on two devices: replicated
    -> column sharded reads at offsets beyond 2^32 inside a tile, column sharded -> replicated writes
    there.  64 KiB rows go by bulk copies, 96-byte rows (48-byte runs) through the zip kernels."""
    mesh = (2,)
    total = g[0] * g[1] * 4
    assert total >= 2**32
    G = wl.global_array_bytes(g, 4, "linear_u32", 0)
    repl, cols = (g, ((), ())), (g, ((), (0,)))
    oracle.set_threads(oracle.max_threads())
    try:
        col_tiles = oracle.reslice(mesh, cols, G)
    finally:
        oracle.set_threads(1)
    one = torch.from_numpy(G.reshape(-1)).cuda()
    plan = api.Plan(mesh, repl, cols, 4)
    assert plan.launch_info(0).variant == variant
    nb = plan.local_elems(1) * 4
    out = [torch.empty(nb, dtype=torch.uint8, device="cuda") for _ in range(2)]
    plan.execute([one, one], out)                      # replicas alias one buffer
    torch.cuda.synchronize()
    assert_same([t.cpu().numpy() for t in out], col_tiles, "replicated -> columns")
    back = api.Plan(mesh, cols, repl, 4)
    assert back.launch_info(0).variant == variant
    full = [torch.empty(total, dtype=torch.uint8, device="cuda") for _ in range(2)]
    back.execute(out, full)
    torch.cuda.synchronize()
    for d in range(2):
        assert torch.equal(full[d], one), f"columns -> replicated, device {d}"
    del full, out, one
    torch.cuda.empty_cache()


def test_zero_bulk_copy_timeouts_after_everything_above():
    """The bounded waits of the bulk-copy kernels never ran out."""
    torch.cuda.synchronize()
    assert api.redist_bulk_timeouts() == 0
