"""Seeded synthetic workloads: meshes, global arrays and (source type, target type) pairs.

This module only *describes* inputs.  It holds none of the method's arithmetic (no base
offsets, no tiling, no plan): it names meshes and distributed types and fills global arrays.
It imports nothing else from this package, so test infrastructure can use it without loading
the CUDA library.

Notation (Section 2.1 of the paper, "Distributed array types"): a distributed type gives, per
array dimension, the ordered list of mesh axes that partition it, listed minor-to-major (the
first listed axis varies fastest).  Axes are named here by their index into ``mesh_shape``.
A virtual device id is the row-major index of its coordinates over ``mesh_shape`` (last mesh
axis fastest).

The paper's evaluation samples 1000 problems with 3 mesh axes, arrays of up to 6 dimensions
and 64 MB-800 MB of global data, each mesh axis either replicated or partitioning one
dimension (Section 8, "Evaluation").  Those problems are not published; the workloads below
stand in for them with the same structure.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

AxesPerDim = Tuple[Tuple[int, ...], ...]


@dataclass(frozen=True)
class DistType:
    """A distributed array type: global shape plus, per dimension, its mesh axes (minor first)."""

    global_shape: Tuple[int, ...]
    axes: AxesPerDim

    def __post_init__(self):
        if len(self.global_shape) != len(self.axes):
            raise ValueError("one axis list per dimension is required")

    @property
    def rank(self) -> int:
        return len(self.global_shape)

    def notation(self, mesh_shape: Sequence[int], names: Sequence[str] | None = None) -> str:
        """Render as the paper writes types, e.g. ``[2{x}8, 2048, 2048{y}4096]``."""
        names = list(names) if names is not None else [f"a{i}" for i in range(len(mesh_shape))]
        parts = []
        for s, ax in zip(self.global_shape, self.axes):
            if not ax:
                parts.append(str(s))
                continue
            k = 1
            for a in ax:
                k *= mesh_shape[a]
            tile = s // k if s % k == 0 else f"{s}/{k}"
            parts.append(f"{tile}{{{','.join(names[a] for a in ax)}}}{s}")
        return "[" + ", ".join(parts) + "]"


def dist_type(global_shape: Sequence[int], axes: Sequence[Sequence[int]]) -> DistType:
    return DistType(tuple(int(s) for s in global_shape), tuple(tuple(int(a) for a in ax) for ax in axes))


@dataclass(frozen=True)
class Workload:
    """One redistribution problem: mesh, element size, source and target type, fill recipe."""

    name: str
    mesh_shape: Tuple[int, ...]
    axis_names: Tuple[str, ...]
    elem_bytes: int
    src: DistType
    dst: DistType
    fill: str          # "linear_u32" or "random_bits"
    seed: int
    note: str = ""

    @property
    def n_devices(self) -> int:
        n = 1
        for k in self.mesh_shape:
            n *= k
        return n

    @property
    def global_elems(self) -> int:
        n = 1
        for s in self.src.global_shape:
            n *= s
        return n

    def reversed(self) -> "Workload":
        return Workload(self.name + "_back", self.mesh_shape, self.axis_names, self.elem_bytes,
                        self.dst, self.src, self.fill, self.seed, self.note)

    def scaled(self, global_shape: Sequence[int], name_suffix: str = "_small") -> "Workload":
        """Same mesh and axis placement on a different global shape (for parity-sized cases)."""
        gs = tuple(int(s) for s in global_shape)
        return Workload(self.name + name_suffix, self.mesh_shape, self.axis_names, self.elem_bytes,
                        DistType(gs, self.src.axes), DistType(gs, self.dst.axes), self.fill, self.seed,
                        self.note)


def global_array_bytes(shape: Sequence[int], elem_bytes: int, fill: str, seed: int) -> np.ndarray:
    """The logical global array as raw bytes, shape ``(*shape, elem_bytes)``, dtype uint8.

    ``linear_u32``: element value is its global row-major linear index (4-byte little endian).
    ``random_bits``: every bit drawn from ``numpy.random.default_rng(seed)``; bf16/f32 arrays
    are filled this way so the patterns include NaNs and denormals (comparison is bytewise).
    """
    shape = tuple(int(s) for s in shape)
    n = 1
    for s in shape:
        n *= s
    if fill == "linear_u32":
        if elem_bytes != 4:
            raise ValueError("linear_u32 fill needs 4-byte elements")
        g = np.arange(n, dtype="<u4").view(np.uint8)
    elif fill == "random_bits":
        rng = np.random.default_rng(seed)
        g = rng.integers(0, 256, size=n * elem_bytes, dtype=np.uint8)
    else:
        raise ValueError(f"unknown fill {fill!r}")
    return g.reshape(shape + (elem_bytes,))


# ----------------------------------------------------------------------------------------------
# The five benchmark configurations (full size).  Axis lists are minor-to-major.
# ----------------------------------------------------------------------------------------------

def config1() -> Workload:
    """uint32 [256,256], value = global linear index, mesh (x:2, y:2); {d0:x,d1:y} -> {d0:y,d1:x}."""
    gs = (256, 256)
    return Workload("c1", (2, 2), ("x", "y"), 4, dist_type(gs, [[0], [1]]), dist_type(gs, [[1], [0]]),
                    "linear_u32", 2112010751, "swap across dimensions")


def config2() -> Workload:
    """bf16 [8,2048,4096], mesh (x:4, y:2); {d0:x,d2:y} -> {d1:(x,y)} (x minor)."""
    gs = (8, 2048, 4096)
    return Workload("c2", (4, 2), ("x", "y"), 2, dist_type(gs, [[0], [], [1]]), dist_type(gs, [[], [0, 1], []]),
                    "random_bits", 2112010752, "activation reshard")


def config3(which: str) -> Workload:
    """bf16 [16384,16384], mesh (a:8): 'a' row->col, 'b' replicated->row, 'c' col->replicated."""
    gs = (16384, 16384)
    rows, cols, repl = dist_type(gs, [[0], []]), dist_type(gs, [[], [0]]), dist_type(gs, [[], []])
    src, dst = {"a": (rows, cols), "b": (repl, rows), "c": (cols, repl)}[which]
    return Workload("c3" + which, (8,), ("a",), 2, src, dst, "random_bits", 2112010753, "weight reshard")


def config5(which: str) -> Workload:
    """bf16 [32768,32768], mesh (x:4,y:4,z:4): 'a' {d0:(x,y),d1:z}->{d0:(y,x),d1:z}; 'b' ->{d0:z,d1:(y,x)}."""
    gs = (32768, 32768)
    src = dist_type(gs, [[0, 1], [2]])
    dst = {"a": dist_type(gs, [[1, 0], [2]]), "b": dist_type(gs, [[2], [1, 0]])}[which]
    return Workload("c5" + which, (4, 4, 4), ("x", "y", "z"), 2, src, dst, "random_bits", 2112010755,
                    "permutation heavy")


CONFIG4_MESH = (2, 4, 2)
CONFIG4_SHAPE = (64, 128, 256, 512)
CONFIG4_PAIR_SEED = 2112010764
CONFIG4_FILL_SEED = 2112010754


def _draw_type(rng: np.random.Generator, mesh_shape: Sequence[int], global_shape: Sequence[int]) -> DistType:
    """Each mesh axis independently: replicated or partitions one uniformly chosen dimension;
    the axis list of every dimension is then shuffled (ordered subsets, multi-axis dims allowed)."""
    rank = len(global_shape)
    per_dim: List[List[int]] = [[] for _ in range(rank)]
    for a in range(len(mesh_shape)):
        choice = int(rng.integers(0, rank + 1))      # rank == replicated
        if choice < rank:
            per_dim[choice].append(a)
    out = []
    for k in range(rank):
        ax = per_dim[k]
        if len(ax) > 1:
            ax = [ax[i] for i in rng.permutation(len(ax))]
        out.append(ax)
    return dist_type(global_shape, out)


def random_pairs(n_pairs: int, mesh_shape: Sequence[int], global_shape: Sequence[int], seed: int,
                 elem_bytes: int = 4, fill_seed: int = 0, name: str = "rand") -> List[Workload]:
    """Seeded random (source, target) pairs in the shape of the paper's sampled problems."""
    rng = np.random.default_rng(seed)
    names = tuple("xyzuvw"[: len(mesh_shape)])
    out = []
    for i in range(n_pairs):
        src = _draw_type(rng, mesh_shape, global_shape)
        dst = _draw_type(rng, mesh_shape, global_shape)
        out.append(Workload(f"{name}{i:03d}", tuple(mesh_shape), names, elem_bytes, src, dst,
                            "random_bits", fill_seed, "random sweep"))
    return out


def config4(n_pairs: int = 100, global_shape: Sequence[int] = CONFIG4_SHAPE) -> List[Workload]:
    """f32 [64,128,256,512], mesh (x:2,y:4,z:2): 100 seeded random (src, dst) pairs."""
    return random_pairs(n_pairs, CONFIG4_MESH, global_shape, CONFIG4_PAIR_SEED, 4, CONFIG4_FILL_SEED, "c4_")


def bench_workloads() -> Dict[str, Workload]:
    """Named single problems of the benchmark configurations at full size."""
    c1, c2 = config1(), config2()
    w = {"c1": c1, "c1_back": c1.reversed(), "c2": c2, "c2_back": c2.reversed()}
    for k in "abc":
        w["c3" + k] = config3(k)
    for k in "ab":
        w["c5" + k] = config5(k)
    return w


def adversarial_problems() -> List[Workload]:
    """The four problems of the paper's table of largest slow-downs (Section 8), printed there with
    their axis sizes inline (three mesh axes a, b, c of size 2): 4-byte elements, 64-162 MB global
    data, up to six dimensions, sizes that are not powers of two."""
    mesh, names = (2, 2, 2), ("a", "b", "c")
    a, b, c = 0, 1, 2
    spec = [
        ("P1", (360, 368, 320), [[], [c], []], [[c, a], [], [b]]),
        ("P2", (80, 80, 72, 64), [[], [c], [], []], [[b], [], [c], []]),
        ("P3", (296, 360, 312), [[], [], [c]], [[b, c], [a], []]),
        ("P4", (16, 16, 16, 16, 16, 16), [[c], [], [], [a], [], [b]], [[], [], [], [], [], [a]]),
    ]
    return [Workload(n, mesh, names, 4, dist_type(g, s), dist_type(g, d), "random_bits", 2112010760 + i,
                     "adversarial table") for i, (n, g, s, d) in enumerate(spec)]


def structured_probes() -> List[Workload]:
    """Shapes a random sample seldom draws: every mesh axis on ONE dimension, over 8, 16, 32 and 64 devices, with
    odd widths per device.  Row-to-column transposes (2- and 4-byte elements, widths of 3 to 257 elements),
    and slices / allgathers of the last dimension of a replicated array (4-byte elements, widths of 33 to 401).
    About 256 MB (transposes) and 200 MB (slices) of global data each."""
    meshes = {8: (2, 2, 2), 16: (2, 2, 4), 32: (2, 4, 4), 64: (4, 4, 4)}
    names = ("a", "b", "c")
    out: List[Workload] = []
    for n, mesh in meshes.items():
        axes = [0, 1, 2]
        for e in (4, 2):
            for w in (3, 7, 13, 33, 65, 129, 257):
                cols = n * w
                rows = max(n, ((256 << 20) // (cols * e)) // n * n)
                g = (rows, cols)
                out.append(Workload(f"t{n}_e{e}_w{w}", mesh, names, e, dist_type(g, [axes, []]), dist_type(g, [[], axes]),
                                    "random_bits", 0, "row-sharded to column-sharded"))
    for n, mesh in meshes.items():
        if n == 64:
            continue
        axes = [0, 1, 2]
        for w in (33, 65, 93, 129, 255, 401):
            cols = n * w
            g = (max(64, (200 << 20) // (cols * 4)), cols)
            out.append(Workload(f"s{n}_w{w}", mesh, names, 4, dist_type(g, [[], []]), dist_type(g, [[], axes]),
                                "random_bits", 0, "replicated to sliced along the last dimension"))
            out.append(Workload(f"g{n}_w{w}", mesh, names, 4, dist_type(g, [[], axes]), dist_type(g, [[], []]),
                                "random_bits", 0, "sliced along the last dimension to replicated"))
    return out


def evaluation_like_problems(n: int, seed: int = 2112010770) -> List[Workload]:
    """Random problems in the shape of the paper's evaluation sample (Section 8): three mesh axes,
    arrays of two to six dimensions holding 64 MB-800 MB of 4-byte elements, every axis either
    replicated or partitioning one dimension.  Dimension sizes are balanced around the geometric
    mean of the array (within a factor of four), as in the four problems the paper prints
    ([360,368,320], [80,80,72,64], [296,360,312], [16]*6), and need not be powers of two.
    Used for planner throughput and for the odd-shape sweep."""
    rng = np.random.default_rng(seed)
    lo, hi = 16 * 2**20, 200 * 2**20                      # elements
    out: List[Workload] = []
    while len(out) < n:
        mesh = tuple(int(rng.choice([2, 2, 2, 4])) for _ in range(3))
        rank = int(rng.integers(2, 7))
        unit = [1] * rank
        src, dst = _draw_type(rng, mesh, unit), _draw_type(rng, mesh, unit)
        need = []
        for k in range(rank):
            f1 = f2 = 1
            for a in src.axes[k]:
                f1 *= mesh[a]
            for a in dst.axes[k]:
                f2 *= mesh[a]
            need.append(int(np.lcm(f1, f2)))
        target = float(rng.integers(lo, hi))
        gm = target ** (1.0 / rank)
        shape = []
        for k in range(rank):
            want = gm * 2.0 ** float(rng.uniform(-2.0, 2.0))
            shape.append(need[k] * max(1, int(round(want / need[k]))))
        total = 1
        for v in shape:
            total *= v
        if not lo <= total <= hi:
            continue
        out.append(Workload(f"eval{len(out):04d}", mesh, ("a", "b", "c"), 4, dist_type(shape, src.axes),
                            dist_type(shape, dst.axes), "random_bits", 0, "evaluation-like"))
    return out
