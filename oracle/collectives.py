"""TEST INFRASTRUCTURE -- the paper's typing rules, cost model and a numpy step simulator.

Used to check a synthesized sequence of collectives step by step; never imported by the product.

A *type* here is a list, per array dimension, of mesh-axis indices (minor-to-major, Section 2.1)
over a mesh given as a tuple of axis sizes; the global shape is carried separately.

Rules follow the figure "Typing collective operations" (T-AllGather, T-DynSlice, T-AllToAll,
T-Permute), their multi-axes forms (Section 7.1, "Merging collective operations": the single axis
x becomes a sequence of axes), and the low-level forms of the figure "Semantics of low-level
collective operations" in which the acted-on axes may sit anywhere in their dimension and are
first brought to the front by relabelling devices, which moves no data.

Costs follow the figure "Costs derived from the total number of bytes communicated":
permute = localsize before, dynslice = 0, allgather = localsize after, alltoall = localsize before.

The simulator works on *operational* readings of the collectives (Appendix B, "Derivation of
data transfer cost": alltoall splits the local tile in n parts, sends part b to group member b,
which concatenates what it receives; allgather concatenates the group's tiles; dynslice keeps a
sub-block).  Tests compare every simulated state with the slice its type prescribes, which pins
the operational readings against the base-offset semantics.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Sequence, Tuple

import numpy as np

Axes = Tuple[Tuple[int, ...], ...]


class TypeError_(ValueError):
    """A collective does not type-check."""


def _prod(xs) -> int:
    n = 1
    for x in xs:
        n *= int(x)
    return n


def norm_axes(axes) -> Axes:
    return tuple(tuple(int(a) for a in ax) for ax in axes)


def well_formed(mesh: Sequence[int], gshape: Sequence[int], axes) -> bool:
    """Rules wf-dim and wf-type."""
    seen = set()
    if len(gshape) != len(axes):
        return False
    for s, ax in zip(gshape, axes):
        k = 1
        for a in ax:
            if a < 0 or a >= len(mesh) or a in seen:
                return False
            seen.add(a)
            k *= mesh[a]
        if s % k:
            return False
    return True


def localtype(mesh, gshape, axes) -> Tuple[int, ...]:
    if not well_formed(mesh, gshape, axes):
        raise TypeError_("ill-formed type")
    return tuple(int(s) // _prod(mesh[a] for a in ax) for s, ax in zip(gshape, axes))


def localsize(mesh, gshape, axes) -> int:
    return _prod(localtype(mesh, gshape, axes))


def used_axes(axes) -> set:
    return {a for ax in axes for a in ax}


# ---------------------------------------------------------------------------------- typing rules

def t_allgather(mesh, gshape, axes, i: int, n_axes: int = 1) -> Axes:
    """Remove the ``n_axes`` minor-most axes of dimension ``i``."""
    axes = norm_axes(axes)
    if n_axes < 1 or len(axes[i]) < n_axes:
        raise TypeError_("allgather: dimension has too few axes")
    out = list(axes)
    out[i] = axes[i][n_axes:]
    return tuple(out)


def t_dynslice(mesh, gshape, axes, i: int, new_axes: Sequence[int]) -> Axes:
    """Introduce ``new_axes`` as the minor-most axes of dimension ``i``."""
    axes = norm_axes(axes)
    new_axes = tuple(int(a) for a in new_axes)
    if not new_axes or len(set(new_axes)) != len(new_axes):
        raise TypeError_("dynslice: bad axis sequence")
    if used_axes(axes) & set(new_axes):
        raise TypeError_("dynslice: axis already partitions a dimension")
    c = localtype(mesh, gshape, axes)[i]
    if c % _prod(mesh[a] for a in new_axes):
        raise TypeError_("dynslice: local size not divisible")
    out = list(axes)
    out[i] = new_axes + axes[i]
    return tuple(out)


def t_alltoall(mesh, gshape, axes, i: int, j: int, n_axes: int = 1) -> Axes:
    """Move the ``n_axes`` minor-most axes of dimension ``i`` to the minor-most end of ``j``."""
    axes = norm_axes(axes)
    if i == j or n_axes < 1 or len(axes[i]) < n_axes:
        raise TypeError_("alltoall: bad dimensions or too few axes")
    moved = axes[i][:n_axes]
    c = localtype(mesh, gshape, axes)[j]
    if c % _prod(mesh[a] for a in moved):
        raise TypeError_("alltoall: local size of the target dimension not divisible")
    out = list(axes)
    out[i] = axes[i][n_axes:]
    out[j] = moved + axes[j]
    return tuple(out)


def t_permute_ok(mesh, gshape, axes1, axes2) -> bool:
    return localtype(mesh, gshape, axes1) == localtype(mesh, gshape, axes2)


def to_front(axes, i: int, which: Sequence[int]) -> Axes:
    """Low-level rules: the axes acted on are brought to the front of dimension ``i`` (beta')."""
    axes = norm_axes(axes)
    which = tuple(int(a) for a in which)
    if not set(which) <= set(axes[i]) or len(set(which)) != len(which):
        raise TypeError_("axes are not in the dimension")
    out = list(axes)
    out[i] = which + tuple(a for a in axes[i] if a not in which)
    return tuple(out)


# ------------------------------------------------------------------------------------- cost model

def step_cost(kind: str, mesh, gshape, before, after) -> int:
    if kind == "dynslice":
        return 0
    if kind == "allgather":
        return localsize(mesh, gshape, after)
    if kind in ("alltoall", "allpermute"):
        return localsize(mesh, gshape, before)
    raise ValueError(kind)


def height(mesh, gshape, types) -> int:
    return max(localsize(mesh, gshape, t) for t in types)


NORMAL_FORM = __import__("re").compile(r"^(d)*(a|p)*(g)*$")


def is_normal_form(kinds: Sequence[str]) -> bool:
    """dynslice* {alltoall | allpermute}* allgather* (definition of normal form, Section 4.3)."""
    code = {"dynslice": "d", "alltoall": "a", "allpermute": "p", "allgather": "g"}
    return NORMAL_FORM.match("".join(code[k] for k in kinds)) is not None


# ---------------------------------------------------------------------------- base offsets (D, T)

def dim_offset(mesh, c: int, ax: Sequence[int], coord: Sequence[int]) -> int:
    """D[[c{x, xs}n]](i) = c*i_x + D[[(c*k){xs}n]](i); D[[c{}c]] = 0  -- written recursively."""
    if not ax:
        return 0
    x = ax[0]
    return c * coord[x] + dim_offset(mesh, c * mesh[x], ax[1:], coord)


def type_offsets(mesh, gshape, axes, coord) -> Tuple[int, ...]:
    lt = localtype(mesh, gshape, axes)
    return tuple(dim_offset(mesh, lt[k], axes[k], coord) for k in range(len(gshape)))


# --------------------------------------------------------------------------------- step simulator

@dataclass
class State:
    """A device assignment <phi, beta> with data: ``coords[d]`` are the logical mesh coordinates
    of physical device ``d`` (phi^-1), ``axes`` the current type, ``tiles[d]`` the local tile as a
    uint8 array of shape ``(*localtype, elem_bytes)``."""

    mesh: Tuple[int, ...]
    gshape: Tuple[int, ...]
    axes: Axes
    coords: List[Tuple[int, ...]]
    tiles: List[np.ndarray]

    def offsets(self, d: int) -> Tuple[int, ...]:
        return type_offsets(self.mesh, self.gshape, self.axes, self.coords[d])

    def expected_tile(self, G: np.ndarray, d: int) -> np.ndarray:
        lt = localtype(self.mesh, self.gshape, self.axes)
        off = self.offsets(d)
        sl = tuple(slice(o, o + c) for o, c in zip(off, lt))
        return G[sl]

    def check_against(self, G: np.ndarray) -> None:
        for d in range(len(self.tiles)):
            exp = self.expected_tile(G, d)
            if self.tiles[d].shape != exp.shape or not np.array_equal(self.tiles[d], exp):
                raise AssertionError(f"device {d}: tile is not the slice its type prescribes")


def _group_key(coord, acting: Sequence[int]):
    return tuple(c for a, c in enumerate(coord) if a not in acting)


def _group_pos(mesh, coord, acting: Sequence[int]) -> int:
    """Position inside the group: mixed radix over the acting axes, first listed = fastest."""
    pos, stride = 0, 1
    for a in acting:
        pos += coord[a] * stride
        stride *= mesh[a]
    return pos


def _groups(state: State, acting: Sequence[int]) -> Dict[tuple, List[int]]:
    n = _prod(state.mesh[a] for a in acting)
    groups: Dict[tuple, List[int]] = {}
    for d, c in enumerate(state.coords):
        groups.setdefault(_group_key(c, acting), [None] * n)[_group_pos(state.mesh, c, acting)] = d
    for g in groups.values():
        assert all(m is not None for m in g), "device map is not a bijection on the group"
    return groups


def relabel(state: State, new_coords: Sequence[Sequence[int]], new_axes) -> State:
    """Change <phi, beta> to an equivalent <phi', beta'>: legal iff no device's base offset
    changes (beta' o phi'^-1 = beta o phi^-1), so no data moves."""
    new = State(state.mesh, state.gshape, norm_axes(new_axes), [tuple(c) for c in new_coords], state.tiles)
    if sorted(new.coords) != sorted(state.coords) or len(set(new.coords)) != len(new.coords):
        raise AssertionError("relabelled device map is not a bijection onto the mesh")
    for d in range(len(state.tiles)):
        if new.offsets(d) != state.offsets(d):
            raise AssertionError(f"relabel changes the base offset of device {d}")
    return new


def sim_allgather(state: State, i: int, acting: Sequence[int]) -> State:
    """Every group member receives the concatenation along dim ``i`` of the group's tiles."""
    if tuple(state.axes[i][: len(acting)]) != tuple(acting):
        raise TypeError_("allgather: acting axes are not minor-most")
    new_axes = t_allgather(state.mesh, state.gshape, state.axes, i, len(acting))
    tiles = [None] * len(state.tiles)
    for members in _groups(state, acting).values():
        cat = np.concatenate([state.tiles[m] for m in members], axis=i)
        for m in members:
            tiles[m] = cat
    return State(state.mesh, state.gshape, new_axes, state.coords, tiles)


def sim_dynslice(state: State, i: int, acting: Sequence[int]) -> State:
    """Every device keeps sub-block number (its position on the new axes) of its tile along ``i``."""
    new_axes = t_dynslice(state.mesh, state.gshape, state.axes, i, acting)
    n = _prod(state.mesh[a] for a in acting)
    tiles = []
    for d, t in enumerate(state.tiles):
        b = _group_pos(state.mesh, state.coords[d], acting)
        tiles.append(np.split(t, n, axis=i)[b])
    return State(state.mesh, state.gshape, new_axes, state.coords, tiles)


def sim_alltoall(state: State, i: int, j: int, acting: Sequence[int]) -> State:
    """Member a splits its tile in n parts along ``j`` and sends part b to member b; member b
    concatenates the parts it received along ``i`` in the order of the senders."""
    if tuple(state.axes[i][: len(acting)]) != tuple(acting):
        raise TypeError_("alltoall: acting axes are not minor-most")
    new_axes = t_alltoall(state.mesh, state.gshape, state.axes, i, j, len(acting))
    n = _prod(state.mesh[a] for a in acting)
    tiles = [None] * len(state.tiles)
    for members in _groups(state, acting).values():
        parts = [np.split(state.tiles[m], n, axis=j) for m in members]
        for b, m in enumerate(members):
            tiles[m] = np.concatenate([parts[a][b] for a in range(n)], axis=i)
    return State(state.mesh, state.gshape, new_axes, state.coords, tiles)


def sim_permute(state: State, source_of: Sequence[int], new_coords, new_axes) -> State:
    """Device d receives the whole tile of device ``source_of[d]`` (a bijection on devices)."""
    if sorted(source_of) != list(range(len(state.tiles))):
        raise AssertionError("allpermute: not a bijection")
    if not t_permute_ok(state.mesh, state.gshape, state.axes, new_axes):
        raise TypeError_("allpermute: local types differ")
    tiles = [state.tiles[s] for s in source_of]
    return State(state.mesh, state.gshape, norm_axes(new_axes), [tuple(c) for c in new_coords], tiles)
