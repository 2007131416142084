"""TEST INFRASTRUCTURE -- ctypes front end of the C oracle ``redist_oracle.c``.

A distributed type is passed as ``(global_shape, axes)`` where ``axes[k]`` lists the mesh axes
(indices into ``mesh_shape``) that partition dimension ``k``, minor-to-major (Section 2.1 of the
paper).  Tiles are numpy ``uint8`` arrays of shape ``(*tile_shape, elem_bytes)``; everything is
compared bytewise because the synthetic bf16/f32 patterns include NaNs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "redist_oracle.c")
_LIB = os.path.join(_HERE, "libredist_oracle.so")
_lib = None

_ERR = {1: "invalid argument", 2: "ill-formed type", 3: "tile size does not divide", 4: "replicas differ"}


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}: {_ERR.get(code, '?')}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP when available).  Building is not using it."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-o", tmp, _SRC]
    try:
        subprocess.run(cmd, check=True, capture_output=True, text=True)
    except subprocess.CalledProcessError:
        cmd.remove("-fopenmp")
        subprocess.run(cmd, check=True, capture_output=True, text=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_max_threads.restype = ctypes.c_int
        _lib.orc_get_threads.restype = ctypes.c_int
    return _lib


def set_threads(n: int) -> None:
    _load().orc_set_threads(ctypes.c_int(int(n)))


def max_threads() -> int:
    return int(_load().orc_max_threads())


def _i64(seq):
    return (ctypes.c_int64 * len(seq))(*[int(v) for v in seq])


def _type_args(mesh_shape: Sequence[int], dtype: Tuple[Sequence[int], Sequence[Sequence[int]]]):
    gshape, axes = dtype
    off, flat = [0], []
    for ax in axes:
        flat.extend(int(a) for a in ax)
        off.append(len(flat))
    return (ctypes.c_int(len(mesh_shape)), _i64(mesh_shape), ctypes.c_int(len(gshape)), _i64(gshape),
            (ctypes.c_int32 * len(off))(*off), (ctypes.c_int32 * max(1, len(flat)))(*flat))


def _n_devices(mesh_shape) -> int:
    n = 1
    for k in mesh_shape:
        n *= int(k)
    return n


def base_offsets(mesh_shape, dtype) -> Tuple[Tuple[int, ...], np.ndarray]:
    """``(tile_shape, offsets[N, rank])``: every device's base offset T[[tau]](d)."""
    lib = _load()
    rank, n = len(dtype[0]), _n_devices(mesh_shape)
    tile = (ctypes.c_int64 * rank)()
    off = np.zeros((n, rank), dtype=np.int64)
    rc = lib.orc_base_offsets(*_type_args(mesh_shape, dtype), tile, off.ctypes.data_as(ctypes.c_void_p))
    if rc:
        raise OracleError(rc)
    return tuple(int(t) for t in tile), off


def _ptr_array(arrs: Sequence[np.ndarray]):
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def materialize(mesh_shape, dtype, shards: Sequence[np.ndarray], check: bool = True) -> np.ndarray:
    """Assemble the global array (uint8, shape ``(*global_shape, elem_bytes)``) from source tiles."""
    lib = _load()
    gshape = tuple(int(s) for s in dtype[0])
    e = int(shards[0].shape[-1])
    tile, _ = base_offsets(mesh_shape, dtype)
    if len(shards) != _n_devices(mesh_shape):
        raise ValueError("one tile per device is required")
    shards = [np.ascontiguousarray(s, dtype=np.uint8) for s in shards]
    for s in shards:
        if tuple(s.shape) != tile + (e,):
            raise ValueError(f"tile shape {s.shape} != {tile + (e,)}")
    G = np.empty(gshape + (e,), dtype=np.uint8)
    rc = lib.orc_materialize(*_type_args(mesh_shape, dtype), ctypes.c_int(e), _ptr_array(shards),
                             G.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(1 if check else 0))
    if rc:
        raise OracleError(rc)
    return G


def reslice(mesh_shape, dtype, G: np.ndarray, out: List[np.ndarray] | None = None) -> List[np.ndarray]:
    """Every device's tile of the global array ``G`` under ``dtype``."""
    lib = _load()
    gshape = tuple(int(s) for s in dtype[0])
    G = np.ascontiguousarray(G, dtype=np.uint8)
    e = int(G.shape[-1])
    if tuple(G.shape[:-1]) != gshape:
        raise ValueError("global array shape does not match the type")
    tile, _ = base_offsets(mesh_shape, dtype)
    n = _n_devices(mesh_shape)
    if out is None:
        out = [np.empty(tile + (e,), dtype=np.uint8) for _ in range(n)]
    rc = lib.orc_reslice(*_type_args(mesh_shape, dtype), ctypes.c_int(e), G.ctypes.data_as(ctypes.c_void_p),
                         _ptr_array(out))
    if rc:
        raise OracleError(rc)
    return out


def tile_of(mesh_shape, dtype, G: np.ndarray, device: int) -> np.ndarray:
    """One device's tile of the global array ``G`` under ``dtype``: the block of ``G`` that starts at the
    device's base offset T[[tau]](d) and has the local tile shape (the same definition as ``reslice``,
    for callers that cannot hold every tile at once).  Returns a view into ``G``."""
    tile, off = base_offsets(mesh_shape, dtype)
    if tuple(G.shape[:-1]) != tuple(int(s) for s in dtype[0]):
        raise ValueError("global array shape does not match the type")
    return G[tuple(slice(int(o), int(o) + int(c)) for o, c in zip(off[device], tile))]


def redistribute(mesh_shape, src_type, dst_type, shards: Sequence[np.ndarray], check: bool = True) -> List[np.ndarray]:
    """The definition: assemble the global array under ``src_type``, slice it under ``dst_type``.

    Valid only when both types describe the same global array (Section 2.5, redistribution
    semantics)."""
    if tuple(src_type[0]) != tuple(dst_type[0]):
        raise OracleError(1)
    return reslice(mesh_shape, dst_type, materialize(mesh_shape, src_type, shards, check))
