"""Thin Python binding of the C boundary declared in ``include/redist.h``.

Argument marshalling only: every step of a redistribution runs in the CUDA library.  PyTorch is
used for device memory and streams, nothing else.  There is no CPU fallback: if the library has
not been built, loading fails with an error that says how to build it.

A distributed type is ``(global_shape, axes)`` -- or any object with ``global_shape`` and ``axes``
attributes -- where ``axes[k]`` lists the mesh axes (indices into ``mesh_shape``) that partition
dimension ``k``, minor-to-major (Section 2.1 of the paper).
"""
from __future__ import annotations

import contextlib
import ctypes
import json
import os
from typing import List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("REDIST_LIB") or os.path.join(HERE, "libredist_b200.so")

FUSE_ADJACENT, FUSE_NONE, FUSE_ALL, NAIVE = 0, 1, 2, 3
NO_OVERPARTITION = 16
COST_PERMUTE = 32
NO_CACHE = 64
MAX_RANK = 8
STATIC_SCRATCH_BYTES = 8 << 20

STEP_KINDS = ("dynslice", "alltoall", "allgather", "allpermute", "copy")
KERNELS = ("dynslice", "alltoall", "allgather", "allpermute", "copy", "fused", "naive_gather", "naive_slice")

EXPORTS = (
    "redist_plan", "redist_plan_destroy", "redist_execute", "redist_execute_host", "redist_execute_static",
    "redist_bind", "redist_bound_execute", "redist_bound_destroy",
    "redist_plan_cache_stats", "redist_plan_cache_clear",
    "redist_tuning_set", "redist_tuning_get", "redist_tuning_reset", "redist_debug_bounds_report",
    "redist_plan_gpu_split",
    "redist_plan_num_devices", "redist_plan_rank", "redist_plan_local_elems", "redist_plan_scratch_bytes",
    "redist_plan_scratch_bytes_per_device", "redist_plan_staging_bytes", "redist_plan_alignment",
    "redist_plan_height", "redist_plan_cost", "redist_plan_num_steps", "redist_plan_num_launches",
    "redist_plan_step_info", "redist_plan_launch_info", "redist_plan_describe", "redist_base_offsets",
    "redist_status_string", "redist_last_cuda_error", "redist_bulk_timeouts",
)


class RedistError(RuntimeError):
    def __init__(self, status: int, what: str = ""):
        self.status = int(status)
        msg = _status_string(status)
        super().__init__(f"{what}: {msg} (status {status})" if what else f"{msg} (status {status})")


class _Type(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("global_shape", ctypes.POINTER(ctypes.c_int64)),
                ("axes_off", ctypes.POINTER(ctypes.c_int32)), ("axes", ctypes.POINTER(ctypes.c_int32))]


class StepInfo(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("dim_i", ctypes.c_int32), ("dim_j", ctypes.c_int32),
                ("factor", ctypes.c_int64), ("local_before", ctypes.c_int64 * MAX_RANK),
                ("local_after", ctypes.c_int64 * MAX_RANK), ("cost", ctypes.c_int64),
                ("localsize_after", ctypes.c_int64)]


class LaunchInfo(ctypes.Structure):
    _fields_ = [("first_step", ctypes.c_int32), ("n_steps", ctypes.c_int32), ("kernel", ctypes.c_int32),
                ("vector_bytes", ctypes.c_int32), ("run_bytes", ctypes.c_int64), ("bytes_read", ctypes.c_int64),
                ("bytes_written", ctypes.c_int64), ("n_items", ctypes.c_int64), ("fanout", ctypes.c_int32),
                ("variant", ctypes.c_int32)]


_lib = None


def load() -> ctypes.CDLL:
    """Load ``libredist_b200.so``; raise if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2112_01075_b200.build` "
            "(needs nvcc; cross-compiles for sm_100a without a GPU)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.redist_plan.argtypes = [i32, ctypes.POINTER(i64), ctypes.POINTER(_Type), ctypes.POINTER(_Type), i32,
                                ctypes.c_uint32, ctypes.POINTER(vp)]
    lib.redist_plan.restype = i32
    lib.redist_plan_destroy.argtypes = [vp]
    lib.redist_plan_destroy.restype = None
    lib.redist_execute.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, sz, vp]
    lib.redist_execute.restype = i32
    lib.redist_execute_static.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
    lib.redist_execute_static.restype = i32
    lib.redist_execute_host.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, sz, vp, sz, vp, sz, vp]
    lib.redist_execute_host.restype = i32
    for name, res in (("redist_plan_num_devices", i32), ("redist_plan_rank", i32),
                      ("redist_plan_scratch_bytes", sz), ("redist_plan_scratch_bytes_per_device", sz),
                      ("redist_plan_alignment", i32), ("redist_plan_height", i64), ("redist_plan_cost", i64),
                      ("redist_plan_num_steps", i32), ("redist_plan_num_launches", i32)):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = res
    lib.redist_plan_local_elems.argtypes = [vp, i32]
    lib.redist_plan_local_elems.restype = i64
    lib.redist_plan_staging_bytes.argtypes = [vp, i32]
    lib.redist_plan_staging_bytes.restype = sz
    lib.redist_plan_step_info.argtypes = [vp, i32, ctypes.POINTER(StepInfo)]
    lib.redist_plan_step_info.restype = i32
    lib.redist_plan_launch_info.argtypes = [vp, i32, ctypes.POINTER(LaunchInfo)]
    lib.redist_plan_launch_info.restype = i32
    lib.redist_plan_describe.argtypes = [vp, ctypes.c_char_p, sz]
    lib.redist_plan_describe.restype = sz
    lib.redist_base_offsets.argtypes = [i32, ctypes.POINTER(i64), ctypes.POINTER(_Type), ctypes.POINTER(i64),
                                        ctypes.POINTER(i64)]
    lib.redist_base_offsets.restype = i32
    lib.redist_status_string.argtypes = [i32]
    lib.redist_status_string.restype = ctypes.c_char_p
    lib.redist_last_cuda_error.argtypes = []
    lib.redist_last_cuda_error.restype = i32
    lib.redist_bulk_timeouts.argtypes = []
    lib.redist_bulk_timeouts.restype = i64
    lib.redist_bind.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, sz, ctypes.POINTER(vp)]
    lib.redist_bind.restype = i32
    lib.redist_bound_execute.argtypes = [vp, vp]
    lib.redist_bound_execute.restype = i32
    lib.redist_bound_destroy.argtypes = [vp]
    lib.redist_bound_destroy.restype = None
    lib.redist_plan_cache_stats.argtypes = [ctypes.POINTER(i64)] * 3
    lib.redist_plan_cache_stats.restype = None
    lib.redist_plan_cache_clear.argtypes = []
    lib.redist_plan_cache_clear.restype = None
    lib.redist_tuning_set.argtypes = [ctypes.c_char_p, i64]
    lib.redist_tuning_set.restype = i32
    lib.redist_tuning_get.argtypes = [ctypes.c_char_p, ctypes.POINTER(i64)]
    lib.redist_tuning_get.restype = i32
    lib.redist_tuning_reset.argtypes = []
    lib.redist_tuning_reset.restype = None
    lib.redist_plan_gpu_split.argtypes = [vp, i32, i32, ctypes.POINTER(i64)]
    lib.redist_plan_gpu_split.restype = i32
    lib.redist_debug_bounds_report.argtypes = [ctypes.POINTER(i64)]
    lib.redist_debug_bounds_report.restype = i32
    _lib = lib
    return lib


def _status_string(status: int) -> str:
    try:
        return load().redist_status_string(int(status)).decode()
    except Exception:
        return "?"


def _split(t):
    if hasattr(t, "global_shape"):
        return tuple(t.global_shape), tuple(tuple(a) for a in t.axes)
    return tuple(t[0]), tuple(tuple(a) for a in t[1])


class _CType:
    """Keeps the ctypes arrays of a redist_type alive."""

    def __init__(self, t):
        gshape, axes = _split(t)
        off, flat = [0], []
        for ax in axes:
            flat.extend(int(a) for a in ax)
            off.append(len(flat))
        self.shape = (ctypes.c_int64 * max(1, len(gshape)))(*[int(s) for s in gshape])
        self.off = (ctypes.c_int32 * len(off))(*off)
        self.flat = (ctypes.c_int32 * max(1, len(flat)))(*flat)
        self.struct = _Type(len(gshape), self.shape, self.off, self.flat)


def _mesh(mesh_shape):
    return (ctypes.c_int64 * max(1, len(mesh_shape)))(*[int(k) for k in mesh_shape])


def redist_base_offsets(mesh_shape: Sequence[int], dtype):
    """``(tile_shape, offsets)`` with ``offsets[d][k]`` the base offset of device ``d`` in dim ``k``."""
    lib = load()
    ct = _CType(dtype)
    rank = ct.struct.rank
    n = 1
    for k in mesh_shape:
        n *= int(k)
    tile = (ctypes.c_int64 * max(1, rank))()
    off = (ctypes.c_int64 * max(1, n * rank))()
    rc = lib.redist_base_offsets(len(mesh_shape), _mesh(mesh_shape), ctypes.byref(ct.struct), tile, off)
    if rc:
        raise RedistError(rc, "redist_base_offsets")
    return tuple(tile[:rank]), [tuple(off[d * rank:(d + 1) * rank]) for d in range(n)]


class Plan:
    """A synthesized redistribution (``redist_plan``).  Immutable; free with ``close()`` or GC."""

    def __init__(self, mesh_shape: Sequence[int], src, dst, elem_bytes: int, flags: int = FUSE_ADJACENT):
        lib = load()
        self._lib = lib
        self._h = ctypes.c_void_p()
        s, d = _CType(src), _CType(dst)
        rc = lib.redist_plan(len(mesh_shape), _mesh(mesh_shape), ctypes.byref(s.struct), ctypes.byref(d.struct),
                             int(elem_bytes), int(flags), ctypes.byref(self._h))
        if rc:
            self._h = None
            raise RedistError(rc, "redist_plan")
        self.mesh_shape = tuple(int(k) for k in mesh_shape)
        self.src, self.dst = _split(src), _split(dst)
        self.elem_bytes = int(elem_bytes)
        self.flags = int(flags)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.redist_plan_destroy(self._h)
            self._h = None

    __del__ = close

    # ---- queries
    @property
    def n_devices(self) -> int:
        return self._lib.redist_plan_num_devices(self._h)

    @property
    def scratch_bytes(self) -> int:
        return self._lib.redist_plan_scratch_bytes(self._h)

    @property
    def scratch_bytes_per_device(self) -> int:
        return self._lib.redist_plan_scratch_bytes_per_device(self._h)

    @property
    def alignment(self) -> int:
        return self._lib.redist_plan_alignment(self._h)

    @property
    def height(self) -> int:
        return self._lib.redist_plan_height(self._h)

    @property
    def cost(self) -> int:
        return self._lib.redist_plan_cost(self._h)

    @property
    def num_steps(self) -> int:
        return self._lib.redist_plan_num_steps(self._h)

    @property
    def num_launches(self) -> int:
        return self._lib.redist_plan_num_launches(self._h)

    def local_elems(self, which: int) -> int:
        return self._lib.redist_plan_local_elems(self._h, which)

    def staging_bytes(self, which: int) -> int:
        return self._lib.redist_plan_staging_bytes(self._h, which)

    def step_info(self, step: int) -> StepInfo:
        out = StepInfo()
        rc = self._lib.redist_plan_step_info(self._h, step, ctypes.byref(out))
        if rc:
            raise RedistError(rc, "redist_plan_step_info")
        return out

    def launch_info(self, launch: int) -> LaunchInfo:
        out = LaunchInfo()
        rc = self._lib.redist_plan_launch_info(self._h, launch, ctypes.byref(out))
        if rc:
            raise RedistError(rc, "redist_plan_launch_info")
        return out

    def step_kinds(self) -> List[str]:
        return [STEP_KINDS[self.step_info(s).kind] for s in range(self.num_steps)]

    def launch_kernels(self) -> List[str]:
        return [KERNELS[self.launch_info(s).kernel] for s in range(self.num_launches)]

    def bytes_moved(self):
        """(read, written) HBM bytes summed over the launches."""
        infos = [self.launch_info(q) for q in range(self.num_launches)]
        return sum(i.bytes_read for i in infos), sum(i.bytes_written for i in infos)

    def gpu_split(self, n_gpus: int, launch: int):
        """``redist_plan_gpu_split``: ``m[s][t]`` = bytes GPU ``s`` would read locally and write to GPU ``t``
        if the virtual devices were spread over ``n_gpus`` GPUs by a prefix of the mesh axes."""
        out = (ctypes.c_int64 * (n_gpus * n_gpus))()
        rc = self._lib.redist_plan_gpu_split(self._h, n_gpus, launch, out)
        if rc:
            raise RedistError(rc, "redist_plan_gpu_split")
        return [[int(out[s * n_gpus + t]) for t in range(n_gpus)] for s in range(n_gpus)]

    def describe(self) -> dict:
        n = self._lib.redist_plan_describe(self._h, None, 0)
        buf = ctypes.create_string_buffer(n + 1)
        self._lib.redist_plan_describe(self._h, buf, n + 1)
        return json.loads(buf.value.decode())

    def pretty(self, axis_names: Optional[Sequence[str]] = None) -> str:
        """The synthesized sequence in the paper's notation, one collective per line, over the
        prime-factor mesh (axis ``x`` of size 4 appears as ``x.0, x.1``), followed by the launches."""
        d = self.describe()
        names = list(axis_names) if axis_names else [f"a{i}" for i in range(len(d["mesh_shape"]))]
        count: dict = {}
        pnames = []
        for p in d["primes"]:
            k = count.get(p["parent"], 0)
            count[p["parent"]] = k + 1
            pnames.append(f"{names[p['parent']]}.{k}")
        multi = {par for par, c in count.items() if c > 1}
        pnames = [n if d["primes"][i]["parent"] in multi else n.split(".")[0] for i, n in enumerate(pnames)]
        sizes = [p["size"] for p in d["primes"]]

        def fmt(axes):
            parts = []
            for s_k, ax in zip(d["global_shape"], axes):
                if not ax:
                    parts.append(str(s_k))
                    continue
                k = 1
                for a in ax:
                    k *= sizes[a]
                parts.append(f"{s_k // k}{{{','.join(pnames[a] for a in ax)}}}{s_k}")
            return "[" + ", ".join(parts) + "]"

        lines = [fmt(d["src_axes"])]
        for st in d["steps"]:
            label = st["kind"]
            if st["kind"] == "alltoall":
                label += f"({st['i']},{st['j']})"
            elif st["kind"] in ("allgather", "dynslice"):
                label += f"({st['i']})"
            if st["acting"]:
                label += "{" + ",".join(pnames[a] for a in st["acting"]) + "}"
            lines.append(f"  --{label}, cost {st['cost']}--> {fmt(st['post_axes'])}")
        for L in d["launches"]:
            g = L["geometry"]
            how = "ragged rows, TMA bulk loads" if g["bulk"] == 2 else "TMA bulk copies" if g["bulk"] else ("rows", "chunks", "units", "gather walk", "zip through shared memory", "super-boxes through shared memory")[g["mode"]]
            lines.append(f"  launch {L['kernel']}: steps {L['first_step']}..{L['first_step'] + L['n_steps'] - 1}, "
                         f"{L['from']} -> {L['to']}, runs of {L['run_bytes']} B, {g['n_items']} items, {how}")
        lines.append(f"  cost {d['cost']}, height {d['height']} <= max(localsize) "
                     f"{max(d['local_src'], d['local_dst'])}, scratch per device {d['scratch_per_device']} B")
        return "\n".join(lines)

    # ---- execution
    def execute_ptrs(self, src_ptrs: Sequence[int], dst_ptrs: Sequence[int], scratch_ptr: int = 0,
                     scratch_bytes: int = 0, stream: int = 0) -> None:
        """``redist_execute`` on raw device addresses."""
        n = len(src_ptrs)
        s = (ctypes.c_void_p * n)(*src_ptrs)
        d = (ctypes.c_void_p * len(dst_ptrs))(*dst_ptrs)
        rc = self._lib.redist_execute(self._h, s, d, ctypes.c_void_p(scratch_ptr or None), scratch_bytes,
                                      ctypes.c_void_p(stream or None))
        if rc:
            raise RedistError(rc, "redist_execute")

    def bind(self, src_ptrs: Sequence[int], dst_ptrs: Sequence[int], scratch_ptr: int = 0,
             scratch_bytes: int = 0):
        """``redist_bind``: validate the buffers and prepare every launch once; the returned callable runs
        ``redist_bound_execute`` on a stream (``call(stream_ptr)``) -- the kernel launches and nothing else.
        The buffers must stay alive and in place as long as the callable is used."""
        if len(src_ptrs) != self.n_devices or len(dst_ptrs) != self.n_devices:
            raise RedistError(1, "one tile per virtual device is required")
        s = (ctypes.c_void_p * len(src_ptrs))(*src_ptrs)
        d = (ctypes.c_void_p * len(dst_ptrs))(*dst_ptrs)
        h = ctypes.c_void_p()
        rc = self._lib.redist_bind(self._h, s, d, ctypes.c_void_p(scratch_ptr or None), scratch_bytes, ctypes.byref(h))
        if rc:
            raise RedistError(rc, "redist_bind")
        return _Bound(self, h)

    def _check_tiles(self, src_shards, dst_shards, cuda: bool = True) -> None:
        """What the C entry points cannot know: one tile per virtual device, each a contiguous tensor in
        the right memory holding exactly localsize*elem_bytes bytes."""
        if len(src_shards) != self.n_devices or len(dst_shards) != self.n_devices:
            raise RedistError(1, "one tile per virtual device is required")
        sb, db = self.local_elems(0) * self.elem_bytes, self.local_elems(1) * self.elem_bytes
        for t, need in [(x, sb) for x in src_shards] + [(x, db) for x in dst_shards]:
            if t.is_cuda != cuda or not t.is_contiguous() or t.numel() * t.element_size() != need:
                raise RedistError(1, "tiles must be contiguous %s tensors of the local size" % ("CUDA" if cuda else "host"))

    def execute(self, src_shards, dst_shards, scratch=None, stream=None) -> None:
        """``redist_execute`` on lists of CUDA tensors (one per virtual device), asynchronous."""
        import torch

        self._check_tiles(src_shards, dst_shards)
        if stream is None:
            stream = torch.cuda.current_stream()
        sp = scratch.data_ptr() if scratch is not None else 0
        sn = scratch.numel() * scratch.element_size() if scratch is not None else 0
        self.execute_ptrs([t.data_ptr() for t in src_shards], [t.data_ptr() for t in dst_shards], sp, sn,
                          stream.cuda_stream)

    def execute_static(self, src_shards, dst_shards, stream=None) -> None:
        """``redist_execute_static``: like ``execute`` but the scratch of an unfused plan comes from
        the fixed array built into the library, for callers that cannot allocate device memory
        (plans needing more than ``STATIC_SCRATCH_BYTES`` are refused)."""
        import torch

        self._check_tiles(src_shards, dst_shards)
        if stream is None:
            stream = torch.cuda.current_stream()
        n = self.n_devices
        s = (ctypes.c_void_p * n)(*[t.data_ptr() for t in src_shards])
        d = (ctypes.c_void_p * n)(*[t.data_ptr() for t in dst_shards])
        rc = self._lib.redist_execute_static(self._h, s, d, ctypes.c_void_p(stream.cuda_stream or None))
        if rc:
            raise RedistError(rc, "redist_execute_static")

    def execute_host(self, src_host, dst_host, dev_src, dev_dst, scratch=None, stream=None) -> None:
        """``redist_execute_host``: host tiles in, host tiles out, staged through ``dev_src``/``dev_dst``."""
        import torch

        self._check_tiles(src_host, dst_host, cuda=False)
        if stream is None:
            stream = torch.cuda.current_stream()
        n = self.n_devices
        s = (ctypes.c_void_p * n)(*[t.data_ptr() for t in src_host])
        d = (ctypes.c_void_p * n)(*[t.data_ptr() for t in dst_host])
        sp = scratch.data_ptr() if scratch is not None else 0
        sn = scratch.numel() * scratch.element_size() if scratch is not None else 0
        rc = self._lib.redist_execute_host(self._h, s, d, ctypes.c_void_p(dev_src.data_ptr()),
                                           dev_src.numel() * dev_src.element_size(),
                                           ctypes.c_void_p(dev_dst.data_ptr()),
                                           dev_dst.numel() * dev_dst.element_size(), ctypes.c_void_p(sp or None), sn,
                                           ctypes.c_void_p(stream.cuda_stream or None))
        if rc:
            raise RedistError(rc, "redist_execute_host")

    def alloc_scratch(self, device="cuda"):
        import torch

        n = self.scratch_bytes
        return torch.empty(n, dtype=torch.uint8, device=device) if n else None


class _Bound:
    """A plan bound to one set of buffers (``redist_bind``); calling it launches the kernels on a stream."""

    def __init__(self, plan: Plan, handle):
        self._plan, self._h = plan, handle          # the plan object stays alive with its bound form
        self._fn, self._destroy = plan._lib.redist_bound_execute, plan._lib.redist_bound_destroy

    def __call__(self, stream_ptr: int = 0) -> None:
        rc = self._fn(self._h, stream_ptr or None)      # argtypes convert the integer; nothing is built per call
        if rc:
            raise RedistError(rc, "redist_bound_execute")

    def close(self):
        if getattr(self, "_h", None):
            self._destroy(self._h)
            self._h = None

    __del__ = close


def tuning_set(name: str, value: int) -> None:
    """``redist_tuning_set``: change a tuning value for the plans created from now on."""
    rc = load().redist_tuning_set(name.encode(), int(value))
    if rc:
        raise RedistError(rc, f"redist_tuning_set({name!r}, {value})")


def tuning_get(name: str) -> int:
    out = ctypes.c_int64()
    rc = load().redist_tuning_get(name.encode(), ctypes.byref(out))
    if rc:
        raise RedistError(rc, f"redist_tuning_get({name!r})")
    return int(out.value)


def tuning_reset() -> None:
    load().redist_tuning_reset()


@contextlib.contextmanager
def tuning(**values):
    """``with tuning(bulk=0, gather=0): plan = Plan(...)`` -- plans created inside get these values."""
    try:
        for k, v in values.items():
            tuning_set(k, v)
        yield
    finally:
        tuning_reset()


def plan_cache_stats():
    """``(hits, misses, entries)`` of the plan cache."""
    h, m, e = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    load().redist_plan_cache_stats(ctypes.byref(h), ctypes.byref(m), ctypes.byref(e))
    return int(h.value), int(m.value), int(e.value)


def plan_cache_clear() -> None:
    load().redist_plan_cache_clear()


def debug_bounds_report():
    """Checked build only: ``(violations, line, block, side, distance)`` since the last call."""
    out = (ctypes.c_int64 * 5)()
    rc = load().redist_debug_bounds_report(out)
    if rc:
        raise RedistError(rc, "redist_debug_bounds_report")
    return tuple(int(v) for v in out)


def redist_bulk_timeouts() -> int:
    """Work items whose bounded bulk-copy wait ran out on the current device (0 in a healthy run)."""
    return int(load().redist_bulk_timeouts())


def redist_plan(mesh_shape, src, dst, elem_bytes: int, flags: int = FUSE_ADJACENT) -> Plan:
    return Plan(mesh_shape, src, dst, elem_bytes, flags)


def redist_execute(plan: Plan, src_shards, dst_shards, scratch=None, stream=None) -> None:
    plan.execute(src_shards, dst_shards, scratch, stream)


def shard_global(G, mesh_shape, dtype) -> list:
    """Cut a global tensor ``G`` (any device) into the tiles the type prescribes, one contiguous
    tensor per virtual device, using the library's base offset map."""
    tile, offs = redist_base_offsets(mesh_shape, dtype)
    out = []
    for off in offs:
        t = G
        for k, (o, c) in enumerate(zip(off, tile)):
            t = t.narrow(k, int(o), int(c))
        out.append(t.contiguous())
    return out
