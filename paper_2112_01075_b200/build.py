"""Build step: compile the CUDA library for sm_100a with nvcc, in-tree.

``python -m paper_2112_01075_b200.build`` (or ``build()``) produces, next to this file,

* ``libredist_b200.so`` -- the library, and
* ``libredist_b200_bounds.so`` -- the same sources with the kernels compiled with ``-DREDIST_BOUNDS``:
  every global and shared-memory access is tested against the launch's tiles and skipped if it fails,
  the first failure is recorded (``redist_debug_bounds_report``).  Only the tests load it.

nvcc cross-compiles without a GPU.  The CUDA runtime is linked statically, so the libraries load (and
their host-only entry points work) on a machine without a driver.  Sources compile in parallel into
``_obj/`` -- the kernels as three parts (``-DREDIST_PART=1|2|3``), which brings a full build from over three
minutes to under two on eight cores; only what changed is recompiled.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_obj")
LIB = os.path.join(HERE, "libredist_b200.so")
LIB_BOUNDS = os.path.join(HERE, "libredist_b200_bounds.so")
SOURCES = ["api.cu", "kernels.cu", "static_scratch.cu", "planner.cpp", "descriptor.cpp", "describe.cpp", "multi_gpu.cpp"]
HEADERS = ["plan.hpp", "copy_params.h", "kernels.h"]
CHECKED = ["kernels.cu"]          # sources that differ in the checked build
# (source, object name, defines): the kernels compile as three parts side by side (see REDIST_PART in kernels.cu)
UNITS = [(s, os.path.splitext(s)[0], []) for s in SOURCES if s != "kernels.cu"] + \
        [("kernels.cu", f"kernels_p{k}", [f"REDIST_PART={k}"]) for k in (1, 2, 3)]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _deps():
    return [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "redist.h"),
                                                                   os.path.abspath(__file__)]


def needs_build() -> bool:
    newest = max(os.path.getmtime(d) for d in _deps())
    return any(not os.path.exists(lib) or os.path.getmtime(lib) < newest for lib in (LIB, LIB_BOUNDS))


def _compile(src: str, obj: str, defines, verbose: bool) -> str:
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC,-Wall,-Wno-unknown-pragmas", "-c",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", obj] + [f"-D{d}" for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    res = subprocess.run(cmd + [os.path.join(CSRC, src)], capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError(f"nvcc failed on {src}")
    return res.stdout + res.stderr


def _link(objs, lib: str) -> None:
    tmp = lib + f".tmp{os.getpid()}"
    res = subprocess.run([_nvcc(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                          "-o", tmp] + objs, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    newest_header = max(os.path.getmtime(d) for d in _deps() if not d.endswith((".cu", ".cpp")))
    jobs = []
    for src, name, unit_defines in UNITS:
        variants = [("", [])] + ([("_bounds", ["REDIST_BOUNDS"])] if src in CHECKED else [])
        for suffix, defines in variants:
            obj = os.path.join(OBJ, name + suffix + ".o")
            stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(
                newest_header, os.path.getmtime(os.path.join(CSRC, src)))
            jobs.append((src, obj, unit_defines + defines, stale))
    jobs.sort(key=lambda j: not j[0].startswith("kernels"))      # the long compiles first
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        logs = list(pool.map(lambda j: _compile(j[0], j[1], j[2], verbose) if j[3] else "", jobs))
    if verbose:
        sys.stderr.write("".join(logs))
    plain = [os.path.join(OBJ, name + ".o") for _, name, _ in UNITS]
    checked = [os.path.join(OBJ, name + ("_bounds" if src in CHECKED else "") + ".o") for src, name, _ in UNITS]
    _link(plain, LIB)
    _link(checked, LIB_BOUNDS)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
