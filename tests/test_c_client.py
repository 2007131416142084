"""The boundary used from plain C: ``tests/c_client.c`` is compiled with gcc as C99 against ``include/redist.h``
and linked with the in-tree library, without Python between the caller and the library.

* CPU: the client compiles and links (the header really is C, every entry point it calls is exported).
* GPU: the client runs the smallest benchmark configuration forward and back on tiles cut by the oracle; the
  forward result it writes is compared with the oracle's tiles byte for byte, the way back must return the
  source tiles (checked by the client), and its timing line is reported: host time per ``redist_bound_execute``
  and per ``redist_execute`` call over 10 000 calls each, device time of forward + back.
"""
import json
import os
import subprocess

import numpy as np
import pytest

import oracle
from paper_2112_01075_b200 import api, workloads as wl
from _plancheck import types_of

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
PKG = os.path.join(ROOT, "paper_2112_01075_b200")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_client(out_dir):
    api.load()                                                  # builds the library if it is missing
    exe = os.path.join(str(out_dir), "c_client")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-O2", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(CUDA, "include"), os.path.join(HERE, "c_client.c"), "-o", exe,
           "-L", PKG, "-l:libredist_b200.so", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + PKG, "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr[-3000:]
    return exe


def test_c_client_compiles_and_links_as_c99(tmp_path):
    if not os.path.exists(os.path.join(CUDA, "include", "cuda_runtime_api.h")):
        pytest.skip("no CUDA toolkit headers")
    exe = build_client(tmp_path)
    res = subprocess.run([exe], capture_output=True, text=True)    # no arguments: usage, nothing touches a GPU
    assert res.returncode == 2 and "usage" in res.stderr


@pytest.mark.gpu
def test_c_client_matches_the_oracle_and_reports_host_time(tmp_path, record_property):
    w = wl.config1()
    src, dst = types_of(w)
    G = wl.global_array_bytes(w.src.global_shape, w.elem_bytes, w.fill, w.seed)
    tiles = oracle.reslice(w.mesh_shape, src, G)
    want = oracle.reslice(w.mesh_shape, dst, G)
    fin, fout = tmp_path / "in.bin", tmp_path / "out.bin"
    fin.write_bytes(b"".join(np.ascontiguousarray(t).tobytes() for t in tiles))
    exe = build_client(tmp_path)
    res = subprocess.run([exe, str(fin), str(fout)], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout[-1000:] + res.stderr[-2000:]
    got = np.frombuffer(fout.read_bytes(), dtype=np.uint8).reshape(len(want), -1)
    for d, t in enumerate(want):
        assert np.array_equal(got[d], np.ascontiguousarray(t).reshape(-1).view(np.uint8)), f"tile {d}"
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["bulk_timeouts"] == 0 and line["calls"] == 10000
    # reported, with a loose ceiling only (a launch costs the CUDA runtime about 2 us on its own)
    assert 0 < line["host_us_per_bound_call"] < 50 and 0 < line["host_us_per_execute_call"] < 50
    assert line["host_us_per_bound_call"] <= line["host_us_per_execute_call"] * 1.25
    for k, v in line.items():
        record_property(k, v)
    print("c client:", json.dumps(line))
