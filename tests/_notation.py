"""Parser for the paper's type notation and for the sequence fixtures under tests/golden/."""
from __future__ import annotations

import os
import re
from typing import Dict, List, Tuple

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

_DIM = re.compile(r"^\s*(\d+)\s*(?:\{([^}]*)\}\s*(\d+))?\s*$")


def parse_mesh(text: str) -> Tuple[List[str], Tuple[int, ...]]:
    names, sizes = [], []
    for item in text.split():
        n, k = item.split(":")
        names.append(n)
        sizes.append(int(k))
    return names, tuple(sizes)


def parse_type(text: str, names: List[str], mesh: Tuple[int, ...]):
    """``[32{x,y}512, 128]`` -> (global_shape, axes, printed_tile_sizes)."""
    body = text.strip()
    assert body[0] == "[" and body[-1] == "]", text
    dims, depth, cur = [], 0, ""
    for ch in body[1:-1]:
        if ch == "{":
            depth += 1
        if ch == "}":
            depth -= 1
        if ch == "," and depth == 0:
            dims.append(cur)
            cur = ""
        else:
            cur += ch
    dims.append(cur)
    gshape, axes, tiles = [], [], []
    for d in dims:
        m = _DIM.match(d)
        assert m, d
        if m.group(2) is None:
            gshape.append(int(m.group(1)))
            axes.append(())
            tiles.append(int(m.group(1)))
        else:
            tiles.append(int(m.group(1)))
            gshape.append(int(m.group(3)))
            axes.append(tuple(names.index(a.strip()) for a in m.group(2).split(",") if a.strip()))
    return tuple(gshape), tuple(axes), tuple(tiles)


def load_sequences(fname: str):
    """Yield dicts {mesh, names, types: [(gshape, axes, tiles)], steps: [tokens], costs, total}."""
    names, mesh = None, None
    seqs, cur = [], None
    with open(os.path.join(GOLDEN, fname)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(" ")
            if key == "mesh":
                names, mesh = parse_mesh(rest)
            elif key == "type":
                if cur is None:
                    cur = {"mesh": mesh, "names": names, "types": [], "steps": [], "costs": {}, "total": None}
                cur["types"].append(parse_type(rest, names, mesh))
            elif key == "step":
                cur["steps"].append(rest.split())
            elif key == "cost":
                cur["costs"][len(cur["steps"]) - 1] = int(rest)
            elif key == "total":
                cur["total"] = int(rest)
            elif key == "end":
                seqs.append(cur)
                cur = None
            else:
                raise ValueError(line)
    return seqs


def load_offset_table(fname: str):
    names, mesh, typ, rows = None, None, None, []
    with open(os.path.join(GOLDEN, fname)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(" ")
            if key == "mesh":
                names, mesh = parse_mesh(rest)
            elif key == "type":
                typ = parse_type(rest, names, mesh)
            else:
                rows.append(tuple(int(v) for v in line.split()))
    return names, mesh, typ, rows
