"""Test-side interpreter of the launch descriptors a plan reports (``redist_plan_describe``).

It replays, in numpy on host byte arrays, exactly the index arithmetic the descriptor encodes
(boxes -> tiles and offsets, row digits, contiguous runs, fan-out), so descriptor construction can
be checked against the oracle without a GPU.  It is not a product path.
"""
from __future__ import annotations

import numpy as np


def _prod(xs):
    n = 1
    for x in xs:
        n *= int(x)
    return n


def run_launch(L: dict, src_bufs, dst_bufs):
    """src_bufs / dst_bufs: callables device -> 1-D uint8 array (device -1 = the shared buffer)."""
    G = L["geometry"]
    fan = G["fanout"]
    run = G["run_bytes"]
    assert run == L["run_bytes"] and run > 0
    unit_n = G["unit_n"]
    n_boxes = _prod(unit_n)
    rows = _prod(G["row_n"])
    tab_rows = G["rows"]
    assert tab_rows * G["tab_inner"] == rows
    inner, span, mul = G["inner_n"], G["inner_span"], G["inner_mul"]
    assert inner * mul == span
    assert G["n_items"] == n_boxes * G["items_per_box"] * inner
    unit = G["unit_bytes"]
    assert unit in (1, 2, 4, 8, 16) and (G["aligned"] == 1) == (unit == 16) and run % unit == 0
    max_chunks = run // 16
    if G["mode"] == 3:      # gather walk: target stretches of a table row in whole chunks
        u = G["inner_digit"]
        m1, m2 = G["unit_m1"][u], G["unit_m2"][u]
        long_dst = G["gl_long_dst"] == 1
        assert unit >= 4 and run < 256 and inner == 1 and mul == span == max(m1, m2) == G["gl_m"] and min(m1, m2) == 1
        assert (m2 > 1) == long_dst and G["units_per_run"] * unit == run
        assert (G["unit_b2"][u] if long_dst else G["unit_b1"][u]) == run
        lv = G["gl_levels"]
        assert 0 <= lv <= 2 and (long_dst or lv >= 1) and G["n_row_tab"] == len(G["row_n"]) - lv
        S = mul * run if long_dst else run
        for l in range(lv):
            q = len(G["row_n"]) - 1 - l
            assert G["row_b2"][q] == S and G["gl_n"][l] == G["row_n"][q] and G["gl_b1"][l] == G["row_b1"][q]
            S *= G["row_n"][q]
        assert S == G["gl_stretch"] and 32 <= S < 2 ** 31 and G["tab_inner"] == _prod(G["row_n"][len(G["row_n"]) - lv:])
        assert 1 <= G["rows_per_item"] <= 1024 and G["col_blocks"] * G["per_block"] >= S // 16
        assert G["items_per_box"] == -(-tab_rows // G["rows_per_item"]) * G["col_blocks"]
    elif G["mode"] == 4:    # zip: both sides contiguous across the innermost row digit, staged by bulk copies
        u = G["inner_digit"]
        m1, m2 = G["unit_m1"][u], G["unit_m2"][u]
        long_dst = G["gl_long_dst"] == 1
        m = max(m1, m2)
        assert unit >= 4 and run < 2048 and inner == 1 and mul == span == m == G["gl_m"] and min(m1, m2) == 1 and m <= 16
        assert (m2 > 1) == long_dst and G["units_per_run"] * unit == run
        assert (G["unit_b2"][u] if long_dst else G["unit_b1"][u]) == run
        n = G["row_n"][-1]
        assert G["tab_inner"] == n and G["n_row_tab"] == len(G["row_n"]) - 1
        assert G["row_b1"][-1] == (run if long_dst else m * run) and G["row_b2"][-1] == (m * run if long_dst else run)
        rpb, rpi, nseg = G["per_block"], G["rows_per_item"], (m if long_dst else 1)
        assert 1 <= rpb <= n and G["col_blocks"] == -(-n // rpb) and 1 <= rpi and rpi * nseg <= 256
        seg = rpb * (run if long_dst else m * run)
        assert G["zip_seg_pitch"] % 16 == 0 and G["zip_seg_pitch"] >= seg + 30
        assert G["stage_pitch"] == G["zip_seg_pitch"] * nseg and G["stage_pitch"] * rpi <= 38 * 1024
        if G["zip_period"]:
            import math
            lb = m * run if long_dst else run
            assert G["zip_period"] == lb // math.gcd(16, lb) and G["zip_period_rows"] == 16 // math.gcd(16, lb)
            assert G["zip_period"] * (m if not long_dst and run <= 16 else 1) <= 255 and rpb * lb // 16 >= 2 * G["zip_period"]
            assert G["zip_width"] % G["zip_period"] == 0 and G["zip_period"] <= G["zip_width"] <= 256
        if G["zip_cpr"]:
            assert not G["zip_period"] and not G["zip_lut_units"] and run >= 32 and unit < 16
            assert G["zip_cpr"] == -(-run // 16) and G["zip_slots"] == rpb * (m if long_dst else 1) * G["zip_cpr"] >= 256
        else:
            assert G["zip_slots"] >= rpb * (m * run if long_dst else run) // 16
        if G["zip_lut_units"]:
            assert not G["zip_period"] and G["zip_lut_units"] == rpb * (m * run if long_dst else run) // unit <= 2048
            assert G["stage_pitch"] * rpi + 4 * G["zip_lut_units"] <= 42 * 1024
        assert G["items_per_box"] == -(-tab_rows // rpi) * G["col_blocks"]
    elif G["mode"] == 0:    # rows: aligned runs of at most 256 chunks
        assert unit == 16 and max_chunks <= 256 and G["lanes"] == max_chunks
        assert G["rows_per_pass"] == 256 // G["lanes"] and G["rows_per_item"] % G["rows_per_pass"] == 0
        assert G["items_per_box"] * G["rows_per_item"] >= rows and tab_rows == rows
    else:                   # flat walk over (row, chunk) or (row, unit piece)
        per_row = max_chunks if G["mode"] == 1 else G["tab_inner"] * (run // unit)
        assert (G["mode"] == 1 and run >= 256) or (G["mode"] == 2 and run < 256 and unit < 16)
        assert G["mode"] == 2 or G["tab_inner"] == 1
        assert G["tab_inner"] == 1 or (G["tab_inner"] == G["row_n"][-1] and G["n_row_tab"] == len(G["row_n"]) - 1)
        assert 1 <= G["rows_per_item"] <= 1024
        assert G["col_blocks"] * G["per_block"] >= per_row
        assert G["items_per_box"] == -(-tab_rows // G["rows_per_item"]) * G["col_blocks"]
    # row offsets (mixed radix, last digit fastest)
    r = np.arange(rows, dtype=np.int64)
    s1 = np.zeros(rows, dtype=np.int64)
    s2 = np.zeros(rows, dtype=np.int64)
    for q in range(len(G["row_n"]) - 1, -1, -1):
        dg = r % G["row_n"][q]
        r = r // G["row_n"][q]
        s1 += dg * G["row_b1"][q]
        s2 += dg * G["row_b2"][q]
    col = np.arange(run, dtype=np.int64)
    written = {}
    for boxp in range(n_boxes * span):
        box, piece = divmod(boxp, span)          # a gather item covers `mul` consecutive pieces
        rem, t1, t2, o1, o2 = box, 0, 0, 0, 0
        for u in range(len(unit_n) - 1, -1, -1):
            q = rem % unit_n[u]
            rem //= unit_n[u]
            if u == G["inner_digit"]:
                q = q * span + piece
            a1, b1 = divmod(q, G["unit_m1"][u])
            a2, b2 = divmod(q, G["unit_m2"][u])
            t1 += a1 * G["unit_ts1"][u]
            t2 += a2 * G["unit_ts2"][u]
            o1 += b1 * G["unit_b1"][u]
            o2 += b2 * G["unit_b2"][u]
        assert o1 % unit == 0 and o2 % unit == 0 and np.all(s1 % unit == 0) and np.all(s2 % unit == 0)
        src = src_bufs(L["src_holder"][t1])
        data = src[(o1 + s1)[:, None] + col[None, :]]
        for f in range(fan):
            dev = L["dst_devs"][t2 * fan + f]
            dst = dst_bufs(dev)
            idx = (o2 + s2)[:, None] + col[None, :]
            dst[idx] = data
            w = written.setdefault(dev, np.zeros(dst.shape[0], dtype=np.int32))
            np.add.at(w, idx.reshape(-1), 1)
    return written


def run_plan(desc: dict, src_tiles):
    """Execute all launches; returns (dst tiles as flat uint8 arrays, per-launch write-count maps)."""
    n = desc["n_devices"]
    e = desc["elem_bytes"]
    src = [np.ascontiguousarray(t).reshape(-1).view(np.uint8) for t in src_tiles]
    dst = [np.full(desc["local_dst"] * e, 0xEE, dtype=np.uint8) for _ in range(n)]
    slot = desc["slot_bytes"]
    scratch = np.full(max(1, desc["scratch_bytes"]), 0xDD, dtype=np.uint8)

    def buf(kind):
        def get(dev):
            if kind == "src":
                return src[dev]
            if kind == "dst":
                return dst[dev]
            if kind == "scratch0":
                return scratch[dev * slot:(dev + 1) * slot]
            if kind == "scratch1":
                return scratch[(n + dev) * slot:(n + dev + 1) * slot]
            return scratch
        return get

    counts = []
    for L in desc["launches"]:
        counts.append(run_launch(L, buf(L["from"]), buf(L["to"])))
    return dst, counts
