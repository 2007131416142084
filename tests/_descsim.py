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
    unit_mul = G["unit_mul"]
    assert all(m >= 1 for m in unit_mul) and (G["mode"] == 5 or all(m == 1 for m in unit_mul))
    n_boxes = _prod(unit_n)
    rows = _prod(G["row_n"])
    tab_rows = G["rows"]
    assert tab_rows * G["tab_inner"] == rows or G["mode"] == 5
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
        assert run < 256 and inner == 1 and mul == span == max(m1, m2) == G["gl_m"] and min(m1, m2) == 1
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
        assert run < 2048 and inner == 1 and mul == span == m == G["gl_m"] and min(m1, m2) == 1 and m <= 64
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
    elif G["mode"] == 5:    # super-boxes: lcm(source tile, target tile) in the inner dimensions, staged by bulk copies
        nb = G["bx_n"]
        rpi = G["rows_per_item"]
        assert 1 <= nb <= 3 and inner == span == mul == 1 and 1 <= rpi <= 32
        c1, c2, n1, n2 = G["bx_c1"], G["bx_c2"], G["bx_n1"], G["bx_n2"]
        trail = G["bx_trail"] * unit
        for q in range(nb):
            assert c1[q] % c2[q] == 0 or c2[q] % c1[q] == 0          # separable places
            assert c1[q] * n1[q] == c2[q] * n2[q] == max(c1[q], c2[q])
            assert G["bx_st1"][q] == trail * _prod(c1[q + 1:]) and G["bx_seg"][q] == _prod(n1[q + 1:])
        assert G["bx_s1"] == trail * _prod(c1) and G["bx_s2"] == trail * _prod(c2)
        assert G["bx_nseg"] == _prod(n1) and G["bx_nrng"] == _prod(n2) and rpi * max(G["bx_nseg"], G["bx_nrng"]) <= 256
        assert run == trail and min(c1[-1], c2[-1]) == 1     # the last inner dimension counts runs
        nK, cnt = G["tab_inner"], G["per_block"]
        n_out = G["n_row_tab"]
        assert G["row_n"][n_out] == nK and 1 <= cnt <= nK and G["col_blocks"] == -(-nK // cnt)
        assert tab_rows == _prod(G["row_n"][:n_out]) and rows == tab_rows * nK * _prod(G["row_n"][n_out + 1:])
        if nK > 1:
            assert G["row_b1"][n_out] == G["bx_s1"] and G["row_b2"][n_out] == G["bx_s2"]   # rows of K are contiguous
        assert G["zip_seg_pitch"] % 16 == 0 and G["zip_seg_pitch"] >= cnt * G["bx_s1"] + 30
        assert G["stage_pitch"] == G["zip_seg_pitch"] * G["bx_nseg"] and G["stage_pitch"] * rpi <= 38 * 1024
        assert G["zip_lut_units"] * unit == G["bx_s2"] and G["zip_lut_units"] <= 4096
        assert G["zip_slots"] >= cnt * G["bx_s2"] // 16 + 1 and G["zip_width"] in (1, 2, 4, 8, 16, 32, 64, 128, 256)
        assert G["items_per_box"] == -(-tab_rows // rpi) * G["col_blocks"]
        # the digits of the inner dimensions count super-boxes: unit_mul boxes of the gcd size each
        assert _prod(unit_mul) >= 1
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
    for boxp in range(n_boxes * span * _prod(unit_mul)):
        box, piece = divmod(boxp, span)          # a gather item covers `mul` consecutive pieces
        rem, t1, t2, o1, o2 = box, 0, 0, 0, 0
        for u in range(len(unit_n) - 1, -1, -1):
            # (a super-box digit counts unit_mul boxes: enumerate them all)
            q = rem % (unit_n[u] * unit_mul[u])
            rem //= unit_n[u] * unit_mul[u]
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
    if G["mode"] == 5:
        check_box_items(L, src_bufs, dst_bufs)
    return written


def check_box_items(L: dict, src_bufs, dst_bufs):
    """The super-box kernel works from its own description of an item (segments, ranges, the table of unit
    places and the corners of the target tiles).  Replay that arithmetic item by item, as the kernel does
    it, and require that it reproduces what the box-by-box interpretation above has just written."""
    G = L["geometry"]
    fan, unit = G["fanout"], G["unit_bytes"]
    nb = G["bx_n"]
    c1, c2, n1, n2 = G["bx_c1"], G["bx_c2"], G["bx_n1"], G["bx_n2"]
    s1, s2, pitch = G["bx_s1"], G["bx_s2"], G["zip_seg_pitch"]
    n_out = G["n_row_tab"]
    place = np.zeros(G["zip_lut_units"], dtype=np.int64)
    for p in range(G["zip_lut_units"]):
        rest, off = divmod(p, G["bx_trail"])
        off *= unit
        for q in range(nb - 1, -1, -1):
            rest, i = divmod(rest, c2[q])
            hi, lo = divmod(i, c1[q])
            off += hi * G["bx_seg"][q] * pitch + lo * G["bx_st1"][q]
        assert off < 65536
        place[p] = off
    for item in range(G["n_items"]):
        rest, part = divmod(item, G["items_per_box"])          # inner_n = fast_boxes = 1 in this mode
        t1 = t2 = o1 = o2 = 0
        for u in range(len(G["unit_n"]) - 1, -1, -1):
            rest, q = divmod(rest, G["unit_n"][u])
            q *= G["unit_mul"][u]
            a1, b1 = divmod(q, G["unit_m1"][u])
            a2, b2 = divmod(q, G["unit_m2"][u])
            t1 += a1 * G["unit_ts1"][u]
            t2 += a2 * G["unit_ts2"][u]
            o1 += b1 * G["unit_b1"][u]
            o2 += b2 * G["unit_b2"][u]
        group, cb = divmod(part, G["col_blocks"])
        a = cb * G["per_block"]
        cnt = min(G["per_block"], G["tab_inner"] - a)
        row0 = group * G["rows_per_item"]
        nr = min(G["rows_per_item"], G["rows"] - row0)
        stage = np.zeros(G["stage_pitch"] * G["rows_per_item"] + 64, dtype=np.uint8)
        offs = []
        for r in range(nr):
            r1 = r2 = 0
            rem = row0 + r
            for q in range(n_out - 1, -1, -1):
                rem, dg = divmod(rem, G["row_n"][q])
                r1 += dg * G["row_b1"][q]
                r2 += dg * G["row_b2"][q]
            so, d0 = o1 + r1 + a * s1, o2 + r2 + a * s2
            offs.append((so % 16, d0))
            for t in range(G["bx_nseg"]):
                rem, tile = t, t1
                for q in range(nb - 1, -1, -1):
                    rem, d = divmod(rem, n1[q])
                    tile += d * G["bx_ts1"][q]
                src = src_bufs(L["src_holder"][tile])
                assert so + cnt * s1 <= src.shape[0]
                at = (r * G["bx_nseg"] + t) * pitch + so % 16
                stage[at:at + cnt * s1] = src[so:so + cnt * s1]
        for r in range(nr):
            mis, d0 = offs[r]
            for t in range(G["bx_nrng"]):
                rem, tile, base = t, t2, r * G["stage_pitch"] + mis
                for q in range(nb - 1, -1, -1):
                    rem, d = divmod(rem, n2[q])
                    tile += d * G["bx_ts2"][q]
                    hi, lo = divmod(d * c2[q], c1[q])
                    base += hi * G["bx_seg"][q] * pitch + lo * G["bx_st1"][q]
                x = np.arange(0, cnt * s2, unit, dtype=np.int64)
                at = base + (x // s2) * s1 + place[(x % s2) // unit]
                got = stage[at[:, None] + np.arange(unit)[None, :]].reshape(-1)
                for f in range(fan):
                    dst = dst_bufs(L["dst_devs"][tile * fan + f])
                    assert d0 + cnt * s2 <= dst.shape[0]
                    assert np.array_equal(dst[d0:d0 + cnt * s2], got), (item, r, t, f)


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
