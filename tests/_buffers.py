"""Device buffers for the GPU tests, carved out of ONE allocation so that stray accesses show.

The boundary promises no more than this: every tile and the scratch buffer start on a multiple of
``redist_plan_alignment`` (16) bytes -- 256 for the scratch -- and hold exactly
``localsize * elem_bytes`` bytes.  Allocators hand out far more (512-byte alignment, padded sizes),
which would hide a kernel that leans on it.  So the tests place everything themselves:

    [band] src tile 0 | src tile 1 | ... (packed, each start rounded up to 16 only) [band]
    [band] dst tile 0 [band] dst tile 1 [band] ...        (starts = 16 mod 32: 16-byte aligned, not more)
    [band] scratch [band]                                   (256-aligned, as the boundary requires)

The whole buffer is filled with ``CANARY``; destination tiles then get ``0xEE`` and the scratch ``0xDD`` so
that missing writes show too.  ``Carved.check()`` asserts that every band -- and the gaps between the
packed source tiles -- still hold the canary and that the source tiles are unchanged: a store outside a
destination tile cannot go unnoticed, and cannot land anywhere but in the test's own buffer.
"""
from __future__ import annotations

import numpy as np

CANARY = 0xA5
BAND = 256


def _up(v: int, a: int) -> int:
    return (v + a - 1) // a * a


class Carved:
    def __init__(self, torch, src_tiles, n_dst, dst_bytes, scratch_bytes, keep_sources_below=64 << 20):
        self.torch = torch
        src_flat = [np.ascontiguousarray(t).reshape(-1).view(np.uint8) for t in src_tiles]
        pos = BAND + 16
        self.src_at = []
        for t in src_flat:
            pos = _up(pos, 16)
            self.src_at.append((pos, t.size))
            pos += t.size
        pos = _up(pos, 32) + BAND
        self.dst_at = []
        for _ in range(n_dst):
            pos = _up(pos, 32) + 16                       # 16-byte aligned and no better
            self.dst_at.append((pos, dst_bytes))
            pos += dst_bytes + BAND
        self.scratch_at = None
        if scratch_bytes:
            pos = _up(pos, 256)
            self.scratch_at = (pos, scratch_bytes)
            pos += scratch_bytes + BAND
        self.total = _up(pos, 256)
        self.buf = torch.full((self.total,), CANARY, dtype=torch.uint8, device="cuda")
        assert self.buf.data_ptr() % 256 == 0
        self.src = []
        for (at, n), t in zip(self.src_at, src_flat):
            view = self.buf[at:at + n]
            view.copy_(torch.from_numpy(t))
            self.src.append(view)
        self.dst = []
        for at, n in self.dst_at:
            view = self.buf[at:at + n]
            view.fill_(0xEE)
            self.dst.append(view)
        self.scratch = None
        if self.scratch_at:
            at, n = self.scratch_at
            self.scratch = self.buf[at:at + n]
            self.scratch.fill_(0xDD)
        self._src_copy = None
        if sum(t.size for t in src_flat) <= keep_sources_below:
            self._src_copy = [t.copy() for t in src_flat]

    def check(self, what=""):
        """Every byte outside the tiles and the scratch still holds the canary; sources are unchanged."""
        torch = self.torch
        torch.cuda.synchronize()
        used = sorted(self.src_at + self.dst_at + ([self.scratch_at] if self.scratch_at else []))
        pos = 0
        for at, n in used + [(self.total, 0)]:
            if at > pos:
                gap = self.buf[pos:at]
                if not bool((gap == CANARY).all()):
                    bad = int(torch.nonzero(gap != CANARY)[0]) + pos
                    near = min(used, key=lambda u: min(abs(bad - u[0]), abs(bad - (u[0] + u[1]))))
                    raise AssertionError(f"{what}: guard byte {bad} was overwritten (nearest region starts at "
                                         f"{near[0]}, {near[1]} bytes long)")
            pos = max(pos, at + n)
        if self._src_copy is not None:
            for d, (view, ref) in enumerate(zip(self.src, self._src_copy)):
                if not np.array_equal(view.cpu().numpy(), ref):
                    raise AssertionError(f"{what}: source tile {d} was modified")

    def results(self):
        return [t.cpu().numpy() for t in self.dst]
