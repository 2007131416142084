// sm_100a copy kernels of the executor.
//
// Every collective of a redistribution moves bytes and never interprets them (Section 4.2: the
// meaning of a collective is how it changes the placement of tiles).  On one GPU, with every
// virtual device's tile in its own buffer, a collective -- or a fused run of them -- is therefore a
// strided gather/scatter between two layouts of the same global array, described by CopyGeometry
// (copy_params.h).  The work is bound by HBM bandwidth: every source byte is read once and written
// once per target replica from registers (allgather stores the same registers `fanout` times
// instead of re-reading).
//
// A contiguous run is moved in 16-byte chunks that are aligned on the *target* side, so stores are
// always full 16-byte vectors.  When run length and offsets are multiples of 16 (ALIGNED) the source
// chunk is one aligned load.  Otherwise (odd shapes) the source chunk is assembled from the two
// aligned 16-byte blocks that contain it (byte funnel shift), and the few bytes before the first and
// after the last target-aligned chunk of a run are copied in `unit_bytes` pieces.  Loads only ever
// touch 16-byte blocks that hold at least one byte of the tile.
//
// Aligned runs of 512 bytes or more do not pass through registers at all: each row segment of a work
// item is one TMA bulk copy global -> shared (cp.async.bulk, byte-counted completion on an mbarrier)
// and one bulk copy shared -> global per target replica, issued by a few threads (bulk_body below;
// measured 1-3 % faster than the register path on every benchmark configuration).  Everything else
// uses the item shapes below (CopyGeometry::mode):
//   kModeRows    aligned runs below the bulk threshold: a block of 256 threads covers rows_per_pass
//                rows of `lanes` chunks; a thread keeps its column and walks down the rows of its work
//                item, kUnroll independent loads in flight before the stores.
//   kModeChunks  ragged runs of 256 bytes or more (and aligned long runs when bulk copies are switched
//                off): the rows of an item are decoded once into shared memory and all threads walk the
//                (row, chunk) space of the item with a flat index.  With bulk copies on, the source
//                bytes of a ragged item are first brought into shared memory by one bulk copy per row
//                (ragged_bulk_body) and the walk shifts its chunks out of shared memory.
//   kModeUnits   ragged runs below 256 bytes: the same flat walk over pieces of unit_bytes.
//   kModeGather  runs below 256 bytes that are interleaved into long target rows: the walk follows the
//                target in whole 16-byte chunks and fetches every unit from its computed source.
//   kModeZip     the same interleaving (either direction) when the row digit next to it is contiguous
//                on both sides: source segments staged in shared memory by bulk copies (zip_body).
//   kModeBox     short runs that interleave along several dimensions at once: the item is widened to a
//                super-box that covers whole tiles of both sides in those dimensions, staged in shared
//                memory segment by segment and written out range by range (box_body).
// Index decoding uses multiply-shift division by host-computed constants; the per-item decode (box ->
// tiles and base offsets) is amortised over ~32 KiB of data.  Every kernel starts with
// griddepcontrol.launch_dependents and places griddepcontrol.wait after the decode of its first work
// item, just before its first access to global memory (programmatic dependent launch).
//
// Checked build (-DREDIST_BOUNDS, a second library used by the tests): every global load, store and
// bulk-copy range is tested against the tiles of the launch's pointer tables (on the read side a tile
// counts up to the next 16-byte boundary past its end, which the ragged paths may read), and every
// index into dynamic shared memory against the launch's shared-memory size.  An access that fails the
// test is skipped, never performed; the first one is recorded (source line of the access, block, which
// side, distance from the nearest tile base) and all are counted.  In the normal build the tests
// compile to `true`.
#include <cuda_runtime.h>

#include "copy_params.h"
#include "kernels.h"

// The file compiles as one translation unit (REDIST_PART undefined or 0) or as three that build in parallel
// (-DREDIST_PART=1: register, bulk-copy and gather kernels plus the host side; 2: zip kernels; 3: super-box
// kernels).  Kernel templates are instantiated only where entry_for names them, so each part carries its own
// kernels and nothing else; each part also has its own copy of the device-side counters, which the readers
// in part 1 add up.
#ifndef REDIST_PART
#define REDIST_PART 0
#endif
#define REDIST_IN(part) (REDIST_PART == 0 || REDIST_PART == (part))

namespace redist {

namespace {

#ifdef REDIST_BOUNDS
__device__ unsigned long long g_bounds_count = 0;
__device__ unsigned int g_bounds_taken = 0;
__device__ long long g_bounds_first[4] = {0, 0, 0, 0};   // source line, block, side (1 read, 2 write, 3 shared), distance

__device__ __noinline__ void bounds_violation(int line, int side, long long distance)
{
    atomicAdd(&g_bounds_count, 1ull);
    if (atomicExch(&g_bounds_taken, 1u) == 0u) {
        g_bounds_first[0] = line;
        g_bounds_first[1] = blockIdx.x;
        g_bounds_first[2] = side;
        g_bounds_first[3] = distance;
    }
}

// [p, p + bytes) must lie inside one tile of the table (`slack`: the tile counts up to the next 16-byte boundary)
template <class PTR>
__device__ __noinline__ bool bounds_in_table(PTR const *tab, uint32_t n, uint64_t tile_bytes, bool slack, const void *p,
                                             uint64_t bytes, int line, int side)
{
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    const uint64_t lim = slack ? ((tile_bytes + 15u) & ~uint64_t(15)) : tile_bytes;
    long long best = -1;
    for (uint32_t t = 0; t < n; ++t) {
        const uintptr_t b = reinterpret_cast<uintptr_t>(tab[t]);
        if (a >= b) {
            if (a - b + bytes <= lim) return true;
            if (best < 0 || (long long)(a - b) < best) best = (long long)(a - b);
        }
    }
    bounds_violation(line, side, best);
    return false;
}

__device__ __forceinline__ bool bounds_in_smem(uint32_t off, uint32_t bytes, int line)
{
    uint32_t dyn;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (uint64_t(off) + bytes <= dyn) return true;
    bounds_violation(line, 3, off);
    return false;
}

__device__ __forceinline__ bool bounds_index(uint32_t i, uint32_t cap, int line)
{
    if (i < cap) return true;
    bounds_violation(line, 3, i);
    return false;
}
#define CHK_SRC(P, ptr, bytes) bounds_in_table((P).src, (P).g.n_src_tab, (P).g.src_tile_bytes, true, (ptr), (bytes), __LINE__, 1)
#define CHK_DST(P, ptr, bytes) bounds_in_table((P).dst, (P).g.n_dst_tab, (P).g.dst_tile_bytes, false, (ptr), (bytes), __LINE__, 2)
#define CHK_SMEM(off, bytes) bounds_in_smem((off), (bytes), __LINE__)
#define CHK_IDX(i, cap) bounds_index((i), (cap), __LINE__)
#else
#define CHK_SRC(P, ptr, bytes) true
#define CHK_DST(P, ptr, bytes) true
#define CHK_SMEM(off, bytes) true
#define CHK_IDX(i, cap) true
#endif

#ifndef REDIST_UNROLL
#define REDIST_UNROLL 4
#endif
constexpr int kUnroll = REDIST_UNROLL;

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv &f)
{
    return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

// Programmatic dependent launch: a kernel may start while the previous kernel of the stream still runs;
// it must not touch global memory before this wait (kernel parameters and shared memory are free), so
// every body decodes its first work item first and waits just before its first load.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// streaming accesses: the data is touched once
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) { __stcs(p, v); }

// The 16 bytes that start m bytes (0 < m < 16) into the 32 bytes (a, b).
__device__ __forceinline__ uint4 funnel_shift16(const uint4 &a, const uint4 &b, uint32_t m)
{
    const uint32_t bs = (m & 3u) * 8u;
    uint4 o;
    switch (m >> 2) {
    case 0:
        o.x = __funnelshift_r(a.x, a.y, bs); o.y = __funnelshift_r(a.y, a.z, bs);
        o.z = __funnelshift_r(a.z, a.w, bs); o.w = __funnelshift_r(a.w, b.x, bs);
        break;
    case 1:
        o.x = __funnelshift_r(a.y, a.z, bs); o.y = __funnelshift_r(a.z, a.w, bs);
        o.z = __funnelshift_r(a.w, b.x, bs); o.w = __funnelshift_r(b.x, b.y, bs);
        break;
    case 2:
        o.x = __funnelshift_r(a.z, a.w, bs); o.y = __funnelshift_r(a.w, b.x, bs);
        o.z = __funnelshift_r(b.x, b.y, bs); o.w = __funnelshift_r(b.y, b.z, bs);
        break;
    default:
        o.x = __funnelshift_r(a.w, b.x, bs); o.y = __funnelshift_r(b.x, b.y, bs);
        o.z = __funnelshift_r(b.y, b.z, bs); o.w = __funnelshift_r(b.z, b.w, bs);
        break;
    }
    return o;
}

// 16 bytes starting at an arbitrary address: the aligned block that holds the first byte and, when
// the address is not a multiple of 16, the next one (which then holds the last byte).
__device__ __forceinline__ uint4 ld_shifted(const char *src)
{
    const uint32_t m = uint32_t(reinterpret_cast<uintptr_t>(src)) & 15u;
    const uint4 *p = reinterpret_cast<const uint4 *>(src - m);
    const uint4 a = __ldg(p);
    if (m == 0) return a;
    return funnel_shift16(a, __ldg(p + 1), m);
}

// Copy `count` pieces of `unit` bytes (unit = 1, 2, 4 or 8; all addresses are multiples of it) from
// src to every target replica; pieces are dealt to threads first, first + step, ...
template <int NT>
__device__ __forceinline__ void copy_units(const CopyParams<NT> &P, char *const *dtab, uint32_t fanout, int64_t doff,
                                           const char *src, uint32_t count, uint32_t unit, uint32_t first, uint32_t step)
{
    for (uint32_t u = first; u < count; u += step) {
        const int64_t off = int64_t(u) * unit;
        if (!CHK_SRC(P, src + off, unit)) continue;
#ifdef REDIST_BOUNDS
        bool all = true;
        for (uint32_t f = 0; f < fanout; ++f) all = CHK_DST(P, dtab[f] + doff + off, unit) && all;
        if (!all) continue;
#endif
        switch (unit) {
        case 8: {
            const uint2 v = *reinterpret_cast<const uint2 *>(src + off);
            for (uint32_t f = 0; f < fanout; ++f) *reinterpret_cast<uint2 *>(dtab[f] + doff + off) = v;
            break;
        }
        case 4: {
            const uint32_t v = *reinterpret_cast<const uint32_t *>(src + off);
            for (uint32_t f = 0; f < fanout; ++f) *reinterpret_cast<uint32_t *>(dtab[f] + doff + off) = v;
            break;
        }
        case 2: {
            const uint16_t v = *reinterpret_cast<const uint16_t *>(src + off);
            for (uint32_t f = 0; f < fanout; ++f) *reinterpret_cast<uint16_t *>(dtab[f] + doff + off) = v;
            break;
        }
        default: {
            const uint8_t v = *reinterpret_cast<const uint8_t *>(src + off);
            for (uint32_t f = 0; f < fanout; ++f) *reinterpret_cast<uint8_t *>(dtab[f] + doff + off) = v;
            break;
        }
        }
    }
}

// row number inside a box -> byte offsets of the row on the source and target side
__device__ __forceinline__ void row_offsets(const CopyGeometry &g, uint32_t row, int64_t &s1, int64_t &s2,
                                            int n_row)
{
    s1 = 0;
    s2 = 0;
    uint32_t r = row;
    for (int q = n_row - 1; q > 0; --q) {
        const uint32_t nxt = fdiv(r, g.row_n[q]);
        const uint32_t dg = r - nxt * g.row_n[q].d;
        r = nxt;
        s1 += int64_t(dg) * g.row_b1[q];
        s2 += int64_t(dg) * g.row_b2[q];
    }
    if (n_row > 0) {
        s1 += int64_t(r) * g.row_b1[0];
        s2 += int64_t(r) * g.row_b2[0];
    }
}

// head bytes before the first target-aligned chunk and number of whole chunks of a run
__device__ __forceinline__ void split_run(uint64_t len, int64_t dst_off, uint32_t &head, uint32_t &chunks)
{
    const uint32_t h = (16u - (uint32_t(dst_off) & 15u)) & 15u;
    head = uint64_t(h) < len ? h : uint32_t(len);
    chunks = uint32_t((len - head) >> 4);
}

struct RowEntry {
    int64_t s1, s2;
};

struct BoxBase {
    const char *sbase;       // source tile base + offset of the box
    char *const *dtab;       // target replica base pointers
    int64_t o1, o2;          // offset of the box inside the source / target tile
    uint32_t t1, t2;         // source / target tile index
    uint32_t part;           // item number inside the box
};

template <int NT>
__device__ __forceinline__ BoxBase decode_box(const CopyParams<NT> &P, uint32_t item)
{
    const CopyGeometry &g = P.g;
    // item = ((slow boxes * items_per_box + part) * fast_boxes + fast box) * inner_n + piece
    const uint32_t outer = fdiv(item, g.inner_n);
    const uint32_t piece = item - outer * g.inner_n.d;
    const uint32_t rest = fdiv(outer, g.fast_boxes);
    const uint32_t slow = fdiv(rest, g.items_per_box);
    uint32_t t1 = 0, t2 = 0, rem = slow * g.fast_boxes.d + (outer - rest * g.fast_boxes.d);
    int64_t o1 = 0, o2 = 0;
    for (int u = int(g.n_unit) - 1; u >= 0; --u) {
        const uint32_t nxt = fdiv(rem, g.unit_n[u]);
        uint32_t q = rem - nxt * g.unit_n[u].d;
        rem = nxt;
        if (uint32_t(u) == g.inner_digit) q = q * g.inner_span + piece * g.inner_mul;
        q *= g.unit_mul[u];
        const uint32_t a1 = fdiv(q, g.unit_m1[u]);
        const uint32_t a2 = fdiv(q, g.unit_m2[u]);
        t1 += a1 * g.unit_ts1[u];
        t2 += a2 * g.unit_ts2[u];
        o1 += int64_t(q - a1 * g.unit_m1[u].d) * g.unit_b1[u];
        o2 += int64_t(q - a2 * g.unit_m2[u].d) * g.unit_b2[u];
    }
    BoxBase b;
    b.sbase = P.src[t1] + o1;
    b.dtab = &P.dst[t2 * g.fanout];
    b.o1 = o1;
    b.o2 = o2;
    b.t1 = t1;
    b.t2 = t2;
    b.part = rest - slow * g.items_per_box.d;
    return b;
}

// ---- kModeRows: thread (ty, tx) handles chunk tx of rows ty, ty + rows_per_pass, ... ------------
template <int NT>
__device__ __forceinline__ void rows_body(const CopyParams<NT> &P)
{
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t fanout = g.fanout;
    const uint32_t lanes = g.lanes;
    const uint32_t ty = fdiv(tid, g.lanes_div);
    const uint32_t tx = tid - ty * lanes;
    const uint32_t rpp = g.rows_per_pass;
    const bool active = ty < rpp;
    for (uint32_t item = blockIdx.x; item < g.n_items; item += gridDim.x) {
        const BoxBase b = decode_box(P, item);
        if (item == blockIdx.x) wait_for_previous_kernel();
        const char *sb = b.sbase + int64_t(tx) * 16;
        const int64_t dcol = b.o2 + int64_t(tx) * 16;
        const uint32_t row0 = b.part * g.rows_per_item;
        const uint32_t row_end = min(row0 + g.rows_per_item, g.rows);
        for (uint32_t rb = row0; rb < row_end; rb += rpp * kUnroll) {
            uint4 v[kUnroll];
            int64_t d2[kUnroll];
            bool ok[kUnroll];
#pragma unroll
            for (int k = 0; k < kUnroll; ++k) {
                const uint32_t row = rb + k * rpp + ty;
                int64_t s1, s2;
                row_offsets(g, row, s1, s2, int(g.n_row));
                ok[k] = active && row < row_end;
                d2[k] = dcol + s2;
                ok[k] = ok[k] && CHK_SRC(P, sb + s1, 16);
                if (ok[k]) v[k] = ld_stream(reinterpret_cast<const uint4 *>(sb + s1));
            }
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dbase = b.dtab[f];
#pragma unroll
                for (int k = 0; k < kUnroll; ++k)
                    if (ok[k] && CHK_DST(P, dbase + d2[k], 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d2[k]), v[k]);
            }
        }
    }
}

// rows of the item -> shared table (decoded once, by the first threads)
__device__ __forceinline__ uint32_t fill_rowtab(const CopyGeometry &g, RowEntry *rowtab, uint32_t group)
{
    const uint32_t row0 = group * g.rows_per_item;
    const uint32_t nr = min(g.rows_per_item, g.rows - row0);
    __syncthreads();
    for (uint32_t r = threadIdx.x; r < nr; r += kBlockThreads) {
        RowEntry e;
        row_offsets(g, row0 + r, e.s1, e.s2, int(g.n_row_tab));
        rowtab[r] = e;
    }
    __syncthreads();
    return nr;
}

// ---- kModeChunks: flat walk over (row, 16-byte chunk) ------------------------------------------
template <bool ALIGNED, int NT>
__device__ __forceinline__ void chunks_body(const CopyParams<NT> &P, RowEntry *rowtab)
{
    // ragged chunks cost two loads and more registers each: fewer in flight per thread, more blocks per SM
    constexpr int kU = ALIGNED ? kUnroll : 2;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t fanout = g.fanout;
    const uint64_t len = g.run_bytes;
    const uint32_t cpb = g.per_block;
    for (uint32_t item = blockIdx.x; item < g.n_items; item += gridDim.x) {
        const BoxBase b = decode_box(P, item);
        const uint32_t group = fdiv(b.part, g.col_blocks);
        const uint32_t cb = b.part - group * g.col_blocks.d;
        const uint32_t nr = fill_rowtab(g, rowtab, group);
        if (item == blockIdx.x) wait_for_previous_kernel();
        const uint32_t total = nr * cpb;
        const uint32_t c0 = cb * cpb;
        for (uint32_t base = tid; base < total; base += kBlockThreads * kU) {
            uint4 v[kU];
            int64_t d2[kU];
            bool ok[kU];
#pragma unroll
            for (int k = 0; k < kU; ++k) {
                const uint32_t idx = base + k * kBlockThreads;
                const uint32_t r = fdiv(idx, g.per_block_div);
                const uint32_t j = c0 + (idx - r * cpb);
                const RowEntry e = rowtab[r < nr ? r : 0];
                uint32_t head = 0, chunks = uint32_t(len >> 4);
                if (!ALIGNED) split_run(len, b.o2 + e.s2, head, chunks);
                ok[k] = idx < total && j < chunks;
                const int64_t col = int64_t(head) + (int64_t(j) << 4);
                d2[k] = b.o2 + e.s2 + col;
#ifdef REDIST_BOUNDS
                if (ok[k]) {
                    const char *sp = b.sbase + e.s1 + col;
                    const uint32_t mis = uint32_t(reinterpret_cast<uintptr_t>(sp)) & 15u;
                    ok[k] = ALIGNED ? CHK_SRC(P, sp, 16) : CHK_SRC(P, sp - mis, mis ? 32 : 16);
                }
#endif
                if (ok[k]) {
                    if (ALIGNED)
                        v[k] = ld_stream(reinterpret_cast<const uint4 *>(b.sbase + e.s1 + col));
                    else
                        v[k] = ld_shifted(b.sbase + e.s1 + col);
                }
            }
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dbase = b.dtab[f];
#pragma unroll
                for (int k = 0; k < kU; ++k)
                    if (ok[k] && CHK_DST(P, dbase + d2[k], 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d2[k]), v[k]);
            }
        }
        if (!ALIGNED) {
            // ragged ends: the bytes before the first target-aligned chunk belong to the first column
            // block, those after the last whole chunk to the last; flat walk over (row, slot)
            const uint32_t unit = g.unit_bytes;
            const uint32_t slots = 16u / unit - 1u;          // at most 15 bytes on either end
            const bool first = cb == 0, last = cb + 1 == g.col_blocks.d;
            const uint32_t ends = (first ? 1u : 0u) + (last ? 1u : 0u);
            for (uint32_t idx = tid; idx < nr * slots * ends; idx += kBlockThreads) {
                const uint32_t r = idx / (slots * ends);
                const uint32_t w = idx - r * (slots * ends);
                const bool is_head = first && w < slots;
                const uint32_t slot = is_head ? w : (first ? w - slots : w);
                const RowEntry e = rowtab[r];
                uint32_t head, chunks;
                split_run(len, b.o2 + e.s2, head, chunks);
                const int64_t toff = int64_t(head) + (int64_t(chunks) << 4);
                const uint32_t count = is_head ? head / unit : uint32_t(len - uint64_t(toff)) / unit;
                const int64_t off = is_head ? 0 : toff;
                if (slot < count)
                    copy_units(P, b.dtab, fanout, b.o2 + e.s2 + off, b.sbase + e.s1 + off, slot + 1, unit, slot, slots + 1);
            }
        }
    }
}

// ---- kModeUnits: flat walk over (table row, run of the innermost row digit, piece of UNIT bytes) --
template <typename T, bool INNER, int NT>
__device__ __forceinline__ void units_walk(const CopyParams<NT> &P, RowEntry *rowtab)
{
    constexpr int kU = 2 * kUnroll;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t fanout = g.fanout;
    const uint32_t cpb = g.per_block;                 // pieces of one table row in a column block
    const uint32_t upr = g.units_per_run.d;
    const uint32_t payload = g.tab_inner.d * upr;     // pieces per table row
    const int64_t in1 = g.n_row_tab < g.n_row ? g.row_b1[g.n_row - 1] : 0;   // strides of the innermost digit
    const int64_t in2 = g.n_row_tab < g.n_row ? g.row_b2[g.n_row - 1] : 0;
    for (uint32_t item = blockIdx.x; item < g.n_items; item += gridDim.x) {
        const BoxBase b = decode_box(P, item);
        const uint32_t group = fdiv(b.part, g.col_blocks);
        const uint32_t cb = b.part - group * g.col_blocks.d;
        const uint32_t nr = fill_rowtab(g, rowtab, group);
        if (item == blockIdx.x) wait_for_previous_kernel();
        const uint32_t total = nr * cpb;
        const uint32_t c0 = cb * cpb;
        for (uint32_t base = tid; base < total; base += kBlockThreads * kU) {
            T v[kU];
            int64_t d2[kU];
            bool ok[kU];
#pragma unroll
            for (int k = 0; k < kU; ++k) {
                const uint32_t idx = base + k * kBlockThreads;
                const uint32_t r = fdiv(idx, g.per_block_div);
                const uint32_t c = c0 + (idx - r * cpb);
                const RowEntry e = rowtab[r < nr ? r : 0];
                ok[k] = idx < total && c < payload;
                int64_t a1 = e.s1 + int64_t(c) * sizeof(T), a2 = e.s2 + int64_t(c) * sizeof(T);
                if (INNER) {   // c = run number * pieces per run + piece
                    const uint32_t i = fdiv(c, g.units_per_run);
                    const uint32_t u = c - i * upr;
                    a1 = e.s1 + int64_t(i) * in1 + int64_t(u) * sizeof(T);
                    a2 = e.s2 + int64_t(i) * in2 + int64_t(u) * sizeof(T);
                }
                d2[k] = b.o2 + a2;
                ok[k] = ok[k] && CHK_SRC(P, b.sbase + a1, uint32_t(sizeof(T)));
                if (ok[k]) v[k] = __ldg(reinterpret_cast<const T *>(b.sbase + a1));
            }
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dbase = b.dtab[f];
#pragma unroll
                for (int k = 0; k < kU; ++k)
                    if (ok[k] && CHK_DST(P, dbase + d2[k], uint32_t(sizeof(T)))) *reinterpret_cast<T *>(dbase + d2[k]) = v[k];
            }
        }
    }
}

template <int NT>
__device__ __forceinline__ void units_body(const CopyParams<NT> &P, RowEntry *rowtab)
{
    if (P.g.tab_inner.d > 1) {
        switch (P.g.unit_bytes) {
        case 8: units_walk<uint2, true, NT>(P, rowtab); break;
        case 4: units_walk<uint32_t, true, NT>(P, rowtab); break;
        case 2: units_walk<uint16_t, true, NT>(P, rowtab); break;
        default: units_walk<uint8_t, true, NT>(P, rowtab); break;
        }
    } else {
        switch (P.g.unit_bytes) {
        case 8: units_walk<uint2, false, NT>(P, rowtab); break;
        case 4: units_walk<uint32_t, false, NT>(P, rowtab); break;
        case 2: units_walk<uint16_t, false, NT>(P, rowtab); break;
        default: units_walk<uint8_t, false, NT>(P, rowtab); break;
        }
    }
}

// VARIANT: 0 rows (aligned), 1 chunks aligned, 2 chunks ragged, 3 units
template <int VARIANT, int NT>
__device__ __forceinline__ void copy_body(const CopyParams<NT> &P)
{
    // Programmatic dependent launch: blocks of this grid may be scheduled while the previous kernel
    // on the stream drains; nothing is read or written before that kernel has completed and its
    // stores are visible.  The next kernel is released to do the same as soon as every block of this
    // grid has started.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (VARIANT == 0) {
        rows_body<NT>(P);
    } else {
        __shared__ RowEntry rowtab[kMaxRowsFlat];
        if (VARIANT == 1) chunks_body<true, NT>(P, rowtab);
        if (VARIANT == 2) chunks_body<false, NT>(P, rowtab);
        if (VARIANT == 3) units_body<NT>(P, rowtab);
    }
}

// ---- kModeGather: target stretches in whole chunks, every unit fetched from its computed source ----
// Position x (bytes, a multiple of sizeof(T)) inside the stretch of table row `e` -> source address.
// Long target rows: x = ((row digits..., piece j), byte in run); piece j lives in source tile t1 + j * ts.
// Long source rows: the stretch belongs to target tile j; x = ((row digits...), byte in run) and the
// source row holds the m pieces side by side.
template <bool LONG_DST, typename T, int NT>
__device__ __forceinline__ const T *gather_src(const CopyParams<NT> &P, const BoxBase &b, const RowEntry &e,
                                               uint32_t j, uint32_t x)
{
    const CopyGeometry &g = P.g;
    const uint32_t xu = x / uint32_t(sizeof(T));
    const uint32_t k = fdiv(xu, g.units_per_run);
    int64_t off = int64_t((xu - k * g.units_per_run.d) * uint32_t(sizeof(T)));
    uint32_t rr = k;
    if (LONG_DST) {
        rr = fdiv(k, g.gl_m);
        j = k - rr * g.gl_m.d;
    }
    if (g.gl_levels == 2) {
        const uint32_t nx = fdiv(rr, g.gl_n[0]);
        off += int64_t(rr - nx * g.gl_n[0].d) * g.gl_b1[0] + int64_t(nx) * g.gl_b1[1];
    } else if (g.gl_levels == 1) {
        off += int64_t(rr) * g.gl_b1[0];
    }
    const char *base = LONG_DST ? P.src[b.t1 + j * g.gl_ts] + b.o1 : b.sbase + int64_t(j) * int64_t(g.run_bytes);
    return reinterpret_cast<const T *>(base + e.s1 + off);
}

template <bool LONG_DST, typename T, int NT>
__device__ __forceinline__ uint4 gather_chunk(const CopyParams<NT> &P, const BoxBase &b, const RowEntry &e,
                                              uint32_t j, uint32_t x)
{
    constexpr int kPer = 16 / int(sizeof(T));
    union {
        uint4 v;
        T t[kPer];
    } u;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const T *sp = gather_src<LONG_DST, T, NT>(P, b, e, j, x + uint32_t(i * sizeof(T)));
        u.t[i] = CHK_SRC(P, sp, uint32_t(sizeof(T))) ? __ldg(sp) : T();
    }
    return u.v;
}

template <bool LONG_DST, typename T, int NT>
__device__ __forceinline__ void gather_body(const CopyParams<NT> &P, RowEntry *rowtab)
{
    constexpr int kU = 2;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t fanout = g.fanout;
    const uint32_t S = g.gl_stretch;
    const uint32_t cpb = g.per_block;
    const uint32_t ns = LONG_DST ? 1u : g.gl_m.d;         // stretches per table row
    for (uint32_t item = blockIdx.x; item < g.n_items; item += gridDim.x) {
        const BoxBase b = decode_box(P, item);
        const uint32_t group = fdiv(b.part, g.col_blocks);
        const uint32_t cb = b.part - group * g.col_blocks.d;
        const uint32_t nr = fill_rowtab(g, rowtab, group);
        if (item == blockIdx.x) wait_for_previous_kernel();
        const uint32_t total = nr * ns * cpb;
        const uint32_t c0 = cb * cpb;
        for (uint32_t base = tid; base < total; base += kBlockThreads * kU) {
            uint4 v[kU];
            int64_t d2[kU];
            uint32_t jt[kU];
            bool ok[kU];
#pragma unroll
            for (int k = 0; k < kU; ++k) {
                const uint32_t idx = base + k * kBlockThreads;
                const uint32_t rs = fdiv(idx, g.per_block_div);
                const uint32_t c = c0 + (idx - rs * cpb);
                uint32_t r = rs, j = 0;
                if (!LONG_DST) {
                    r = fdiv(rs, g.gl_m);
                    j = rs - r * g.gl_m.d;
                }
                const RowEntry e = rowtab[r < nr ? r : 0];
                uint32_t head, chunks;
                split_run(S, b.o2 + e.s2, head, chunks);
                ok[k] = idx < total && c < chunks;
                const uint32_t x = head + (c << 4);
                d2[k] = b.o2 + e.s2 + x;
                jt[k] = j;
                if (ok[k]) v[k] = gather_chunk<LONG_DST, T, NT>(P, b, e, j, x);
            }
            for (uint32_t f = 0; f < fanout; ++f) {
#pragma unroll
                for (int k = 0; k < kU; ++k) {
                    char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + jt[k] * g.gl_ts) * fanout + f];
                    if (ok[k] && CHK_DST(P, dbase + d2[k], 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d2[k]), v[k]);
                }
            }
        }
        // ragged ends of the stretches, unit by unit: heads with the first column block, tails with the last
        constexpr uint32_t kSlots = 16u / uint32_t(sizeof(T)) - 1u;
        if constexpr (kSlots > 0) {
            const bool first = cb == 0, last = cb + 1 == g.col_blocks.d;
            const uint32_t ends = (first ? 1u : 0u) + (last ? 1u : 0u);
            for (uint32_t idx = tid; idx < nr * ns * kSlots * ends; idx += kBlockThreads) {
                const uint32_t rs = idx / (kSlots * ends);
                const uint32_t w = idx - rs * (kSlots * ends);
                const bool is_head = first && w < kSlots;
                const uint32_t slot = is_head ? w : (first ? w - kSlots : w);
                uint32_t r = rs, j = 0;
                if (!LONG_DST) {
                    r = fdiv(rs, g.gl_m);
                    j = rs - r * g.gl_m.d;
                }
                const RowEntry e = rowtab[r];
                uint32_t head, chunks;
                split_run(S, b.o2 + e.s2, head, chunks);
                const uint32_t toff = head + (chunks << 4);
                const uint32_t count = (is_head ? head : S - toff) / uint32_t(sizeof(T));
                if (slot < count) {
                    const uint32_t x = (is_head ? 0u : toff) + slot * uint32_t(sizeof(T));
                    const T *sp = gather_src<LONG_DST, T, NT>(P, b, e, j, x);
                    if (!CHK_SRC(P, sp, uint32_t(sizeof(T)))) continue;
                    const T val = __ldg(sp);
                    for (uint32_t f = 0; f < fanout; ++f) {
                        char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + j * g.gl_ts) * fanout + f];
                        if (CHK_DST(P, dbase + b.o2 + e.s2 + x, uint32_t(sizeof(T)))) *reinterpret_cast<T *>(dbase + b.o2 + e.s2 + x) = val;
                    }
                }
            }
        }
    }
}

// The gather, zip and super-box kernels come in two builds each: SMALL = false for units of 4, 8 and 16
// bytes, SMALL = true for units of 1 and 2 bytes (odd run lengths of 8- and 16-bit elements), where a
// 16-byte chunk is assembled from 8 or 16 units.  They are separate kernels so that the registers the
// small-unit walks need do not lower the occupancy of the others.
template <bool LONG_DST, int NT, bool SMALL>
__device__ __forceinline__ void gather_dispatch(const CopyParams<NT> &P)
{
    __shared__ RowEntry rowtab[kMaxRowsFlat];
    if constexpr (SMALL) {
        if (P.g.unit_bytes == 2)
            gather_body<LONG_DST, uint16_t, NT>(P, rowtab);
        else
            gather_body<LONG_DST, uint8_t, NT>(P, rowtab);
    } else {
        switch (P.g.unit_bytes) {
        case 16: gather_body<LONG_DST, uint4, NT>(P, rowtab); break;
        case 8: gather_body<LONG_DST, uint2, NT>(P, rowtab); break;
        default: gather_body<LONG_DST, uint32_t, NT>(P, rowtab); break;
        }
    }
}

#define REDIST_DEFINE_GATHER_KERNEL(NAME)                                                            \
    template <bool LONG_DST, int NT, bool SMALL>                                                     \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P)  \
    {                                                                                                \
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");                              \
        gather_dispatch<LONG_DST, NT, SMALL>(P);                                                     \
    }

REDIST_DEFINE_GATHER_KERNEL(redist_dynslice_gather_kernel)
REDIST_DEFINE_GATHER_KERNEL(redist_alltoall_gather_kernel)
REDIST_DEFINE_GATHER_KERNEL(redist_allgather_gather_kernel)
REDIST_DEFINE_GATHER_KERNEL(redist_allpermute_gather_kernel)
REDIST_DEFINE_GATHER_KERNEL(redist_fused_gather_kernel)

// ---- bulk-copy variant (aligned runs of at least 512 bytes): TMA moves the segments --------------
// One work item per block.  Every row segment of the item is one bulk asynchronous copy global ->
// shared (cp.async.bulk, completion counted in bytes on an mbarrier) and, once all have landed, one
// bulk copy shared -> global per target replica.  A handful of threads issue the copies; nothing
// passes through registers.  Every copy is addressed to this block's own shared memory only.
//
// The wait on the mbarrier is bounded (CopyGeometry::wait_polls polls).  A thread whose wait runs out
// stores nothing; the first such thread of a block counts the block in g_bulk_timeouts; and before it
// returns, every such thread polls on, with a sleep that grows to 256 ns between polls, for up to
// wait_polls further polls, so that copies still in flight can land while the block still owns its
// shared memory.  Past that cap (about 70 ms with the default limit) the block returns: a copy that
// lands even later would write into shared memory that the SM may have given to another block, and
// that block's output would be wrong as well -- the non-zero counter says that the run is invalid.
__device__ unsigned int g_bulk_timeouts = 0;

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t parity, uint32_t limit)
{
    for (uint32_t it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(mbar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

__device__ __noinline__ void bulk_wait_ran_out(uint32_t mbar, unsigned int *block_flag, uint32_t polls)
{
    if (atomicExch(block_flag, 1u) == 0u) atomicAdd(&g_bulk_timeouts, 1u);
    uint32_t ns = 32;
    for (uint32_t it = 0; it < polls; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(mbar), "r"(0u)
            : "memory");
        if (done) return;
        __nanosleep(ns);
        if (ns < 256) ns <<= 1;
    }
}

template <int NT>
__device__ __forceinline__ void bulk_body(const CopyParams<NT> &P)
{
    extern __shared__ __align__(128) unsigned char stage[];
    __shared__ __align__(8) unsigned long long mbar_storage;
    __shared__ unsigned int wait_failed;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t mbar = smem_addr(&mbar_storage);
    if (tid == 0) {
        wait_failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // (the wait for the previous kernel of the stream comes just before the first access to global
    // memory: decoding the item only reads kernel parameters)
    const uint32_t item = blockIdx.x;
    if (item >= g.n_items) return;
    const BoxBase b = decode_box(P, item);
    // the item's segments: rows [row0, row0 + nr), bytes [seg_off, seg_off + seg_bytes) of every run
    uint32_t row0, nr;
    uint64_t seg_off = 0, seg_bytes = g.run_bytes;
    if (g.mode == kModeRows) {
        row0 = b.part * g.rows_per_item;
        nr = min(g.rows_per_item, g.rows - row0);
    } else {
        const uint32_t group = fdiv(b.part, g.col_blocks);
        const uint32_t cb = b.part - group * g.col_blocks.d;
        row0 = group * g.rows_per_item;
        nr = min(g.rows_per_item, g.rows - row0);
        seg_off = uint64_t(cb) * g.per_block * 16u;
        seg_bytes = min(uint64_t(g.per_block) * 16u, g.run_bytes - seg_off);
    }
    const uint32_t bytes = uint32_t(seg_bytes);
    if (tid == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(nr * bytes + g.test_extra_tx) : "memory");
    }
    __syncthreads();
    int64_t s1 = 0, s2 = 0;
    const bool mine = tid < nr;          // at most one row per thread (the host guarantees nr <= kBulkThreads)
    const uint32_t slot = smem_addr(stage) + tid * bytes;
    if (mine) row_offsets(g, row0 + tid, s1, s2, int(g.n_row));
    wait_for_previous_kernel();
    if (!mine) return;                   // the other threads have nothing to move and nothing to wait for
    const char *src = b.sbase + s1 + int64_t(seg_off);
    uint64_t policy = 0;
    if (g.l2_hint) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    if (CHK_SRC(P, src, bytes) && CHK_SMEM(tid * bytes, bytes)) {
        if (g.l2_hint & 1u)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                         ::"r"(slot), "l"(src), "r"(bytes), "r"(mbar), "l"(policy)
                         : "memory");
        else
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(slot), "l"(src), "r"(bytes), "r"(mbar)
                         : "memory");
    } else {
        // checked build only: the skipped copy's bytes are taken off the count the barrier waits for
        asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
    }
    if (!mbar_wait_bounded(mbar, 0, g.wait_polls)) {
        bulk_wait_ran_out(mbar, &wait_failed, g.wait_polls);
        return;
    }
    for (uint32_t f = 0; f < g.fanout; ++f) {
        char *dst = b.dtab[f] + b.o2 + s2 + int64_t(seg_off);
        if (!CHK_DST(P, dst, bytes)) continue;
        if (g.l2_hint & 2u)
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                         ::"l"(dst), "r"(slot), "r"(bytes), "l"(policy)
                         : "memory");
        else
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(dst), "r"(slot), "r"(bytes)
                         : "memory");
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// One entry per collective so that profiles name the step that ran.
#define REDIST_DEFINE_BULK_KERNEL(NAME)                                                              \
    template <int NT>                                                                                \
    __global__ void __launch_bounds__(kBulkThreads) NAME(const __grid_constant__ CopyParams<NT> P)   \
    {                                                                                                \
        bulk_body<NT>(P);                                                                            \
    }

REDIST_DEFINE_BULK_KERNEL(redist_dynslice_bulk_kernel)
REDIST_DEFINE_BULK_KERNEL(redist_alltoall_bulk_kernel)
REDIST_DEFINE_BULK_KERNEL(redist_allgather_bulk_kernel)
REDIST_DEFINE_BULK_KERNEL(redist_allpermute_bulk_kernel)
REDIST_DEFINE_BULK_KERNEL(redist_fused_bulk_kernel)

// ---- ragged bulk-in (bulk == 2): the ragged chunk walk with its loads done by TMA ----------------
// Same items as the ragged chunk walk.  For every row of the item one thread posts the byte count on
// the mbarrier and issues one bulk copy of the 16-byte blocks that cover the row's source bytes for
// this column block; when all rows have landed, the threads walk (row, chunk) as before but read the
// source chunk from shared memory (two aligned 16-byte reads and a funnel shift), so no thread ever
// waits on a global load.  Ragged heads and tails are copied from shared memory in unit pieces.
struct RaggedRow {
    uint32_t base;           // shared-memory offset of the row-relative source byte 0 (may wrap below the slot)
    uint32_t head, chunks;   // bytes before the first target-aligned chunk, whole chunks of the run
    uint32_t pad;
};

__device__ __forceinline__ uint4 lds_shifted(const unsigned char *tile, uint32_t at)
{
    const uint32_t m = at & 15u;
    const uint4 *p = reinterpret_cast<const uint4 *>(tile + (at - m));
    const uint4 a = p[0];
    if (m == 0) return a;
    return funnel_shift16(a, p[1], m);
}

// 16 bytes of shared memory from any byte address, as five aligned words funnel-shifted into four: no
// branch on the misalignment, so the lanes of a warp may each have their own.  Reads the words that cover
// [at, at + 16), i.e. up to 3 bytes before `at` and up to 4 bytes past at + 16.
__device__ __forceinline__ uint4 lds_unaligned16(const unsigned char *tile, uint32_t at)
{
    const uint32_t bs = (at & 3u) * 8u;
    const uint32_t *w = reinterpret_cast<const uint32_t *>(tile + (at & ~3u));
    const uint32_t w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3], w4 = w[4];
    uint4 o;
    o.x = __funnelshift_r(w0, w1, bs);
    o.y = __funnelshift_r(w1, w2, bs);
    o.z = __funnelshift_r(w2, w3, bs);
    o.w = __funnelshift_r(w3, w4, bs);
    return o;
}

template <int NT>
__device__ __forceinline__ void ragged_bulk_body(const CopyParams<NT> &P)
{
    extern __shared__ __align__(128) unsigned char tile[];
    __shared__ RowEntry rowtab[kRaggedBulkRows];
    __shared__ RaggedRow rinfo[kRaggedBulkRows];
    __shared__ __align__(8) unsigned long long mbar_storage;
    __shared__ unsigned int wait_failed;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t fanout = g.fanout;
    const uint32_t len = uint32_t(g.run_bytes);       // chunk mode with col blocks: runs below 2^32 bytes here
    const uint32_t cpb = g.per_block;
    const uint32_t pitch = g.stage_pitch;
    const uint32_t mbar = smem_addr(&mbar_storage);
    const uint32_t item = blockIdx.x;                 // one item per block (the mbarrier is used once)
    if (item >= g.n_items) return;
    const BoxBase b = decode_box(P, item);
    const uint32_t group = fdiv(b.part, g.col_blocks);
    const uint32_t cb = b.part - group * g.col_blocks.d;
    const bool first = cb == 0, last = cb + 1 == g.col_blocks.d;
    const uint32_t c0 = cb * cpb;
    const uint32_t row0 = group * g.rows_per_item;
    const uint32_t nr = min(g.rows_per_item, g.rows - row0);
    if (tid == 0) {
        wait_failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(nr) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    wait_for_previous_kernel();
    for (uint32_t r = tid; r < nr && CHK_IDX(r, uint32_t(kRaggedBulkRows)); r += kBlockThreads) {
        RowEntry e;
        row_offsets(g, row0 + r, e.s1, e.s2, int(g.n_row_tab));
        rowtab[r] = e;
        uint32_t head, chunks;
        split_run(len, b.o2 + e.s2, head, chunks);
        // row-relative source bytes [b0, b1) belong to this column block
        const uint32_t b0 = first ? 0u : min(len, head + (c0 << 4));
        const uint32_t b1 = last ? len : min(len, head + ((c0 + cpb) << 4));
        const char *src = b.sbase + e.s1 + b0;
        const uint32_t m = uint32_t(reinterpret_cast<uintptr_t>(src)) & 15u;
        RaggedRow ri;
        ri.base = r * pitch + m - b0;                 // unsigned wrap-around is intended: base + x is used for x >= b0
        ri.head = head;
        ri.chunks = chunks;
        ri.pad = 0;
        rinfo[r] = ri;
        if (b1 > b0) {
            const uint32_t bytes = (m + (b1 - b0) + 15u) & ~15u;
            const bool safe = CHK_SRC(P, src - m, bytes) && CHK_SMEM(r * pitch, bytes);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(mbar), "r"((safe ? bytes : 0u) + (r == 0 ? g.test_extra_tx : 0u)) : "memory");
            if (safe)
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_addr(tile) + r * pitch), "l"(src - m), "r"(bytes), "r"(mbar)
                             : "memory");
        } else if (r == 0 && g.test_extra_tx != 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(g.test_extra_tx) : "memory");
        } else {
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
        }
    }
    __syncthreads();
    if (!mbar_wait_bounded(mbar, 0, g.wait_polls)) {
        bulk_wait_ran_out(mbar, &wait_failed, g.wait_polls);
        return;
    }
    // The lanes work in groups of g.lanes (a power of two, at least a warp); the groups share out the rows
    // of the item and a lane strides through its row's chunks.  Everything that depends on the row -- the
    // shift, the places in shared memory and in the target -- is computed once per row, and the lanes of a
    // warp take the same shift path.  Fan-out 1: the target address is kept in a register (the pointer
    // table is read through generic loads, which the stores of the loop would otherwise order behind them).
    // (Measured: +5..7 % at fan-out 1; with more replicas the flat walk below is 5-12 % faster.)
    const uint32_t W = g.lanes;
    const uint32_t n_groups = kBlockThreads / W;
    const uint32_t lane = tid & (W - 1u);
    for (uint32_t r = tid / W; r < nr && fanout == 1; r += n_groups) {
        const RaggedRow ri = rinfo[r];
        if (ri.chunks <= c0) continue;
        const uint32_t n_here = min(ri.chunks - c0, cpb);
        const uint32_t x0 = ri.head + (c0 << 4);          // row-relative byte of the first chunk of this block
        const uint32_t at0 = ri.base + x0;
        const uint32_t m = at0 & 15u;
        const uint4 *p = reinterpret_cast<const uint4 *>(tile + (at0 - m));
        char *const d_only = b.dtab[0] + (b.o2 + rowtab[r].s2 + x0);
        for (uint32_t jj = lane; jj < n_here; jj += W) {
            if (!CHK_SMEM(at0 - m + (jj << 4), m != 0 ? 32u : 16u)) continue;
            const uint4 a = p[jj];
            const uint4 o = m != 0 ? funnel_shift16(a, p[jj + 1u], m) : a;
            if (CHK_DST(P, d_only + (jj << 4), 16)) st_stream(reinterpret_cast<uint4 *>(d_only + (jj << 4)), o);
        }
    }
    // several replicas: flat walk over (row, chunk)
    for (uint32_t idx = tid; idx < nr * cpb && fanout != 1; idx += kBlockThreads) {
        const uint32_t r = fdiv(idx, g.per_block_div);
        const uint32_t j = c0 + (idx - r * cpb);
        const RaggedRow ri = rinfo[r];
        if (j < ri.chunks) {
            const uint32_t x = ri.head + (j << 4);
            if (!CHK_SMEM(((ri.base + x) & ~15u), ((ri.base + x) & 15u) ? 32u : 16u)) continue;
            const uint4 v = lds_shifted(tile, ri.base + x);
            const int64_t doff = b.o2 + rowtab[r].s2 + x;
            for (uint32_t f = 0; f < fanout; ++f)
                if (CHK_DST(P, b.dtab[f] + doff, 16)) st_stream(reinterpret_cast<uint4 *>(b.dtab[f] + doff), v);
        }
    }
    // ragged ends out of shared memory: head with the first column block, tail with the last
    const uint32_t unit = g.unit_bytes;
    const uint32_t slots = 16u / unit - 1u;
    const uint32_t ends = (first ? 1u : 0u) + (last ? 1u : 0u);
    for (uint32_t idx = tid; idx < nr * slots * ends; idx += kBlockThreads) {
        const uint32_t r = idx / (slots * ends);
        const uint32_t w = idx - r * (slots * ends);
        const bool is_head = first && w < slots;
        const uint32_t slot = is_head ? w : (first ? w - slots : w);
        const RaggedRow ri = rinfo[r];
        const uint32_t toff = ri.head + (ri.chunks << 4);
        const uint32_t count = is_head ? ri.head / unit : (len - toff) / unit;
        if (slot < count) {
            const uint32_t x = (is_head ? 0u : toff) + slot * unit;
            if (!CHK_SMEM(ri.base + x, unit)) continue;
            const unsigned char *sp = tile + (ri.base + x);
            const int64_t doff = b.o2 + rowtab[r].s2 + x;
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dp = b.dtab[f] + doff;
                if (!CHK_DST(P, dp, unit)) continue;
                switch (unit) {
                case 8: *reinterpret_cast<uint2 *>(dp) = *reinterpret_cast<const uint2 *>(sp); break;
                case 4: *reinterpret_cast<uint32_t *>(dp) = *reinterpret_cast<const uint32_t *>(sp); break;
                case 2: *reinterpret_cast<uint16_t *>(dp) = *reinterpret_cast<const uint16_t *>(sp); break;
                default: *reinterpret_cast<uint8_t *>(dp) = *sp; break;
                }
            }
        }
    }
}

// ---- kModeZip: m source streams <-> one target stream, through shared memory ---------------------
// One item per block.  Table row r of the item and rows [a, a + cnt) of the zipped digit: the source
// bytes are m segments of cnt runs (long target rows: one per source tile) or one segment of cnt long
// rows (long source rows).  One thread per segment posts its byte count and issues the bulk copy of
// the covering 16-byte blocks; segbase[] remembers where byte 0 of the segment sits in shared memory.
// Then the target ranges -- one per table row, or one per (table row, target tile) -- are written in
// target-aligned 16-byte chunks assembled unit by unit from shared memory, ends in single units.
// The kernel is bound by instruction issue, so the map from a chunk to the places of its units is made
// cheap in one of three ways picked on the host (periodic walk, by-range walk, tabulated places; see
// the branches of zip_body), with a flat walk of two divisions per unit as the fallback.
template <bool LONG_DST, typename T, int NT>
__device__ __forceinline__ const T *zip_src(const CopyGeometry &g, const unsigned char *tile, const uint32_t *segbase,
                                            uint32_t r, uint32_t j, uint32_t x)
{
    const uint32_t xu = x / uint32_t(sizeof(T));
    const uint32_t k = fdiv(xu, g.units_per_run);            // run number inside the range
    const uint32_t w = (xu - k * g.units_per_run.d) * uint32_t(sizeof(T));
    const uint32_t run = uint32_t(g.run_bytes);
    uint32_t at;
    if (LONG_DST) {
        const uint32_t rr = fdiv(k, g.gl_m);
        const uint32_t jj = k - rr * g.gl_m.d;
        at = segbase[r * g.gl_m.d + jj] + rr * run + w;
    } else {
        at = segbase[r] + (k * g.gl_m.d + j) * run + w;
    }
    return reinterpret_cast<const T *>(tile + at);
}

template <bool LONG_DST, typename T, int NT>
__device__ __forceinline__ void zip_body(const CopyParams<NT> &P, unsigned char *tile, RowEntry *rowtab,
                                         uint32_t *segbase, uint32_t mbar, unsigned int *wait_failed)
{
    constexpr int kPer = 16 / int(sizeof(T));
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t nthreads = blockDim.x;             // 128 or 256, chosen at launch
    const uint32_t fanout = g.fanout;
    const uint32_t m = g.gl_m.d;
    const uint32_t run = uint32_t(g.run_bytes);
    const uint32_t nseg = LONG_DST ? m : 1u;
    const uint32_t nrng = LONG_DST ? 1u : m;              // target ranges per table row
    const uint32_t item = blockIdx.x;
    if (item >= g.n_items) return;
    const BoxBase b = decode_box(P, item);
    const uint32_t group = fdiv(b.part, g.col_blocks);
    const uint32_t cb = b.part - group * g.col_blocks.d;
    const uint32_t row0 = group * g.rows_per_item;
    const uint32_t nr = min(g.rows_per_item, g.rows - row0);
    const uint32_t a = cb * g.per_block;
    const uint32_t cnt = min(g.per_block, g.tab_inner.d - a);
    const uint32_t seg_bytes = cnt * run * (LONG_DST ? 1u : m);
    const uint32_t rng_bytes = cnt * run * (LONG_DST ? m : 1u);
    if (tid == 0) {
        *wait_failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(nr * nseg) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    wait_for_previous_kernel();
    for (uint32_t t = tid; t < nr * nseg && CHK_IDX(t, uint32_t(kZipSegments)); t += nthreads) {
        const uint32_t r = fdiv(t, g.gl_m);
        const uint32_t j = LONG_DST ? t - r * m : 0u;
        const uint32_t rr = LONG_DST ? r : t;
        RowEntry e;
        row_offsets(g, row0 + rr, e.s1, e.s2, int(g.n_row_tab));
        if (j == 0) rowtab[rr] = e;
        const char *src = LONG_DST ? P.src[b.t1 + j * g.gl_ts] + b.o1 + e.s1 + int64_t(a) * run
                                   : b.sbase + e.s1 + int64_t(a) * run * m;
        const uint32_t mis = uint32_t(reinterpret_cast<uintptr_t>(src)) & 15u;
        const uint32_t slot = t * g.zip_seg_pitch;
        segbase[t] = slot + mis;
        const uint32_t bytes = (mis + seg_bytes + 15u) & ~15u;
        const bool safe = CHK_SRC(P, src - mis, bytes) && CHK_SMEM(slot, bytes);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     ::"r"(mbar), "r"((safe ? bytes : 0u) + (t == 0 ? g.test_extra_tx : 0u)) : "memory");
        if (safe)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(tile) + slot), "l"(src - mis), "r"(bytes), "r"(mbar)
                         : "memory");
    }
    // short ranges: while the copies are in flight, tabulate for every unit position of a range where
    // the unit sits -- which segment of its table row (upper bits) and at which byte of it (lower 20 bits)
    uint32_t *lut = reinterpret_cast<uint32_t *>(tile + size_t(g.stage_pitch) * g.rows_per_item);
    for (uint32_t u = tid; u < g.zip_lut_units; u += nthreads) {
        if (!CHK_SMEM(g.stage_pitch * g.rows_per_item + u * 4u, 4u)) continue;
        const uint32_t k = fdiv(u, g.units_per_run);
        const uint32_t w = (u - k * g.units_per_run.d) * uint32_t(sizeof(T));
        if (LONG_DST) {
            const uint32_t rr = fdiv(k, g.gl_m);
            lut[u] = ((k - rr * m) << 20) | (rr * run + w);
        } else {
            lut[u] = k * m * run + w;
        }
    }
    __syncthreads();
    if (!mbar_wait_bounded(mbar, 0, g.wait_polls)) {
        bulk_wait_ran_out(mbar, wait_failed, g.wait_polls);
        return;
    }
    // whole chunks of the target ranges
    const uint32_t slots = g.zip_slots.d;
    const uint32_t total = nr * nrng * slots;
    if (g.zip_lut_units != 0) {
        // flat walk over (range, chunk); a unit costs a table read, the read of its segment's base and the
        // read of the unit itself
        for (uint32_t idx = tid; idx < total; idx += nthreads) {
            uint32_t r, c, j = 0;
            if (LONG_DST) {
                r = fdiv(idx, g.zip_slots);
                c = idx - r * slots;
            } else if (g.zip_tile_fastest) {
                const uint32_t t = fdiv(idx, g.gl_m);
                j = idx - t * m;
                r = fdiv(t, g.zip_slots);
                c = t - r * slots;
            } else {
                const uint32_t q = fdiv(idx, g.zip_slots);
                c = idx - q * slots;
                r = fdiv(q, g.gl_m);
                j = q - r * m;
            }
            const int64_t d0 = b.o2 + rowtab[r].s2 + int64_t(a) * (LONG_DST ? run * m : run);
            uint32_t head, chunks;
            split_run(rng_bytes, d0, head, chunks);
            if (c < chunks) {
                const uint32_t x = head + (c << 4);
                const uint32_t u0 = x / uint32_t(sizeof(T));
                const uint32_t sb = LONG_DST ? 0u : segbase[r] + j * run;
                union {
                    uint4 v;
                    T t[kPer];
                } u;
#pragma unroll
                for (int i = 0; i < kPer; ++i) {
                    const uint32_t e = CHK_IDX(u0 + uint32_t(i), g.zip_lut_units) ? lut[u0 + uint32_t(i)] : 0u;
                    const uint32_t at = LONG_DST ? segbase[r * m + (e >> 20)] + (e & 0xfffffu) : sb + e;
                    u.t[i] = CHK_SMEM(at, uint32_t(sizeof(T))) ? *reinterpret_cast<const T *>(tile + at) : T();
                }
                for (uint32_t f = 0; f < fanout; ++f) {
                    char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + j * g.gl_ts) * fanout + f];
                    if (CHK_DST(P, dbase + d0 + x, 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d0 + x), u.v);
                }
            }
        }
    } else
    if (g.zip_period.d != 0) {
        // periodic walk (same branch for every thread): the map from a target chunk to the shared-memory
        // places of its units repeats every zip_period chunks, shifted by a whole number of rows.  A thread
        // decodes the units of its first chunk once per table row and then strides through the range -- and,
        // with long source rows, through the m target tiles -- in steps of S chunks, a multiple of the
        // period: every further chunk costs one add per unit, the unit reads and the stores.
        // Long source rows of very short runs: a thread stays with one target tile (tid mod m), so that
        // neighbouring lanes read neighbouring units of the staged long row; otherwise it takes the tiles in turn.
        uint32_t tl = tid, width = nthreads, jb = 0, jn = nrng;
        if (!LONG_DST && g.zip_tile_fastest) {
            tl = fdiv(tid, g.gl_m);
            jb = tid - tl * m;
            jn = 1;
            width = fdiv(nthreads, g.gl_m);
        }
        // The lanes are split into groups of S (a multiple of the period, at most zip_width: a few chunks of
        // a range per lane); the groups share out the table rows of the item.
        const uint32_t S = min(fdiv(width, g.zip_period) * g.zip_period.d, g.zip_width);
        const uint32_t step = fdiv(S, g.zip_period) * g.zip_period_rows * (LONG_DST ? run : run * m);
        const uint32_t n_groups = width / S;
        const uint32_t grp = tl / S;
        tl -= grp * S;
        // An item with fewer table rows than groups (one row of 46 runs for 16 target tiles, say) would leave
        // most groups without work: the groups then share out (table row, target tile) pairs instead
        // (measured: +1 to +13 % on 40 launches, once +41 %; not from fan-out 8, where the stores of
        // more lanes at once to eight and more replicas cost 1-6 %).
        const bool by_pair = nr < n_groups && jn > 1 && fanout < 8u;   // (jn > 1 means jn == m)
        const uint32_t n_work = by_pair ? nr * jn : nr;
        for (uint32_t q = grp; q < n_work && grp < n_groups; q += n_groups) {
            uint32_t r = q, j0 = jb, j1 = jb + jn;
            if (by_pair) {
                r = fdiv(q, g.gl_m);
                j0 = jb + (q - r * m);
                j1 = j0 + 1u;
            }
            const int64_t d0 = b.o2 + rowtab[r].s2 + int64_t(a) * (LONG_DST ? run * m : run);
            uint32_t head, chunks;
            split_run(rng_bytes, d0, head, chunks);
            uint32_t at[kPer];
#pragma unroll
            for (int i = 0; i < kPer; ++i)
                at[i] = uint32_t(reinterpret_cast<const unsigned char *>(zip_src<LONG_DST, T, NT>(
                                     g, tile, segbase, r, jb, head + (tl << 4) + uint32_t(i * sizeof(T)))) - tile);
            for (uint32_t j = j0; j < j1; ++j) {
                uint32_t o = (j - jb) * run;
                // fan-out 1: the target address is kept in a register (the pointer tables are read through
                // generic loads, which the stores of the loop would otherwise order behind them)
                char *const *dt = LONG_DST ? b.dtab : &P.dst[(b.t2 + j * g.gl_ts) * fanout];
                char *d_first = dt[0] + d0 + head;
                for (uint32_t c = tl; c < chunks; c += S, o += step) {
                    union {
                        uint4 v;
                        T t[kPer];
                    } u;
#pragma unroll
                    for (int i = 0; i < kPer; ++i)
                        u.t[i] = CHK_SMEM(at[i] + o, uint32_t(sizeof(T))) ? *reinterpret_cast<const T *>(tile + (at[i] + o)) : T();
                    if (fanout == 1) {
                        if (CHK_DST(P, d_first + (c << 4), 16)) st_stream(reinterpret_cast<uint4 *>(d_first + (c << 4)), u.v);
                    } else {
                        for (uint32_t f = 0; f < fanout; ++f)
                            if (CHK_DST(P, dt[f] + d0 + head + (c << 4), 16))
                                st_stream(reinterpret_cast<uint4 *>(dt[f] + d0 + head + (c << 4)), u.v);
                    }
                }
            }
        }
    } else if (g.zip_cpr.d != 0) {
        // long ranges of runs of 32 bytes and more (same branch for every thread): the block goes through
        // the ranges one after the other; a thread keeps its chunk number inside a run (ci) and walks down
        // the runs k, k + kstep, ... of the range, so everything that depends on the range is computed
        // once and a chunk costs a few multiply-adds, the unit reads and the stores
        const uint32_t cpr = g.zip_cpr.d;
        const uint32_t kstep = fdiv(nthreads, g.zip_cpr);
        const uint32_t kk = fdiv(tid, g.zip_cpr);
        const uint32_t ci = tid - kk * cpr;
        const uint32_t nruns = cnt * (LONG_DST ? m : 1u);
        for (uint32_t q = 0; q < nr * nrng && kk < kstep; ++q) {
            const uint32_t r = LONG_DST ? q : fdiv(q, g.gl_m);
            const uint32_t j = LONG_DST ? 0u : q - r * m;
            const int64_t d0 = b.o2 + rowtab[r].s2 + int64_t(a) * (LONG_DST ? run * m : run);
            const uint32_t d0lo = uint32_t(d0);
            const uint32_t sb = LONG_DST ? 0u : segbase[r] + j * run;
            for (uint32_t k = kk; k < nruns; k += kstep) {
                const uint32_t xs = k * run;
                const uint32_t x = xs + ((16u - ((d0lo + xs) & 15u)) & 15u) + (ci << 4);
                if (x < xs + run && x + 16u <= rng_bytes) {
                    uint32_t base0, base1;      // shared-memory address of target byte p: base + p
                    if (LONG_DST) {
                        const uint32_t rr = fdiv(k, g.gl_m);
                        const uint32_t jj = k - rr * m;
                        const bool wrap = jj + 1u == m;
                        base0 = segbase[r * m + jj] + rr * run - xs;
                        base1 = segbase[r * m + (wrap ? 0u : jj + 1u)] + (wrap ? rr + 1u : rr) * run - (xs + run);
                    } else {
                        base0 = sb + k * (m - 1u) * run;    // segbase[r] + (k * m + j) * run - xs
                        base1 = base0 + (m - 1u) * run;
                    }
                    union {
                        uint4 v;
                        T t[kPer];
                    } u;
#pragma unroll
                    for (int i = 0; i < kPer; ++i) {
                        const uint32_t p = x + uint32_t(i * sizeof(T));
                        const uint32_t at = (p >= xs + run ? base1 : base0) + p;
                        u.t[i] = CHK_SMEM(at, uint32_t(sizeof(T))) ? *reinterpret_cast<const T *>(tile + at) : T();
                    }
                    for (uint32_t f = 0; f < fanout; ++f) {
                        char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + j * g.gl_ts) * fanout + f];
                        if (CHK_DST(P, dbase + d0 + x, 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d0 + x), u.v);
                    }
                }
            }
        }
    } else
    for (uint32_t idx = tid; idx < total; idx += nthreads) {
        // long source rows of very short runs: neighbouring lanes take the same chunk of neighbouring
        // target tiles, whose units are neighbours in the staged long row (no bank conflicts); with
        // longer runs neighbouring lanes stay in one run and in one target tile (wider stores)
        uint32_t r, c, j = 0;
        if (LONG_DST) {
            r = fdiv(idx, g.zip_slots);
            c = idx - r * slots;
        } else if (g.zip_tile_fastest) {
            const uint32_t t = fdiv(idx, g.gl_m);
            j = idx - t * m;
            r = fdiv(t, g.zip_slots);
            c = t - r * slots;
        } else {
            const uint32_t q = fdiv(idx, g.zip_slots);
            c = idx - q * slots;
            r = fdiv(q, g.gl_m);
            j = q - r * m;
        }
        const int64_t d0 = b.o2 + rowtab[r].s2 + int64_t(a) * (LONG_DST ? run * m : run);
        uint32_t head, chunks;
        split_run(rng_bytes, d0, head, chunks);
        if (c < chunks) {
            const uint32_t x = head + (c << 4);
            union {
                uint4 v;
                T t[kPer];
            } u;
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const T *sp = zip_src<LONG_DST, T, NT>(g, tile, segbase, r, j, x + uint32_t(i * sizeof(T)));
                u.t[i] = CHK_SMEM(uint32_t(reinterpret_cast<const unsigned char *>(sp) - tile), uint32_t(sizeof(T))) ? *sp : T();
            }
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + j * g.gl_ts) * fanout + f];
                if (CHK_DST(P, dbase + d0 + x, 16)) st_stream(reinterpret_cast<uint4 *>(dbase + d0 + x), u.v);
            }
        }
    }
    // ragged ends of the ranges, unit by unit
    constexpr uint32_t kSlots = 16u / uint32_t(sizeof(T)) - 1u;
    if constexpr (kSlots > 0) {
        for (uint32_t idx = tid; idx < nr * nrng * kSlots * 2u; idx += nthreads) {
            const uint32_t q = idx / (kSlots * 2u);
            const uint32_t w = idx - q * (kSlots * 2u);
            const bool is_head = w < kSlots;
            const uint32_t slot = is_head ? w : w - kSlots;
            const uint32_t r = LONG_DST ? q : fdiv(q, g.gl_m);
            const uint32_t j = LONG_DST ? 0u : q - r * m;
            const int64_t d0 = b.o2 + rowtab[r].s2 + int64_t(a) * (LONG_DST ? run * m : run);
            uint32_t head, chunks;
            split_run(rng_bytes, d0, head, chunks);
            const uint32_t toff = head + (chunks << 4);
            const uint32_t count = (is_head ? head : rng_bytes - toff) / uint32_t(sizeof(T));
            if (slot < count) {
                const uint32_t x = (is_head ? 0u : toff) + slot * uint32_t(sizeof(T));
                const T *sp = zip_src<LONG_DST, T, NT>(g, tile, segbase, r, j, x);
                if (!CHK_SMEM(uint32_t(reinterpret_cast<const unsigned char *>(sp) - tile), uint32_t(sizeof(T)))) continue;
                const T val = *sp;
                for (uint32_t f = 0; f < fanout; ++f) {
                    char *dbase = LONG_DST ? b.dtab[f] : P.dst[(b.t2 + j * g.gl_ts) * fanout + f];
                    if (CHK_DST(P, dbase + d0 + x, uint32_t(sizeof(T)))) *reinterpret_cast<T *>(dbase + d0 + x) = val;
                }
            }
        }
    }
}

#define REDIST_DEFINE_ZIP_KERNEL(NAME)                                                               \
    template <bool LONG_DST, int NT, bool SMALL>                                                     \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P)  \
    {                                                                                                \
        extern __shared__ __align__(128) unsigned char tile[];                                       \
        __shared__ RowEntry rowtab[kZipSegments];                                                    \
        __shared__ uint32_t segbase[kZipSegments];                                                   \
        __shared__ __align__(8) unsigned long long mbar_storage;                                     \
        __shared__ unsigned int wait_failed;                                                         \
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");                              \
        const uint32_t mbar = smem_addr(&mbar_storage);                                              \
        if constexpr (SMALL) {                                                                       \
            if (P.g.unit_bytes == 2)                                                                 \
                zip_body<LONG_DST, uint16_t, NT>(P, tile, rowtab, segbase, mbar, &wait_failed);      \
            else                                                                                     \
                zip_body<LONG_DST, uint8_t, NT>(P, tile, rowtab, segbase, mbar, &wait_failed);       \
        } else {                                                                                     \
            switch (P.g.unit_bytes) {                                                                \
            case 16: zip_body<LONG_DST, uint4, NT>(P, tile, rowtab, segbase, mbar, &wait_failed); break; \
            case 8: zip_body<LONG_DST, uint2, NT>(P, tile, rowtab, segbase, mbar, &wait_failed); break; \
            default: zip_body<LONG_DST, uint32_t, NT>(P, tile, rowtab, segbase, mbar, &wait_failed); break; \
            }                                                                                        \
        }                                                                                            \
    }

REDIST_DEFINE_ZIP_KERNEL(redist_dynslice_zip_kernel)
REDIST_DEFINE_ZIP_KERNEL(redist_alltoall_zip_kernel)
REDIST_DEFINE_ZIP_KERNEL(redist_allgather_zip_kernel)
REDIST_DEFINE_ZIP_KERNEL(redist_allpermute_zip_kernel)
REDIST_DEFINE_ZIP_KERNEL(redist_fused_zip_kernel)

// ---- kModeBox: super-box items, several interleaving dimensions at once -------------------------
// One item per block: rows_per_item outer rows times per_block rows (of the dimension K outside the inner
// ones) of one super-box.  Source side, per outer row: bx_nseg segments, one per source tile the
// super-box touches, each cnt * bx_s1 contiguous bytes at the same offset inside its tile (so the segments
// of a row share one misalignment), brought into shared memory at a uniform pitch by one bulk copy each.
// Target side, per outer row: bx_nrng ranges, one per target tile, each cnt * bx_s2 contiguous bytes at
// the same offset inside its tile.  The place in shared
// memory of the unit at byte x of range t is
//     base[t] + (x / bx_s2) * bx_s1 + place[(x % bx_s2) / unit]
// base[t]: where the target tile's corner lies (segment and offset inside the segment's row), place[]:
// where a position inside one target row lies relative to that corner.  Both are sums over the inner
// dimensions of (index / source tile extent) * segment step * pitch + (index % source tile extent) *
// byte stride, which is additive in "corner index + index inside the tile" because in every inner
// dimension one tile extent divides the other.  The block tabulates place[] (one target row) and base[]
// while its copies are in flight; a unit then costs a table read and the read of the unit.
// The kernel is bound by instruction issue, not by memory, so work that every thread would repeat is
// given to one warp: warp 0 alone decodes the item (unit digits -> tiles and offsets), issues the bulk
// copies and tabulates base[] and the range offsets, while the other warps tabulate place[]; the walk
// over the ranges then reads everything item-specific from those tables.  Lanes work in groups of
// zip_width (a power of two) that share out the ranges; a lane strides through its range's chunks and
// keeps (row, position in row) by adding a constant per step instead of dividing.  The host picks the
// width: a warp or more per range as a rule, fewer lanes -- several ranges per warp -- where the units of
// one range would all fall into a few shared-memory banks.
// PIECE (units of 1 and 2 bytes on runs of 64 bytes and more, a kernel of its own): a chunk that lies inside
// one run -- contiguous on both sides -- is read as one unaligned 16-byte piece instead of 8 or 16 units
// (measured on the super-box launches of the 1-byte sweep 1.2-1.3x, of the 2-byte sweep 1.0-1.1x; the same in
// the zip kernels measured 0.93-0.98x and is not built).
template <typename T, int NT, bool PIECE>
__device__ __forceinline__ void box_body(const CopyParams<NT> &P, unsigned char *tile, uint32_t *base_of,
                                         uint32_t *tile_of, int64_t *row_d0, uint32_t mbar, unsigned int *wait_failed)
{
    constexpr int kPer = 16 / int(sizeof(T));
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t nthreads = blockDim.x;
    const uint32_t fanout = g.fanout;
    const uint32_t item = blockIdx.x;
    if (item >= g.n_items) return;
    // which part of its box the item is (cheap, every thread): group of outer rows, block of rows of K
    const uint32_t slow = fdiv(item, g.items_per_box);           // inner_n = fast_boxes = 1 in this mode
    const uint32_t part = item - slow * g.items_per_box.d;
    const uint32_t group = fdiv(part, g.col_blocks);
    const uint32_t cb = part - group * g.col_blocks.d;
    const uint32_t row0 = group * g.rows_per_item;
    const uint32_t nr = min(g.rows_per_item, g.rows - row0);
    const uint32_t a = cb * g.per_block;                       // first row of dimension K
    const uint32_t cnt = min(g.per_block, g.tab_inner.d - a);
    const uint32_t s1 = g.bx_s1, s2 = g.bx_s2.d;
    const uint32_t nseg = g.bx_nseg, nrng = g.bx_nrng;
    const uint32_t pitch = g.zip_seg_pitch;
    const uint32_t seg_bytes = cnt * s1, rng_bytes = cnt * s2;
    const uint32_t row_units = g.zip_lut_units;
    uint16_t *place = reinterpret_cast<uint16_t *>(tile + size_t(g.stage_pitch) * g.rows_per_item);
    if (tid == 0) {
        *wait_failed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(nr * nseg) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid < 32u) {
        const BoxBase b = decode_box(P, item);
        wait_for_previous_kernel();
        // one lane per source segment: (outer row, source tile of the super-box)
        for (uint32_t t = tid; t < nr * nseg && CHK_IDX(t, uint32_t(kBoxSegments)); t += 32u) {
            const uint32_t r = fdiv(t, g.bx_nseg_div);
            uint32_t rem = t - r * nseg, t1 = b.t1;
            for (int q = int(g.bx_n) - 1; q >= 0; --q) {
                const uint32_t nx = fdiv(rem, g.bx_n1[q]);
                t1 += (rem - nx * g.bx_n1[q].d) * g.bx_ts1[q];
                rem = nx;
            }
            int64_t r1, r2;
            row_offsets(g, row0 + r, r1, r2, int(g.n_row_tab));
            const int64_t so = b.o1 + r1 + int64_t(a) * s1;      // offset of the row's segments inside their source tiles
            const uint32_t mis = uint32_t(so) & 15u;             // (tiles start on 16-byte boundaries)
            const char *src = P.src[t1] + so;
            const uint32_t bytes = (mis + seg_bytes + 15u) & ~15u;
            const bool safe = CHK_SRC(P, src - mis, bytes) && CHK_SMEM(t * pitch, bytes);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(mbar), "r"((safe ? bytes : 0u) + (t == 0 ? g.test_extra_tx : 0u)) : "memory");
            if (safe)
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_addr(tile) + t * pitch), "l"(src - mis), "r"(bytes), "r"(mbar)
                             : "memory");
        }
        // the corner of every target tile in every outer row, and where every outer row's ranges start
        for (uint32_t t = tid; t < nr * nrng && CHK_IDX(t, uint32_t(kBoxSegments)); t += 32u) {
            const uint32_t r = fdiv(t, g.bx_nrng_div);
            const uint32_t tt = t - r * nrng;
            int64_t r1, r2;
            row_offsets(g, row0 + r, r1, r2, int(g.n_row_tab));
            const uint32_t mis = uint32_t(b.o1 + r1 + int64_t(a) * s1) & 15u;
            uint32_t rem = tt, t2 = b.t2, off = r * g.stage_pitch + mis;
            for (int q = int(g.bx_n) - 1; q >= 0; --q) {
                const uint32_t nx = fdiv(rem, g.bx_n2[q]);
                const uint32_t d = rem - nx * g.bx_n2[q].d;
                rem = nx;
                t2 += d * g.bx_ts2[q];
                const uint32_t x = d * g.bx_c2[q].d;             // index of the tile's corner inside the super-box
                const uint32_t hi = fdiv(x, g.bx_c1[q]);
                off += hi * g.bx_seg[q] * pitch + (x - hi * g.bx_c1[q].d) * g.bx_st1[q];
            }
            base_of[t] = off;
            if (r == 0) tile_of[tt] = t2 * fanout;
            if (tt == 0 && CHK_IDX(r, uint32_t(kBoxRows))) row_d0[r] = b.o2 + r2 + int64_t(a) * s2;
        }
    } else {
        // the place of every unit position of one target row (depends on the launch only)
        for (uint32_t p = tid - 32u; p < row_units; p += nthreads - 32u) {
            uint32_t rest = fdiv(p, g.bx_trail);
            uint32_t off = (p - rest * g.bx_trail.d) * uint32_t(sizeof(T));
            for (int q = int(g.bx_n) - 1; q >= 0; --q) {
                const uint32_t nx = fdiv(rest, g.bx_c2[q]);
                const uint32_t i = rest - nx * g.bx_c2[q].d;
                rest = nx;
                const uint32_t hi = fdiv(i, g.bx_c1[q]);
                off += hi * g.bx_seg[q] * pitch + (i - hi * g.bx_c1[q].d) * g.bx_st1[q];
            }
            if (CHK_SMEM(g.stage_pitch * g.rows_per_item + p * 2u, 2u)) place[p] = uint16_t(off);
        }
        wait_for_previous_kernel();
    }
    __syncthreads();
    if (!mbar_wait_bounded(mbar, 0, g.wait_polls)) {
        bulk_wait_ran_out(mbar, wait_failed, g.wait_polls);
        return;
    }
    // whole chunks: groups of W lanes share out the ranges (outer row, target tile)
    const uint32_t W = g.zip_width;                              // power of two, 1 .. block size
    const uint32_t n_groups = nthreads / W;
    const uint32_t lane = tid & (W - 1u);
    const uint32_t step_units = W * uint32_t(kPer);              // units between a lane's consecutive chunks
    const uint32_t dj = fdiv(step_units, g.bx_row_units_div);
    const uint32_t dp = step_units - dj * row_units;
    for (uint32_t q = tid / W; q < nr * nrng; q += n_groups) {
        const uint32_t r = fdiv(q, g.bx_nrng_div);
        const int64_t d0 = row_d0[r];
        uint32_t head, chunks;
        split_run(rng_bytes, d0, head, chunks);
        if (lane >= chunks) continue;
        char *const *dt = &P.dst[tile_of[q - r * nrng]];
        char *d_first = dt[0] + d0 + head;
        const uint32_t base = base_of[q];
        const uint32_t x0 = head + (lane << 4);
        uint32_t j = fdiv(x0, g.bx_s2);
        uint32_t p = (x0 - j * s2) / uint32_t(sizeof(T));
        for (uint32_t c = lane; c < chunks; c += W) {
            const uint32_t at = base + j * s1;
            union {
                uint4 v;
                T t[kPer];
            } u;
            bool one_piece = false;
            if constexpr (PIECE) {
                const uint32_t in_run = p - fdiv(p, g.bx_trail) * g.bx_trail.d;
                one_piece = in_run + uint32_t(kPer) <= g.bx_trail.d;
                if (one_piece) {
                    const uint32_t w = at + place[p];
                    if (CHK_SMEM(w & ~3u, 20u)) u.v = lds_unaligned16(tile, w);
                }
            }
            if (one_piece) {
            } else if (p + uint32_t(kPer) <= row_units) {
#pragma unroll
                for (int i = 0; i < kPer; ++i) {
                    const uint32_t w = at + place[p + uint32_t(i)];
                    u.t[i] = CHK_SMEM(w, uint32_t(sizeof(T))) ? *reinterpret_cast<const T *>(tile + w) : T();
                }
            } else {
                uint32_t pp = p, aa = at;                        // the chunk runs over the end of a row of K
#pragma unroll
                for (int i = 0; i < kPer; ++i) {
                    if (pp == row_units) {
                        pp = 0;
                        aa += s1;
                    }
                    const uint32_t w = aa + place[pp];
                    u.t[i] = CHK_SMEM(w, uint32_t(sizeof(T))) ? *reinterpret_cast<const T *>(tile + w) : T();
                    ++pp;
                }
            }
            if (fanout == 1) {
                if (CHK_DST(P, d_first + (c << 4), 16)) st_stream(reinterpret_cast<uint4 *>(d_first + (c << 4)), u.v);
            } else {
                for (uint32_t f = 0; f < fanout; ++f)
                    if (CHK_DST(P, dt[f] + d0 + head + (c << 4), 16))
                        st_stream(reinterpret_cast<uint4 *>(dt[f] + d0 + head + (c << 4)), u.v);
            }
            p += dp;
            j += dj;
            if (p >= row_units) {
                p -= row_units;
                ++j;
            }
        }
    }
    // ragged ends of the ranges, unit by unit
    constexpr uint32_t kSlots = 16u / uint32_t(sizeof(T)) - 1u;
    if constexpr (kSlots > 0) {
        for (uint32_t idx = tid; idx < nr * nrng * kSlots * 2u; idx += nthreads) {
            const uint32_t q = idx / (kSlots * 2u);
            const uint32_t w = idx - q * (kSlots * 2u);
            const bool is_head = w < kSlots;
            const uint32_t slot = is_head ? w : w - kSlots;
            const uint32_t r = fdiv(q, g.bx_nrng_div);
            const int64_t d0 = row_d0[r];
            uint32_t head, chunks;
            split_run(rng_bytes, d0, head, chunks);
            const uint32_t toff = head + (chunks << 4);
            const uint32_t count = (is_head ? head : rng_bytes - toff) / uint32_t(sizeof(T));
            if (slot >= count) continue;
            const uint32_t x = (is_head ? 0u : toff) + slot * uint32_t(sizeof(T));
            const uint32_t j = fdiv(x, g.bx_s2);
            const uint32_t at = base_of[q] + j * s1 + place[(x - j * s2) / uint32_t(sizeof(T))];
            if (!CHK_SMEM(at, uint32_t(sizeof(T)))) continue;
            const T val = *reinterpret_cast<const T *>(tile + at);
            char *const *dt = &P.dst[tile_of[q - r * nrng]];
            for (uint32_t f = 0; f < fanout; ++f)
                if (CHK_DST(P, dt[f] + d0 + x, uint32_t(sizeof(T)))) *reinterpret_cast<T *>(dt[f] + d0 + x) = val;
        }
    }
}

#define REDIST_DEFINE_BOX_KERNEL(NAME)                                                               \
    template <int NT, int SMALL>                                                                     \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P)  \
    {                                                                                                \
        extern __shared__ __align__(128) unsigned char tile[];                                       \
        __shared__ uint32_t base_of[kBoxSegments];                                                   \
        __shared__ uint32_t tile_of[kBoxSegments];                                                   \
        __shared__ int64_t row_d0[kBoxRows];                                                         \
        __shared__ __align__(8) unsigned long long mbar_storage;                                     \
        __shared__ unsigned int wait_failed;                                                         \
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");                              \
        const uint32_t mbar = smem_addr(&mbar_storage);                                              \
        if constexpr (SMALL != 0) {      /* 1: units of 1 and 2 bytes, 2: the same with chunks read in one piece */ \
            if (P.g.unit_bytes == 2)                                                                 \
                box_body<uint16_t, NT, SMALL == 2>(P, tile, base_of, tile_of, row_d0, mbar, &wait_failed); \
            else                                                                                     \
                box_body<uint8_t, NT, SMALL == 2>(P, tile, base_of, tile_of, row_d0, mbar, &wait_failed); \
        } else {                                                                                     \
            switch (P.g.unit_bytes) {                                                                \
            case 16: box_body<uint4, NT, false>(P, tile, base_of, tile_of, row_d0, mbar, &wait_failed); break; \
            case 8: box_body<uint2, NT, false>(P, tile, base_of, tile_of, row_d0, mbar, &wait_failed); break; \
            default: box_body<uint32_t, NT, false>(P, tile, base_of, tile_of, row_d0, mbar, &wait_failed); break; \
            }                                                                                        \
        }                                                                                            \
    }

REDIST_DEFINE_BOX_KERNEL(redist_dynslice_box_kernel)
REDIST_DEFINE_BOX_KERNEL(redist_alltoall_box_kernel)
REDIST_DEFINE_BOX_KERNEL(redist_allgather_box_kernel)
REDIST_DEFINE_BOX_KERNEL(redist_allpermute_box_kernel)
REDIST_DEFINE_BOX_KERNEL(redist_fused_box_kernel)

#define REDIST_DEFINE_RAGGED_BULK_KERNEL(NAME)                                                       \
    template <int NT>                                                                                \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P)  \
    {                                                                                                \
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");                              \
        ragged_bulk_body<NT>(P);                                                                     \
    }

REDIST_DEFINE_RAGGED_BULK_KERNEL(redist_dynslice_ragged_bulk_kernel)
REDIST_DEFINE_RAGGED_BULK_KERNEL(redist_alltoall_ragged_bulk_kernel)
REDIST_DEFINE_RAGGED_BULK_KERNEL(redist_allgather_ragged_bulk_kernel)
REDIST_DEFINE_RAGGED_BULK_KERNEL(redist_allpermute_ragged_bulk_kernel)
REDIST_DEFINE_RAGGED_BULK_KERNEL(redist_fused_ragged_bulk_kernel)


#define REDIST_DEFINE_KERNEL(NAME)                                                                   \
    template <int VARIANT, int NT>                                                                   \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P)  \
    {                                                                                                \
        copy_body<VARIANT, NT>(P);                                                                   \
    }

REDIST_DEFINE_KERNEL(redist_dynslice_kernel)
REDIST_DEFINE_KERNEL(redist_alltoall_kernel)
REDIST_DEFINE_KERNEL(redist_allgather_kernel)
REDIST_DEFINE_KERNEL(redist_allpermute_kernel)
REDIST_DEFINE_KERNEL(redist_fused_kernel)

// The part of this file that holds the kernels of a launch (see REDIST_PART at the top).
inline int part_of(const CopyGeometry &geo)
{
    if (geo.bulk) return 1;
    return geo.mode == kModeBox ? 3 : geo.mode == kModeZip ? 2 : 1;
}

// Which kernel entry serves a launch: by collective (so that profiles name the step that ran), by item
// shape and by pointer-table size.
template <int NT>
const void *entry_for(int kernel, const CopyGeometry &geo)
{
    using Fn = void (*)(const CopyParams<NT>);
    Fn fn = nullptr;
#define REDIST_PICK(SUFFIX, ...)                                                          \
    switch (kernel) {                                                                     \
    case 0: case 7: fn = redist_dynslice##SUFFIX<__VA_ARGS__>; break;                     \
    case 1: fn = redist_alltoall##SUFFIX<__VA_ARGS__>; break;                             \
    case 2: case 6: fn = redist_allgather##SUFFIX<__VA_ARGS__>; break;                    \
    case 3: case 4: fn = redist_allpermute##SUFFIX<__VA_ARGS__>; break;                   \
    default: fn = redist_fused##SUFFIX<__VA_ARGS__>; break;                               \
    }
    const bool ld = geo.gl_long_dst != 0;
    const bool small = geo.unit_bytes < 4;
    (void)ld;
    (void)small;
    // (launches on units of 1 and 2 bytes all run under the fused-sequence name: a fifth of the
    // instantiations, and of the time to compile them, for a rare case)
    if (part_of(geo) == 3) {
#if REDIST_IN(3)
        if (small) {
            fn = geo.one_piece ? redist_fused_box_kernel<NT, 2> : redist_fused_box_kernel<NT, 1>;
        } else {
            REDIST_PICK(_box_kernel, NT, 0)
        }
#endif
    } else if (part_of(geo) == 2) {
#if REDIST_IN(2)
        if (small) {
            fn = ld ? redist_fused_zip_kernel<true, NT, true> : redist_fused_zip_kernel<false, NT, true>;
        } else {
            if (ld) { REDIST_PICK(_zip_kernel, true, NT, false) } else { REDIST_PICK(_zip_kernel, false, NT, false) }
        }
#endif
    } else {
#if REDIST_IN(1)
        if (geo.bulk == 2) {
            REDIST_PICK(_ragged_bulk_kernel, NT)
        } else if (geo.bulk) {
            REDIST_PICK(_bulk_kernel, NT)
        } else if (geo.mode == kModeGather) {
            if (small) {
                fn = ld ? redist_fused_gather_kernel<true, NT, true> : redist_fused_gather_kernel<false, NT, true>;
            } else {
                if (ld) { REDIST_PICK(_gather_kernel, true, NT, false) } else { REDIST_PICK(_gather_kernel, false, NT, false) }
            }
        } else if (geo.mode == kModeRows) {
            REDIST_PICK(_kernel, 0, NT)
        } else if (geo.mode == kModeUnits) {
            REDIST_PICK(_kernel, 3, NT)
        } else if (geo.aligned) {
            REDIST_PICK(_kernel, 1, NT)
        } else {
            REDIST_PICK(_kernel, 2, NT)
        }
#endif
    }
#undef REDIST_PICK
    return reinterpret_cast<const void *>(fn);
}

template <int NT>
void fill_params(PreparedLaunch &pl, const CopyGeometry &geo, const char *const *src_tab, int n_src, char *const *dst_tab,
                 int n_dst)
{
    CopyParams<NT> *P = static_cast<CopyParams<NT> *>(pl.params);
    P->g = geo;
    for (int i = 0; i < n_src; ++i) P->src[i] = src_tab[i];
    for (int i = 0; i < n_dst; ++i) P->dst[i] = dst_tab[i];
}

// this part's counters
cudaError_t own_bulk_timeouts(unsigned int *out)
{
    return cudaMemcpyFromSymbol(out, g_bulk_timeouts, sizeof(unsigned int));
}

cudaError_t own_bounds_report(long long out[5])
{
#ifdef REDIST_BOUNDS
    unsigned long long n = 0;
    cudaError_t ce = cudaMemcpyFromSymbol(&n, g_bounds_count, sizeof n);
    if (ce == cudaSuccess) ce = cudaMemcpyFromSymbol(out + 1, g_bounds_first, 4 * sizeof(long long));
    out[0] = (long long)n;
    const unsigned long long zero = 0;
    const unsigned int uz = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyToSymbol(g_bounds_count, &zero, sizeof zero);
    if (ce == cudaSuccess) ce = cudaMemcpyToSymbol(g_bounds_taken, &uz, sizeof uz);
    return ce;
#else
    for (int i = 0; i < 5; ++i) out[i] = -1;
    return cudaErrorNotSupported;
#endif
}

}  // namespace

// What the parts offer each other: the entry point of a launch whose kernels live there, and their counters.
#define REDIST_DECLARE_PART(N)                                                               \
    const void *entry_in_part##N(int kernel, const CopyGeometry &geo, bool small_table);     \
    cudaError_t bulk_timeouts_in_part##N(unsigned int *out);                                  \
    cudaError_t bounds_report_in_part##N(long long out[5]);
#define REDIST_DEFINE_PART(N)                                                                \
    const void *entry_in_part##N(int kernel, const CopyGeometry &geo, bool small_table)      \
    {                                                                                        \
        return small_table ? entry_for<kSmallTable>(kernel, geo) : entry_for<kLargeTable>(kernel, geo); \
    }                                                                                        \
    cudaError_t bulk_timeouts_in_part##N(unsigned int *out) { return own_bulk_timeouts(out); } \
    cudaError_t bounds_report_in_part##N(long long out[5]) { return own_bounds_report(out); }
REDIST_DECLARE_PART(1)
REDIST_DECLARE_PART(2)
REDIST_DECLARE_PART(3)
#if REDIST_PART == 1
REDIST_DEFINE_PART(1)
#elif REDIST_PART == 2
REDIST_DEFINE_PART(2)
#elif REDIST_PART == 3
REDIST_DEFINE_PART(3)
#endif

#if REDIST_PART <= 1      // the host side lives in the single translation unit, or in part 1

cudaError_t read_bulk_timeouts(unsigned int *out)
{
#if REDIST_PART == 0
    return own_bulk_timeouts(out);
#else
    unsigned int a = 0, b = 0, c = 0;
    cudaError_t ce = bulk_timeouts_in_part1(&a);
    if (ce == cudaSuccess) ce = bulk_timeouts_in_part2(&b);
    if (ce == cudaSuccess) ce = bulk_timeouts_in_part3(&c);
    *out = a + b + c;
    return ce;
#endif
}

cudaError_t read_bounds_report(long long out[5])
{
#if REDIST_PART == 0
    return own_bounds_report(out);
#else
    // violations added up; the record of the first part that has one
    long long part[3][5];
    cudaError_t ce = bounds_report_in_part1(part[0]);
    if (ce == cudaSuccess) ce = bounds_report_in_part2(part[1]);
    if (ce == cudaSuccess) ce = bounds_report_in_part3(part[2]);
    if (ce != cudaSuccess) {
        for (int i = 0; i < 5; ++i) out[i] = -1;
        return ce;
    }
    for (int i = 0; i < 5; ++i) out[i] = 0;
    for (int k = 2; k >= 0; --k) {
        out[0] += part[k][0];
        if (part[k][0] > 0)
            for (int i = 1; i < 5; ++i) out[i] = part[k][i];
    }
    return cudaSuccess;
#endif
}

cudaError_t prepare_copy(int kernel, const CopyGeometry &geo, const char *const *src_tab, int n_src,
                         char *const *dst_tab, int n_dst, int pdl, void *storage, size_t storage_bytes,
                         PreparedLaunch &pl)
{
    if (n_src > kLargeTable || n_dst > kLargeTable || n_src < 0 || n_dst < 0) return cudaErrorInvalidValue;
    const bool small = n_src <= kSmallTable && n_dst <= kSmallTable;
    if (!storage || (reinterpret_cast<uintptr_t>(storage) & 15u) || storage_bytes < param_bytes(small ? kSmallTable : kLargeTable))
        return cudaErrorInvalidValue;
    pl.params = storage;
#if REDIST_PART == 0
    pl.fn = small ? entry_for<kSmallTable>(kernel, geo) : entry_for<kLargeTable>(kernel, geo);
#else
    pl.fn = part_of(geo) == 3   ? entry_in_part3(kernel, geo, small)
            : part_of(geo) == 2 ? entry_in_part2(kernel, geo, small)
                                : entry_in_part1(kernel, geo, small);
#endif
    if (small)
        fill_params<kSmallTable>(pl, geo, src_tab, n_src, dst_tab, n_dst);
    else
        fill_params<kLargeTable>(pl, geo, src_tab, n_src, dst_tab, n_dst);
    pl.pdl = pdl;
    // One thread block per work item: the hardware block scheduler balances the load and keeps the tail
    // to one item (measured 6-9 % faster than a grid-stride loop over a few blocks per SM).
    pl.grid = geo.n_items;
    pl.block = kBlockThreads;
    pl.smem = 0;
    if (geo.bulk == 2) {
        pl.smem = size_t(geo.stage_pitch) * geo.rows_per_item;
    } else if (geo.bulk) {
        const uint64_t seg = geo.mode == kModeRows ? geo.run_bytes : uint64_t(geo.per_block) * 16u;
        pl.block = kBulkThreads;
        pl.smem = size_t(seg * geo.rows_per_item);
    } else if (geo.mode == kModeBox) {
        pl.smem = size_t(geo.stage_pitch) * geo.rows_per_item + size_t(geo.zip_lut_units) * 2 + 16;
    } else if (geo.mode == kModeZip) {
        // small items stored to one or two replicas: eight and more blocks fit an SM, and half as many threads
        // per block means half as many threads that decode the item and wait for its copies (measured
        // +4..12 %); large items, and items whose chunks are stored many times, keep 256
        const bool few = size_t(geo.stage_pitch) * geo.rows_per_item <= kZipSmallTile && geo.fanout <= 2 &&
                         geo.zip_period.d * (geo.gl_long_dst == 0 && geo.zip_tile_fastest ? geo.gl_m.d : 1u) <= kBlockThreads / 2;
        pl.block = few ? kBlockThreads / 2 : kBlockThreads;
        pl.smem = size_t(geo.stage_pitch) * geo.rows_per_item + size_t(geo.zip_lut_units) * 4;
    }
    return cudaSuccess;
}

cudaError_t launch_prepared(const PreparedLaunch &pl, cudaStream_t stream)
{
    if (pl.grid == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3(pl.block);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = stream;
    // programmatic stream serialization: the kernel may start before its predecessor in the stream has
    // finished (see wait_for_previous_kernel)
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pl.pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void *args[1] = {pl.params};
    return cudaLaunchKernelExC(&cfg, pl.fn, args);
}

#endif   // REDIST_PART <= 1

}  // namespace redist
