// The copy descriptor every kernel of the executor receives as a kernel parameter.
//
// One launch moves data between two *layouts* (tile shape + which virtual device holds which
// tile) of the same logical global array.  With g_k = gcd(source tile size, target tile size) in
// dimension k, the global array is cut into "boxes" of shape (g_0, ..., g_{r-1}); every box lies in
// exactly one source tile and one target tile.  Box number -> unit digits q_k (one per dimension
// with more than one unit); q_k / m1_k is the source tile coordinate and q_k % m1_k the unit inside
// the source tile (m1_k = source tile size / g_k), likewise m2_k for the target.  Inside a box both
// sides are strided sub-arrays: "row digits" (outer to inner) with byte strides on either side and
// an innermost contiguous run of run_bytes.  Runs are moved in 16-byte chunks aligned on the target
// side; when not every address is a multiple of 16 (`aligned == 0`) the source chunk is assembled
// from two aligned loads and the ragged head and tail of a run go in `unit_bytes` pieces.
//
// Item numbering: the pieces of one long row (the m1*m2 units of the last differing dimension that
// share a source or target tile row) are consecutive items, so blocks that run at the same time fill
// the same memory sectors and partial-sector writes merge in L2 instead of being written back alone;
// then come the boxes of the other unit digits whose units share cache lines (fast_boxes of them), then
// the row groups of a box, then the remaining boxes.
//
// Aligned items whose row segments are at least 512 bytes (`bulk == 1`) are moved by TMA bulk copies
// through shared memory instead of by the register kernels; the item geometry is the same.
//
// Work items, by `mode`:
//   kModeRows   aligned runs of at most 256 chunks: a block covers rows_per_pass rows of `lanes`
//               chunks per pass; an item is rows_per_item rows; every thread decodes its own rows.
//   kModeChunks all other runs of at least 256 bytes: an item is rows_per_item rows times one column
//               block of per_block chunks; the rows are decoded once into shared memory and all
//               threads walk the (row, chunk) space with a flat index.
//   kModeGather runs shorter than 256 bytes whose pieces along the last differing dimension interleave
//               on one side (the long side: m runs from m tiles form one row) while the other side
//               keeps them in m tiles.  The target bytes of a table row -- a "stretch": the m runs of
//               a long row, or the run of a short row, times the innermost row digits over which the
//               target stays contiguous -- are walked in 16-byte chunks aligned on the target; every
//               thread assembles its chunk from unit_bytes pieces whose source addresses it computes
//               from the position inside the stretch, and stores it whole.  Stores fill whole
//               sectors; the loads of neighbouring lanes fall into the same few cache lines.
//   kModeZip    the same interleaving of m short runs, when both sides stay contiguous across the
//               innermost row digit (n rows): a table row is then m source streams of n runs zipped
//               into one target stream of n long rows, or the reverse.  An item covers rows_per_item
//               table rows times a block of per_block rows of that digit; its source bytes -- one
//               contiguous segment per stream -- are brought into shared memory by bulk copies, and
//               the threads assemble target-aligned 16-byte chunks from shared memory, where a
//               scattered access costs no cache-line lookups.
//   kModeBox    short runs whose pieces interleave along SEVERAL dimensions, or along one whose neighbouring
//               row digit is only a few rows long.  The item is widened from a box to a "super-box": in
//               each of the innermost differing dimensions (the inner dimensions, at most kMaxBoxDims) it
//               spans lcm(source tile, target tile) indices, so that it covers whole tiles of both sides
//               there, times per_block rows of the dimension just outside them, times rows_per_item rows of
//               the dimensions further out.  Its source bytes are then
//               one long contiguous segment per source tile it touches, its target bytes one long contiguous
//               range per target tile: the segments come into shared memory by bulk copies, and the ranges
//               are written in target-aligned 16-byte chunks whose units are found through a table of one
//               row's unit places (the place of a unit is separable: a term that depends on the target tile
//               plus a term that depends on the position inside the row).
//   kModeUnits  runs shorter than 256 bytes that are not 16-byte aligned: the same flat walk over
//               pieces of unit_bytes.  Only the outer row digits go through the shared table; the
//               innermost row digit is part of the walk (row payload = tab_inner.d runs), so that a
//               table of 1024 entries still covers tens of KiB when runs are a few bytes long.
#pragma once

#include <cstdint>

namespace redist {

constexpr int kMaxUnitDigits = 8;
constexpr int kMaxRowDigits = 8;
constexpr int kBlockThreads = 256;
constexpr int kBulkThreads = 64;       // block size of the bulk-copy kernels: one row segment per thread
constexpr int kMaxRowsFlat = 1024;     // rows of one item in the flat-walk modes (16 bytes of smem each)
constexpr int kModeRows = 0, kModeChunks = 1, kModeUnits = 2, kModeGather = 3, kModeZip = 4, kModeBox = 5;
constexpr int kMaxBoxDims = 3;         // inner dimensions of a kModeBox item
constexpr int kBoxSegments = 256;      // source segments, and target ranges, of one kModeBox item at most
constexpr int kBoxRows = 32;           // outer rows of one kModeBox item at most
constexpr int kZipSmallTile = 23 * 1024; // kModeZip items with at most this much shared memory run with 128 threads
constexpr int kZipSegments = 256;      // source segments (table rows times streams) of one kModeZip item
constexpr int kMaxGatherLevels = 2;    // innermost row digits that can be part of a stretch (kModeGather)
constexpr int kRaggedBulkRows = 256;   // rows of one item of the ragged bulk-in kernels

// Division of a 31-bit unsigned number by a constant: n / d == umulhi(n, mul) >> shr (d > 1).
struct FastDiv {
    uint32_t d, mul, shr;
};

struct CopyGeometry {
    uint32_t n_unit;                 // unit digits (dimensions with more than one box)
    uint32_t n_row;                  // row digits
    uint32_t fanout;                 // target replicas per box
    uint32_t aligned;                // 1: run length and every offset are multiples of 16 bytes
    uint32_t unit_bytes;             // largest power of two (<= 16) dividing run length and offsets
    uint32_t mode;                   // kModeRows, kModeChunks, kModeUnits, kModeGather or kModeZip
    uint32_t bulk;                   // 1: the item's row segments move by TMA bulk copies (aligned, >= 512 bytes);
                                     // 2: ragged chunk walk whose loads are bulk copies into shared memory
    uint64_t run_bytes;              // contiguous run
    uint32_t lanes;                  // kModeRows: threads per row, 1..kBlockThreads
    uint32_t rows_per_pass;          // kModeRows: kBlockThreads / lanes
    uint32_t rows;                   // rows per box (kModeUnits, kModeGather: table rows, i.e. without the digits walked flat)
    uint32_t rows_per_item;          // kModeRows: multiple of rows_per_pass; else <= kMaxRowsFlat
    uint32_t per_block;              // flat walk: chunks (or units) of one row in a column block
    uint32_t n_items;
    FastDiv per_block_div;           // flat walk: division by per_block
    FastDiv col_blocks;              // flat walk: column blocks per row (1 in kModeRows)
    FastDiv items_per_box;
    FastDiv fast_boxes;              // boxes of the trailing unit digits that vary faster than the row groups of a box (1: none)
    FastDiv inner_n;                 // pieces of one long row that consecutive items handle (1: none, or all in one item)
    uint32_t inner_digit;            // unit digit those pieces belong to
    uint32_t inner_span;             // units of that digit per long row (m1 * m2)
    uint32_t inner_mul;              // units per item along that digit: 1, or all of them (inner_span) in kModeGather
    uint32_t gl_long_dst;            // kModeGather, kModeZip: 1 the target has the long rows, 0 the source
    uint32_t stage_pitch;            // bulk == 2, kModeZip: bytes between the rows staged in shared memory
    uint32_t gl_ts;                  // kModeGather, kModeZip: tile-index stride between the pieces on the short side
    uint32_t gl_levels;              // kModeGather: innermost row digits inside a stretch (0..kMaxGatherLevels)
    uint32_t gl_stretch;             // kModeGather: bytes of one stretch (< 2^31)
    FastDiv gl_m;                    // kModeGather, kModeZip: pieces per long row
    uint32_t zip_seg_pitch;          // kModeZip: shared-memory bytes reserved per source segment
    FastDiv zip_slots;               // kModeZip: chunk slots per target range of an item
    FastDiv zip_cpr;                 // kModeZip: chunk slots per run in the by-range walk; d = 0: walk not used
    FastDiv zip_period;              // kModeZip: chunks after which the chunk -> units map repeats (d = 0: path not used)
    uint32_t zip_period_rows;        // kModeZip: rows of the zipped digit that one period spans
    uint32_t zip_width;              // kModeZip: lanes that walk one table row together (a multiple of zip_period);
                                     // kModeBox: lanes that walk one target range together (a power of two, at least a warp)
    uint32_t zip_lut_units;          // kModeZip: units of the longest range when their places are tabulated in shared memory (0: not)
    uint32_t zip_tile_fastest;       // kModeZip, long source rows: 1 = neighbouring lanes write to neighbouring target tiles
    FastDiv gl_n[kMaxGatherLevels];  // kModeGather: extents of those row digits, innermost first
    int64_t gl_b1[kMaxGatherLevels]; // kModeGather: their source byte strides
    FastDiv lanes_div;
    FastDiv unit_n[kMaxUnitDigits];  // boxes along the digit
    FastDiv unit_m1[kMaxUnitDigits];
    FastDiv unit_m2[kMaxUnitDigits];
    uint32_t unit_ts1[kMaxUnitDigits];   // tile-index stride, source / target
    uint32_t unit_ts2[kMaxUnitDigits];
    int64_t unit_b1[kMaxUnitDigits];     // byte stride of one unit inside the tile
    int64_t unit_b2[kMaxUnitDigits];
    uint32_t n_row_tab;              // row digits decoded through the shared table (n_row, n_row - 1, or n_row - gl_levels)
    FastDiv tab_inner;               // kModeUnits, kModeGather: runs per table row (extent of the digits walked flat, or 1)
    FastDiv units_per_run;           // kModeUnits, kModeGather: run_bytes / unit_bytes
    FastDiv row_n[kMaxRowDigits];
    int64_t row_b1[kMaxRowDigits];       // byte stride of the row digit, source / target
    int64_t row_b2[kMaxRowDigits];
    uint32_t unit_mul[kMaxUnitDigits];   // kModeBox: boxes per super-box along the digit (the digit counts super-boxes); else 1
    uint32_t bx_n;                   // kModeBox: inner dimensions, listed outer to inner below
    FastDiv bx_c2[kMaxBoxDims];      //   target tile extent (a digit of a position inside a target row)
    FastDiv bx_c1[kMaxBoxDims];      //   source tile extent
    FastDiv bx_n1[kMaxBoxDims];      //   source tiles per super-box along the dimension
    FastDiv bx_n2[kMaxBoxDims];      //   target tiles per super-box along the dimension
    uint32_t bx_ts1[kMaxBoxDims];    //   tile-index strides, source / target
    uint32_t bx_ts2[kMaxBoxDims];
    uint32_t bx_st1[kMaxBoxDims];    //   bytes between neighbouring indices of the dimension inside a source segment row
    uint32_t bx_seg[kMaxBoxDims];    //   segments between neighbouring source tiles of the dimension (mixed radix over bx_n1)
    FastDiv bx_trail;                // kModeBox: units of a run (innermost digit of a position inside a target row; the last
                                     //           inner dimension counts runs: its extents below are divided by the gcd)
    FastDiv bx_s2;                   // kModeBox: bytes of one row (of the dimension outside the inner ones) in a target range
    uint32_t bx_s1;                  //           ... in a source segment
    uint32_t bx_nseg, bx_nrng;       // kModeBox: source segments / target ranges of one outer row of an item
    FastDiv bx_nseg_div, bx_nrng_div;
    FastDiv bx_row_units_div;        // kModeBox: division by the units of one target row (zip_lut_units)
    uint32_t wait_polls;             // bulk-copy kernels: mbarrier polls before a block gives up (bounded wait)
    uint32_t l2_hint;                // plain bulk-copy kernels: 1 loads, 2 stores (3 both) carry an L2 evict-first policy
    uint32_t one_piece;              // super-box kernels on units of 1 or 2 bytes: chunks inside one run are read in one piece
    uint32_t test_extra_tx;          // test only: bytes announced on the mbarrier beyond what the copies deliver, so
                                     // that every copy lands but the phase never completes (0 in every real plan)
    uint32_t n_src_tab, n_dst_tab;   // entries of the two pointer tables
    uint64_t src_tile_bytes;         // bytes of one source / target tile (the checked build tests every access
    uint64_t dst_tile_bytes;         // against them; the kernels themselves do not need them)
};

template <int NT>
struct CopyParams {
    CopyGeometry g;
    const char *src[NT];   // source tile index          -> base pointer of a device that holds it
    char *dst[NT];         // target tile index * fanout -> base pointers of the devices that receive it
};

}  // namespace redist
