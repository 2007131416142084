// The copy descriptor every kernel of the executor receives as a kernel parameter.
//
// One launch moves data between two *layouts* (tile shape + which virtual device holds which
// tile) of the same logical global array.  With g_k = gcd(source tile size, target tile size) in
// dimension k, the global array is cut into "boxes" of shape (g_0, ..., g_{r-1}); every box lies in
// exactly one source tile and one target tile.  Box number -> unit digits q_k (one per dimension
// with more than one unit); q_k / m1_k is the source tile coordinate and q_k % m1_k the unit inside
// the source tile (m1_k = source tile size / g_k), likewise m2_k for the target.  Inside a box both
// sides are strided sub-arrays: "row digits" (outer to inner) with byte strides on either side and
// an innermost contiguous run of `lanes` vectors.  A work item is a chunk of rows of one box.
#pragma once

#include <cstdint>

namespace redist {

constexpr int kMaxUnitDigits = 8;
constexpr int kMaxRowDigits = 10;
constexpr int kBlockThreads = 256;

// Division of a 31-bit unsigned number by a constant: n / d == umulhi(n, mul) >> shr (d > 1).
struct FastDiv {
    uint32_t d, mul, shr;
};

struct CopyGeometry {
    uint32_t n_unit;                 // unit digits (dimensions with more than one box)
    uint32_t n_row;                  // row digits
    uint32_t fanout;                 // target replicas per box
    uint32_t vec_bytes;              // bytes per memory access: 16, 8, 4, 2 or 1
    uint32_t lanes;                  // vectors per run, 1..kBlockThreads
    uint32_t rows_per_pass;          // kBlockThreads / lanes
    uint32_t rows;                   // rows per box
    uint32_t rows_per_item;          // multiple of rows_per_pass
    uint32_t n_items;
    FastDiv items_per_box;
    FastDiv lanes_div;
    FastDiv unit_n[kMaxUnitDigits];  // boxes along the digit
    FastDiv unit_m1[kMaxUnitDigits];
    FastDiv unit_m2[kMaxUnitDigits];
    uint32_t unit_ts1[kMaxUnitDigits];   // tile-index stride, source / target
    uint32_t unit_ts2[kMaxUnitDigits];
    int64_t unit_b1[kMaxUnitDigits];     // byte stride of one unit inside the tile
    int64_t unit_b2[kMaxUnitDigits];
    FastDiv row_n[kMaxRowDigits];
    int64_t row_b1[kMaxRowDigits];       // byte stride of the row digit, source / target
    int64_t row_b2[kMaxRowDigits];
};

template <int NT>
struct CopyParams {
    CopyGeometry g;
    const char *src[NT];   // source tile index          -> base pointer of a device that holds it
    char *dst[NT];         // target tile index * fanout -> base pointers of the devices that receive it
};

}  // namespace redist
