// Internal data structures of the planner and the executor (host side).
#pragma once

#include <cstdint>
#include <memory>
#include <string>
#include <vector>

#include "copy_params.h"
#include "redist.h"

namespace redist {

using i64 = int64_t;

// One prime-sized axis of the decomposed mesh (Principle 1, Section 3).  The coordinate of a device
// on it is (coordinate on the parent axis / parent_stride) % size, so that the parent coordinate is
// i_x = i_x1 + p1 * (i_x2 + p2 * ...) and base offsets are unchanged by the decomposition.
struct PrimeAxis {
    int parent;
    i64 size;
    i64 parent_stride;
};

// A device assignment <phi, beta> (Section 6): the current type as per-dimension lists of prime
// axes (minor to major) and, for every physical device d, its logical coordinates phi^-1(d).
struct ConcreteState {
    std::vector<std::vector<int>> ax;
    std::vector<std::vector<int>> lc;   // [N][n_prime_axes]
};

// What the executor needs to know of a state: the tile shape and which tile each device holds.
struct Layout {
    std::vector<i64> tile;          // localtype
    std::vector<i64> ntiles;        // tiles per dimension
    std::vector<int32_t> tile_of;   // [N] row-major tile index held by device d
    bool shared_global = false;     // baseline only: the whole array once, in one shared buffer
};

struct Step {
    int kind = 0;
    int dim_i = -1, dim_j = -1;
    i64 factor = 1;
    std::vector<int> acting;        // prime axes acted on, in block order (first = fastest)
    ConcreteState pre;              // equivalent relabelled assignment the typing rule applies to
    ConcreteState post;             // assignment after the step
    std::vector<int> source_of;     // allpermute: device d receives the tile of source_of[d]
    std::vector<i64> local_before, local_after;
    i64 cost = 0;
    i64 localsize_after = 0;
};

// Tuning values, copied into a plan when it is created (redist_tuning_set changes the values later
// plans get).  Defaults are the measured optima; the tests use them to force the kernel variants that
// the default choice seldom leaves work for, the benchmark to show what a choice is worth.
struct Tuning {
    int64_t bulk = 1;                 // 0: no TMA bulk copies at all (register kernels only)
    int64_t gather = 1;               // gather walk: 0 never, 1 where measured faster, 2 wherever it applies
    int64_t zip = 2;                  // zip kernels: 0 never, 1 only where the gather walk is not chosen, 2 wherever they apply
    int64_t box = 1;                  // super-box kernels: 0 never, 1 where zip / gather / unit walks do badly, 2 wherever they apply
    int64_t box_width = 0;            // super-box kernels: lanes per target range (a power of two), 0: chosen per launch
    int64_t zip_walks = 7;            // chunk -> units maps the zip kernels may use: 1 periodic, 2 by range, 4 tabulated
    int64_t zip_by_range_slots = 256; // fewest chunk slots of a range for the by-range walk
    int64_t item_kb = 0;              // KiB read per work item (0: 32 / 16 / 8 by fan-out, bulk copies 20 / 12 / 6)
    int64_t piece = 1;                // 0: the small-unit super-box kernels never read a chunk in one piece
    int64_t l2_hint = 4;              // plain bulk-copy kernels, L2 evict-first policy on: 0 nothing, 1 loads, 2 stores, 3 both, 4 stores from fan-out 4
    int64_t pdl = 1;                  // 0: plain stream order instead of programmatic dependent launch
    int64_t nvtx = 0;                 // 1: redist_execute wraps every kernel launch in an NVTX range named after the step
    int64_t step_latency = 0;         // elements added to the cost of every collective when searching (Section 8, RQ3)
    int64_t wait_polls = 1 << 18;     // mbarrier polls before a bulk-copy block gives up
    int64_t test_extra_tx = 0;        // test only, see CopyGeometry::test_extra_tx
    int64_t test_shrink_tiles = 0;    // test only: bytes by which the checked build believes every tile to be shorter
    bool operator==(const Tuning &o) const
    {
        return bulk == o.bulk && gather == o.gather && zip == o.zip && box == o.box && box_width == o.box_width && zip_walks == o.zip_walks &&
               zip_by_range_slots == o.zip_by_range_slots && item_kb == o.item_kb && l2_hint == o.l2_hint && piece == o.piece && pdl == o.pdl && nvtx == o.nvtx &&
               step_latency == o.step_latency && wait_polls == o.wait_polls && test_extra_tx == o.test_extra_tx &&
               test_shrink_tiles == o.test_shrink_tiles;
    }
};

enum BufKind { BUF_SRC = 0, BUF_DST = 1, BUF_SCRATCH0 = 2, BUF_SCRATCH1 = 3, BUF_GLOBAL = 4 };

struct Launch {
    int first_step = 0, n_steps = 0, kernel = 0;
    BufKind from = BUF_SRC, to = BUF_DST;
    CopyGeometry geo;                    // what the kernel receives (without pointers)
    std::vector<int32_t> src_tile_of;    // [devices]                source tile each device holds (-1: shared buffer)
    std::vector<int32_t> src_holder;     // [source tiles]           device whose buffer is read
    std::vector<int32_t> dst_devs;       // [target tiles * fanout]  devices that receive the tile
    i64 run_bytes = 0, bytes_read = 0, bytes_written = 0;
    i64 src_tile_bytes = 0, dst_tile_bytes = 0;
    std::vector<i64> src_tile, dst_tile;     // tile shapes of the two layouts
};

struct Plan {
    int n_mesh_axes = 0, rank = 0, elem_bytes = 0, n_devices = 0;
    uint32_t flags = 0;
    Tuning tuning;
    std::vector<i64> mesh_shape, global_shape;
    std::vector<std::vector<int>> src_axes, dst_axes;      // original axes
    std::vector<PrimeAxis> primes;
    std::vector<std::vector<int>> src_pax, dst_pax;        // over prime axes
    ConcreteState initial;
    std::vector<Step> steps;
    std::vector<Launch> launches;
    i64 local_src = 0, local_dst = 0, height = 0, cost = 0;
    i64 slot_bytes = 0;              // one scratch slot of one virtual device
    i64 scratch_bytes = 0;           // total
    i64 scratch_per_device = 0;      // reported share
    int alignment = 16;
    std::string json;
};

}  // namespace redist

// The opaque handle of the C boundary: a reference to an immutable plan, which the plan cache and
// any number of handles may share.
struct redist_plan_s {
    std::shared_ptr<const redist::Plan> ref;
    const redist::Plan &p;
    explicit redist_plan_s(std::shared_ptr<const redist::Plan> r) : ref(std::move(r)), p(*ref) {}
};

namespace redist {

// api.cu: last CUDA error seen by the calling thread inside the library
extern thread_local int tl_cuda_error;

// api.cu: buffer checks (alignment; destination tiles and the `scratch_range` bytes at `scratch` disjoint
// from each other and from every source), then the plan's kernel launches on the stream.  Shared by
// every execute entry point; allocates nothing.
redist_status run_plan(const Plan &p, const void *const *src_shards, void *const *dst_shards, void *scratch,
                       size_t scratch_range, void *cuda_stream);

// planner.cpp
redist_status synthesize(Plan &p);
redist_status check_type(int n_axes, const i64 *mesh, const redist_type *t, std::vector<i64> *tile);
void base_offsets_of(int n_axes, const i64 *mesh, const redist_type *t, const std::vector<i64> &tile,
                     i64 *out);
Layout layout_of(const Plan &p, const ConcreteState &s);
std::vector<i64> localtype_of(const Plan &p, const ConcreteState &s);

// descriptor.cpp
redist_status build_launches(Plan &p);
redist_status build_copy(const Plan &p, const Layout &a, const Layout &b, Launch &out);

// describe.cpp
void describe(Plan &p);

}  // namespace redist
