// Internal data structures of the planner and the executor (host side).
#pragma once

#include <cstdint>
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

enum BufKind { BUF_SRC = 0, BUF_DST = 1, BUF_SCRATCH0 = 2, BUF_SCRATCH1 = 3, BUF_GLOBAL = 4 };

struct Launch {
    int first_step = 0, n_steps = 0, kernel = 0;
    BufKind from = BUF_SRC, to = BUF_DST;
    CopyGeometry geo;                    // what the kernel receives (without pointers)
    std::vector<int32_t> src_holder;     // [source tiles]           device whose buffer is read
    std::vector<int32_t> dst_devs;       // [target tiles * fanout]  devices that receive the tile
    i64 run_bytes = 0, bytes_read = 0, bytes_written = 0;
    i64 src_tile_bytes = 0, dst_tile_bytes = 0;
};

struct Plan {
    int n_mesh_axes = 0, rank = 0, elem_bytes = 0, n_devices = 0;
    uint32_t flags = 0;
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

// The opaque handle of the C boundary.
struct redist_plan_s {
    redist::Plan p;
};

namespace redist {

// api.cu: last CUDA error seen by the calling thread inside the library
extern thread_local int tl_cuda_error;

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
