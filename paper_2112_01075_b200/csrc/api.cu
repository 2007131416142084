// The C boundary: plan creation (with the plan cache and the tuning values), execution and queries.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cstring>
#include <deque>
#include <mutex>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>

#include "kernels.h"
#include "plan.hpp"

using namespace redist;

namespace redist {
thread_local int tl_cuda_error = 0;
}

// A plan bound to one set of buffers: every launch prepared once (entry point, launch shape, parameter
// block with both pointer tables), so that executing it is the kernel launches and nothing else.
struct redist_bound_s {
    std::shared_ptr<const redist::Plan> ref;
    std::vector<redist::PreparedLaunch> launches;
    std::vector<std::vector<max_align_t>> params;     // one parameter block per launch
};

namespace {

struct Range {
    uintptr_t lo, hi;
    int kind;   // 0 source (may alias other sources), 1 written
};

// a written range may not intersect any other range; sources may intersect sources (sweep over the
// ranges sorted by start; sorts `r` in place, allocates nothing)
bool overlaps(Range *r, int n)
{
    std::sort(r, r + n, [](const Range &a, const Range &b) { return a.lo < b.lo; });
    uintptr_t max_hi_written = 0, max_hi_any = 0;
    bool have_w = false, have_any = false;
    for (int i = 0; i < n; ++i) {
        const Range &x = r[i];
        if (x.lo >= x.hi) continue;
        if (x.kind == 1) {
            if (have_any && x.lo < max_hi_any) return true;
        } else {
            if (have_w && x.lo < max_hi_written) return true;
        }
        if (x.kind == 1) {
            max_hi_written = have_w ? std::max(max_hi_written, x.hi) : x.hi;
            have_w = true;
        }
        max_hi_any = have_any ? std::max(max_hi_any, x.hi) : x.hi;
        have_any = true;
    }
    return false;
}

// ---- tuning values and plan cache (process-wide, behind one mutex) ----------------------------
std::mutex g_mutex;
Tuning g_tuning;

struct TuningName {
    const char *name;
    int64_t Tuning::*field;
    int64_t lo, hi;
};
const TuningName kTuningNames[] = {
    {"bulk", &Tuning::bulk, 0, 1},
    {"gather", &Tuning::gather, 0, 2},
    {"zip", &Tuning::zip, 0, 2},
    {"box", &Tuning::box, 0, 2},
    {"box_width", &Tuning::box_width, 0, 256},
    {"zip_walks", &Tuning::zip_walks, 0, 7},
    {"zip_by_range_slots", &Tuning::zip_by_range_slots, 1, 1 << 20},
    {"item_kb", &Tuning::item_kb, 0, 1024},
    {"l2_hint", &Tuning::l2_hint, 0, 4},
    {"piece", &Tuning::piece, 0, 1},
    {"pdl", &Tuning::pdl, 0, 1},
    {"nvtx", &Tuning::nvtx, 0, 1},
    {"step_latency", &Tuning::step_latency, 0, int64_t(1) << 50},
    {"wait_polls", &Tuning::wait_polls, 1, int64_t(1) << 30},
    {"test_extra_tx", &Tuning::test_extra_tx, 0, 1 << 20},
    {"test_shrink_tiles", &Tuning::test_shrink_tiles, 0, 1 << 20},
};

constexpr size_t kCacheEntries = 256;
std::unordered_map<std::string, std::shared_ptr<const Plan>> g_cache;
std::deque<std::string> g_cache_order;     // oldest first
int64_t g_cache_hits = 0, g_cache_misses = 0;

std::string cache_key(int32_t n_mesh_axes, const int64_t *mesh_shape, const redist_type *src, const redist_type *dst,
                      int32_t elem_bytes, uint32_t flags, const Tuning &t)
{
    std::string k;
    auto put = [&k](int64_t v) { k.append(reinterpret_cast<const char *>(&v), sizeof v); };
    put(n_mesh_axes);
    for (int a = 0; a < n_mesh_axes; ++a) put(mesh_shape[a]);
    for (const redist_type *ty : {src, dst}) {
        put(ty->rank);
        for (int d = 0; d < ty->rank; ++d) {
            put(ty->global_shape[d]);
            put(ty->axes_off[d + 1] - ty->axes_off[d]);
            for (int q = ty->axes_off[d]; q < ty->axes_off[d + 1]; ++q) put(ty->axes[q]);
        }
    }
    put(elem_bytes);
    put(flags);
    for (const TuningName &n : kTuningNames) put(t.*(n.field));
    return k;
}

// Buffer checks shared by every execute entry point: pointers present and aligned, destination and
// scratch ranges disjoint from each other and from every source.  Allocates nothing; CAP bounds the
// number of virtual devices (the range table lives on the stack).
template <int CAP>
redist_status check_buffers(const Plan &p, const void *const *src_shards, void *const *dst_shards, const void *scratch,
                            size_t scratch_range)
{
    const int N = p.n_devices;
    if (N > CAP) return REDIST_EINTERNAL;
    const uintptr_t amask = uintptr_t(p.alignment) - 1;
    const i64 sb = p.local_src * p.elem_bytes, db = p.local_dst * p.elem_bytes;
    Range ranges[2 * CAP + 1];
    int n = 0;
    for (int d = 0; d < N; ++d) {
        if (!src_shards[d] || !dst_shards[d]) return REDIST_EINVAL;
        const uintptr_t s = uintptr_t(src_shards[d]), t = uintptr_t(dst_shards[d]);
        if ((s & amask) || (t & amask)) return REDIST_EALIGN;
        ranges[n++] = Range{s, s + uintptr_t(sb), 0};
        ranges[n++] = Range{t, t + uintptr_t(db), 1};
    }
    if (scratch_range > 0) {
        if (uintptr_t(scratch) & 255) return REDIST_EALIGN;
        ranges[n++] = Range{uintptr_t(scratch), uintptr_t(scratch) + uintptr_t(scratch_range), 1};
    }
    return overlaps(ranges, n) ? REDIST_EOVERLAP : REDIST_OK;
}

// Pointer tables of one launch from the caller's buffers (on the stack, CAP entries), then the prepared
// launch with its parameter block written to `storage`.
template <int CAP>
redist_status prepare_launch(const Plan &p, const Launch &L, const void *const *src_shards, void *const *dst_shards,
                             char *scratch, void *storage, size_t storage_bytes, PreparedLaunch &pl)
{
    const int N = p.n_devices;
    auto buffer = [&](BufKind kind, int32_t dev) -> char * {
        switch (kind) {
        case BUF_SRC: return static_cast<char *>(const_cast<void *>(src_shards[dev]));
        case BUF_DST: return static_cast<char *>(dst_shards[dev]);
        case BUF_SCRATCH0: return scratch + i64(dev) * p.slot_bytes;
        case BUF_SCRATCH1: return scratch + (i64(N) + dev) * p.slot_bytes;
        default: return scratch;
        }
    };
    const int ns = int(L.src_holder.size()), nd = int(L.dst_devs.size());
    if (ns > CAP || nd > CAP) return REDIST_EUNSUPPORTED;
    const char *stab[CAP];
    char *dtab[CAP];
    for (int t = 0; t < ns; ++t) stab[t] = buffer(L.from, L.src_holder[t] < 0 ? 0 : L.src_holder[t]);
    for (int t = 0; t < nd; ++t) dtab[t] = buffer(L.to, L.dst_devs[t] < 0 ? 0 : L.dst_devs[t]);
    cudaError_t ce = prepare_copy(L.kernel, L.geo, stab, ns, dtab, nd, int(p.tuning.pdl), storage, storage_bytes, pl);
    if (ce != cudaSuccess) {
        tl_cuda_error = int(ce);
        return REDIST_ECUDA;
    }
    return REDIST_OK;
}

// Checks, then one kernel launch per entry of the plan's launch list; tables and parameter block on
// this frame.
template <int CAP>
redist_status run_plan_with(const Plan &p, const void *const *src_shards, void *const *dst_shards, void *scratch,
                            size_t scratch_range, void *cuda_stream)
{
    redist_status rc = check_buffers<CAP>(p, src_shards, dst_shards, scratch, scratch_range);
    if (rc != REDIST_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    alignas(16) unsigned char storage[param_bytes(CAP)];
    PreparedLaunch pl;
    static const char *const kNames[] = {"redist dynslice", "redist alltoall", "redist allgather", "redist allpermute",
                                         "redist copy", "redist fused", "redist naive gather", "redist naive slice"};
    for (const Launch &L : p.launches) {
        if (L.geo.n_items == 0) continue;
        rc = prepare_launch<CAP>(p, L, src_shards, dst_shards, static_cast<char *>(scratch), storage, sizeof storage, pl);
        if (rc != REDIST_OK) return rc;
        // an NVTX range around every launch names the step for a timeline profiler (tuning value "nvtx")
        const bool mark = p.tuning.nvtx != 0;
        if (mark) nvtxRangePushA(kNames[L.kernel >= 0 && L.kernel < 8 ? L.kernel : 5]);
        cudaError_t ce = launch_prepared(pl, stream);
        if (mark) nvtxRangePop();
        if (ce != cudaSuccess) {
            tl_cuda_error = int(ce);
            return REDIST_ECUDA;
        }
    }
    return REDIST_OK;
}

}  // namespace

namespace redist {

// Checks, then the plan's kernel launches.  Everything lives on this call's stack -- about 8 KiB for
// plans of up to 64 virtual devices, about 100 KiB beyond; nothing is allocated on the host or the device.
redist_status run_plan(const Plan &p, const void *const *src_shards, void *const *dst_shards, void *scratch,
                       size_t scratch_range, void *cuda_stream)
{
    return p.n_devices <= kSmallTable
               ? run_plan_with<kSmallTable>(p, src_shards, dst_shards, scratch, scratch_range, cuda_stream)
               : run_plan_with<kLargeTable>(p, src_shards, dst_shards, scratch, scratch_range, cuda_stream);
}

}  // namespace redist

extern "C" {

const char *redist_status_string(redist_status s)
{
    switch (s) {
    case REDIST_OK: return "ok";
    case REDIST_EINVAL: return "invalid argument";
    case REDIST_EILLFORMED: return "ill-formed distributed type";
    case REDIST_ENOTDIV: return "tile size does not divide the global size";
    case REDIST_EGLOBAL: return "source and target describe different global arrays";
    case REDIST_ESCRATCH: return "scratch or staging buffer missing or too small";
    case REDIST_EOVERLAP: return "destination or scratch overlaps another buffer";
    case REDIST_EALIGN: return "buffer not aligned";
    case REDIST_ENOMEM: return "out of host memory";
    case REDIST_ECUDA: return "CUDA error";
    case REDIST_EUNSUPPORTED: return "beyond a built-in limit";
    case REDIST_EINTERNAL: return "internal plan check failed";
    }
    return "unknown status";
}

int32_t redist_last_cuda_error(void) { return tl_cuda_error; }

int64_t redist_bulk_timeouts(void)
{
    unsigned int n = 0;
    cudaError_t ce = read_bulk_timeouts(&n);
    if (ce != cudaSuccess) {
        tl_cuda_error = int(ce);
        return -1;
    }
    return int64_t(n);
}

redist_status redist_base_offsets(int32_t n_mesh_axes, const int64_t *mesh_shape, const redist_type *type,
                                  int64_t *out_tile, int64_t *out_offsets)
{
    try {
        if (n_mesh_axes < 0 || n_mesh_axes > REDIST_MAX_MESH_AXES || (n_mesh_axes > 0 && !mesh_shape) || !type ||
            !out_tile || !out_offsets)
            return REDIST_EINVAL;
        i64 N = 1;
        for (int a = 0; a < n_mesh_axes; ++a) {
            if (mesh_shape[a] < 1) return REDIST_EINVAL;
            N *= mesh_shape[a];
            if (N > REDIST_MAX_DEVICES) return REDIST_EUNSUPPORTED;
        }
        std::vector<i64> tile;
        redist_status rc = check_type(n_mesh_axes, mesh_shape, type, &tile);
        if (rc != REDIST_OK) return rc;
        std::vector<i64> off(size_t(N) * type->rank);
        base_offsets_of(n_mesh_axes, mesh_shape, type, tile, off.data());
        std::copy(tile.begin(), tile.end(), out_tile);
        std::copy(off.begin(), off.end(), out_offsets);
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

redist_status redist_plan(int32_t n_mesh_axes, const int64_t *mesh_shape, const redist_type *src,
                          const redist_type *dst, int32_t elem_bytes, uint32_t flags, redist_plan_t **out)
{
    if (!out || !src || !dst || n_mesh_axes < 0 || n_mesh_axes > REDIST_MAX_MESH_AXES ||
        (n_mesh_axes > 0 && !mesh_shape))
        return REDIST_EINVAL;
    if (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4 && elem_bytes != 8 && elem_bytes != 16)
        return REDIST_EINVAL;
    if (flags & ~uint32_t(REDIST_MODE_MASK | REDIST_NO_OVERPARTITION | REDIST_COST_PERMUTE | REDIST_NO_CACHE))
        return REDIST_EINVAL;
    i64 N = 1;
    for (int a = 0; a < n_mesh_axes; ++a) {
        if (mesh_shape[a] < 1) return REDIST_EINVAL;
        N *= mesh_shape[a];
        if (N > REDIST_MAX_DEVICES) return REDIST_EUNSUPPORTED;
    }
    std::vector<i64> tile1, tile2;
    redist_status rc = check_type(n_mesh_axes, mesh_shape, src, &tile1);
    if (rc != REDIST_OK) return rc;
    rc = check_type(n_mesh_axes, mesh_shape, dst, &tile2);
    if (rc != REDIST_OK) return rc;
    // a redistribution is valid iff both types have the same global type (Section 2.5)
    if (src->rank != dst->rank) return REDIST_EGLOBAL;
    i64 gsize = 1;
    for (int k = 0; k < src->rank; ++k) {
        if (src->global_shape[k] != dst->global_shape[k]) return REDIST_EGLOBAL;
        if (gsize > (i64(1) << 56) / src->global_shape[k]) return REDIST_EUNSUPPORTED;
        gsize *= src->global_shape[k];
    }
    // plan cache: the same problem under the same tuning values gets the same (immutable) plan again
    const bool cached = (flags & REDIST_NO_CACHE) == 0;
    flags &= ~uint32_t(REDIST_NO_CACHE);
    std::shared_ptr<Plan> fresh;
    try {
        Tuning tuning;
        std::string key;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            tuning = g_tuning;
            if (cached) {
                key = cache_key(n_mesh_axes, mesh_shape, src, dst, elem_bytes, flags, tuning);
                auto it = g_cache.find(key);
                if (it != g_cache.end()) {
                    ++g_cache_hits;
                    redist_plan_s *h = new redist_plan_s(it->second);
                    *out = h;
                    return REDIST_OK;
                }
                ++g_cache_misses;
            }
        }
        fresh = std::make_shared<Plan>();
        Plan &p = *fresh;
        p.tuning = tuning;
        p.n_mesh_axes = n_mesh_axes;
        p.rank = src->rank;
        p.elem_bytes = elem_bytes;
        p.n_devices = int(N);
        p.flags = flags;
        p.mesh_shape.assign(mesh_shape, mesh_shape + n_mesh_axes);
        p.global_shape.assign(src->global_shape, src->global_shape + src->rank);
        auto axes_of = [](const redist_type *t) {
            std::vector<std::vector<int>> v(t->rank);
            for (int k = 0; k < t->rank; ++k)
                for (int q = t->axes_off[k]; q < t->axes_off[k + 1]; ++q) v[k].push_back(t->axes[q]);
            return v;
        };
        p.src_axes = axes_of(src);
        p.dst_axes = axes_of(dst);
        rc = synthesize(p);
        if (rc == REDIST_OK) rc = build_launches(p);
        if (rc == REDIST_OK) {
            // end-state check against the base offset map of the target type as the caller wrote it
            // (original mesh, not the prime one): device d must end with the tile at T[[dst]](d)
            std::vector<i64> off(size_t(N) * dst->rank);
            base_offsets_of(n_mesh_axes, mesh_shape, dst, tile2, off.data());
            const ConcreteState &end = p.steps.empty() ? p.initial : p.steps.back().post;
            Layout l = layout_of(p, end);
            if (l.tile != tile2) rc = REDIST_EINTERNAL;
            for (int d = 0; d < N && rc == REDIST_OK; ++d) {
                i64 lin = 0;
                for (int k = 0; k < p.rank; ++k) lin = lin * l.ntiles[k] + off[size_t(d) * p.rank + k] / tile2[k];
                if (lin != l.tile_of[d]) rc = REDIST_EINTERNAL;
            }
        }
        if (rc == REDIST_OK) describe(p);
        if (rc != REDIST_OK) return rc;
        redist_plan_s *h = new redist_plan_s(fresh);
        if (cached) {
            std::lock_guard<std::mutex> lock(g_mutex);
            if (g_cache.emplace(key, fresh).second) {
                g_cache_order.push_back(key);
                if (g_cache_order.size() > kCacheEntries) {
                    g_cache.erase(g_cache_order.front());
                    g_cache_order.pop_front();
                }
            }
        }
        *out = h;
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

void redist_plan_cache_stats(int64_t *hits, int64_t *misses, int64_t *entries)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (hits) *hits = g_cache_hits;
    if (misses) *misses = g_cache_misses;
    if (entries) *entries = int64_t(g_cache.size());
}

void redist_plan_cache_clear(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    g_cache.clear();
    g_cache_order.clear();
    g_cache_hits = g_cache_misses = 0;
}

redist_status redist_tuning_set(const char *name, int64_t value)
{
    if (!name) return REDIST_EINVAL;
    for (const TuningName &n : kTuningNames)
        if (std::strcmp(name, n.name) == 0) {
            if (value < n.lo || value > n.hi) return REDIST_EINVAL;
            std::lock_guard<std::mutex> lock(g_mutex);
            g_tuning.*(n.field) = value;
            return REDIST_OK;
        }
    return REDIST_EINVAL;
}

redist_status redist_tuning_get(const char *name, int64_t *value)
{
    if (!name || !value) return REDIST_EINVAL;
    for (const TuningName &n : kTuningNames)
        if (std::strcmp(name, n.name) == 0) {
            std::lock_guard<std::mutex> lock(g_mutex);
            *value = g_tuning.*(n.field);
            return REDIST_OK;
        }
    return REDIST_EINVAL;
}

void redist_tuning_reset(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    g_tuning = Tuning();
}

redist_status redist_debug_bounds_report(int64_t out[5])
{
    if (!out) return REDIST_EINVAL;
    long long r[5];
    cudaError_t ce = read_bounds_report(r);
    if (ce == cudaErrorNotSupported) return REDIST_EUNSUPPORTED;
    if (ce != cudaSuccess) {
        tl_cuda_error = int(ce);
        return REDIST_ECUDA;
    }
    for (int i = 0; i < 5; ++i) out[i] = r[i];
    return REDIST_OK;
}

void redist_plan_destroy(redist_plan_t *plan) { delete plan; }

int32_t redist_plan_num_devices(const redist_plan_t *plan) { return plan ? plan->p.n_devices : 0; }
int32_t redist_plan_rank(const redist_plan_t *plan) { return plan ? plan->p.rank : 0; }
int64_t redist_plan_local_elems(const redist_plan_t *plan, int32_t which)
{
    return plan ? (which ? plan->p.local_dst : plan->p.local_src) : 0;
}
size_t redist_plan_scratch_bytes(const redist_plan_t *plan) { return plan ? size_t(plan->p.scratch_bytes) : 0; }
size_t redist_plan_scratch_bytes_per_device(const redist_plan_t *plan)
{
    return plan ? size_t(plan->p.scratch_per_device) : 0;
}
size_t redist_plan_staging_bytes(const redist_plan_t *plan, int32_t which)
{
    if (!plan) return 0;
    const i64 tile = (which ? plan->p.local_dst : plan->p.local_src) * plan->p.elem_bytes;
    return size_t((tile + 255) / 256 * 256 * plan->p.n_devices);
}
int32_t redist_plan_alignment(const redist_plan_t *plan) { return plan ? plan->p.alignment : 0; }
int64_t redist_plan_height(const redist_plan_t *plan) { return plan ? plan->p.height : 0; }
int64_t redist_plan_cost(const redist_plan_t *plan) { return plan ? plan->p.cost : 0; }
int32_t redist_plan_num_steps(const redist_plan_t *plan) { return plan ? int32_t(plan->p.steps.size()) : 0; }
int32_t redist_plan_num_launches(const redist_plan_t *plan) { return plan ? int32_t(plan->p.launches.size()) : 0; }

redist_status redist_plan_step_info(const redist_plan_t *plan, int32_t step, redist_step_info *out)
{
    if (!plan || !out || step < 0 || step >= int32_t(plan->p.steps.size())) return REDIST_EINVAL;
    const Step &s = plan->p.steps[step];
    redist_step_info o;
    std::memset(&o, 0, sizeof o);
    o.kind = s.kind;
    o.dim_i = s.dim_i;
    o.dim_j = s.dim_j;
    o.factor = s.factor;
    for (int k = 0; k < plan->p.rank; ++k) {
        o.local_before[k] = s.local_before[k];
        o.local_after[k] = s.local_after[k];
    }
    o.cost = s.cost;
    o.localsize_after = s.localsize_after;
    *out = o;
    return REDIST_OK;
}

redist_status redist_plan_launch_info(const redist_plan_t *plan, int32_t launch, redist_launch_info *out)
{
    if (!plan || !out || launch < 0 || launch >= int32_t(plan->p.launches.size())) return REDIST_EINVAL;
    const Launch &L = plan->p.launches[launch];
    redist_launch_info o;
    std::memset(&o, 0, sizeof o);
    o.first_step = L.first_step;
    o.n_steps = L.n_steps;
    o.kernel = L.kernel;
    o.vector_bytes = int32_t(L.geo.unit_bytes);
    o.run_bytes = L.run_bytes;
    o.bytes_read = L.bytes_read;
    o.bytes_written = L.bytes_written;
    o.n_items = L.geo.n_items;
    o.fanout = int32_t(L.geo.fanout);
    o.variant = L.geo.bulk == 2 ? 6 : L.geo.bulk ? 4 : (L.geo.mode == kModeBox ? 8 : L.geo.mode == kModeZip ? 7 : L.geo.mode == kModeGather ? 5 : L.geo.mode == kModeRows ? 0 : L.geo.mode == kModeUnits ? 3 : (L.geo.aligned ? 1 : 2));
    *out = o;
    return REDIST_OK;
}

size_t redist_plan_describe(const redist_plan_t *plan, char *buf, size_t cap)
{
    if (!plan) return 0;
    const std::string &j = plan->p.json;
    if (buf && cap > 0) {
        size_t n = std::min(cap - 1, j.size());
        std::memcpy(buf, j.data(), n);
        buf[n] = 0;
    }
    return j.size();
}

redist_status redist_execute(const redist_plan_t *plan, const void *const *src_shards, void *const *dst_shards,
                             void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    try {
        if (!plan || !src_shards || !dst_shards) return REDIST_EINVAL;
        const Plan &p = plan->p;
        if (p.scratch_bytes > 0 && (!scratch || scratch_bytes < size_t(p.scratch_bytes))) return REDIST_ESCRATCH;
        return run_plan(p, src_shards, dst_shards, scratch, size_t(p.scratch_bytes), cuda_stream);
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

redist_status redist_bind(const redist_plan_t *plan, const void *const *src_shards, void *const *dst_shards,
                          void *scratch, size_t scratch_bytes, redist_bound_t **out)
{
    if (!plan || !src_shards || !dst_shards || !out) return REDIST_EINVAL;
    const Plan &p = plan->p;
    if (p.scratch_bytes > 0 && (!scratch || scratch_bytes < size_t(p.scratch_bytes))) return REDIST_ESCRATCH;
    const bool small = p.n_devices <= kSmallTable;
    redist_status rc = small ? check_buffers<kSmallTable>(p, src_shards, dst_shards, scratch, size_t(p.scratch_bytes))
                             : check_buffers<kLargeTable>(p, src_shards, dst_shards, scratch, size_t(p.scratch_bytes));
    if (rc != REDIST_OK) return rc;
    try {
        std::unique_ptr<redist_bound_s> b(new redist_bound_s());
        b->ref = plan->ref;
        size_t n = 0;
        for (const Launch &L : p.launches) n += L.geo.n_items != 0;
        b->launches.resize(n);
        b->params.resize(n);
        const size_t bytes = param_bytes(small ? kSmallTable : kLargeTable);
        size_t q = 0;
        for (const Launch &L : p.launches) {
            if (L.geo.n_items == 0) continue;
            b->params[q].resize((bytes + sizeof(max_align_t) - 1) / sizeof(max_align_t));
            char *sc = static_cast<char *>(scratch);
            rc = small ? prepare_launch<kSmallTable>(p, L, src_shards, dst_shards, sc, b->params[q].data(), bytes, b->launches[q])
                       : prepare_launch<kLargeTable>(p, L, src_shards, dst_shards, sc, b->params[q].data(), bytes, b->launches[q]);
            if (rc != REDIST_OK) return rc;
            ++q;
        }
        *out = b.release();
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

redist_status redist_bound_execute(const redist_bound_t *bound, void *cuda_stream)
{
    if (!bound) return REDIST_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    for (const PreparedLaunch &pl : bound->launches) {
        cudaError_t ce = launch_prepared(pl, stream);
        if (ce != cudaSuccess) {
            tl_cuda_error = int(ce);
            return REDIST_ECUDA;
        }
    }
    return REDIST_OK;
}

void redist_bound_destroy(redist_bound_t *bound) { delete bound; }

redist_status redist_execute_host(const redist_plan_t *plan, const void *const *src_host, void *const *dst_host,
                                  void *dev_src, size_t dev_src_bytes, void *dev_dst, size_t dev_dst_bytes,
                                  void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    try {
        if (!plan || !src_host || !dst_host || !dev_src || !dev_dst) return REDIST_EINVAL;
        const Plan &p = plan->p;
        const int N = p.n_devices;
        if (dev_src_bytes < redist_plan_staging_bytes(plan, 0) || dev_dst_bytes < redist_plan_staging_bytes(plan, 1))
            return REDIST_ESCRATCH;
        if ((uintptr_t(dev_src) & 255) || (uintptr_t(dev_dst) & 255)) return REDIST_EALIGN;
        const i64 sb = p.local_src * p.elem_bytes, db = p.local_dst * p.elem_bytes;
        const i64 sp = (sb + 255) / 256 * 256, dp = (db + 255) / 256 * 256;
        cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
        const void *s[REDIST_MAX_DEVICES];
        void *t[REDIST_MAX_DEVICES];
        for (int d = 0; d < N; ++d) {
            if (!src_host[d] || !dst_host[d]) return REDIST_EINVAL;
            s[d] = static_cast<char *>(dev_src) + d * sp;
            t[d] = static_cast<char *>(dev_dst) + d * dp;
        }
        for (int d = 0; d < N; ++d) {
            cudaError_t ce = cudaMemcpyAsync(const_cast<void *>(s[d]), src_host[d], size_t(sb), cudaMemcpyHostToDevice, stream);
            if (ce != cudaSuccess) {
                tl_cuda_error = int(ce);
                return REDIST_ECUDA;
            }
        }
        redist_status rc = redist_execute(plan, s, t, scratch, scratch_bytes, cuda_stream);
        if (rc != REDIST_OK) return rc;
        for (int d = 0; d < N; ++d) {
            cudaError_t ce = cudaMemcpyAsync(dst_host[d], t[d], size_t(db), cudaMemcpyDeviceToHost, stream);
            if (ce != cudaSuccess) {
                tl_cuda_error = int(ce);
                return REDIST_ECUDA;
            }
        }
        return REDIST_OK;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

}  // extern "C"
