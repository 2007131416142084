// The C boundary: plan creation, execution and queries.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "kernels.h"
#include "plan.hpp"

using namespace redist;

namespace redist {
thread_local int tl_cuda_error = 0;
}

namespace {

// One thread block per work item by default: the hardware block scheduler balances the load and
// keeps the tail to one item.  REDIST_GRID_MULT=k (tuning knob) switches to a grid-stride loop with
// k blocks per SM.
int grid_for(const CopyGeometry &g)
{
    static const long long cap = [] {
        const char *m = std::getenv("REDIST_GRID_MULT");
        if (!m || std::atoi(m) <= 0) return 0ll;
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        return 1ll * n * std::atoi(m);
    }();
    return int(cap > 0 ? std::min<long long>(g.n_items, cap) : g.n_items);
}

struct Range {
    uintptr_t lo, hi;
    int kind;   // 0 source (may alias other sources), 1 written
};

bool overlaps(std::vector<Range> &r)
{
    std::sort(r.begin(), r.end(), [](const Range &a, const Range &b) { return a.lo < b.lo; });
    // sweep: a written range may not intersect any other range; sources may intersect sources
    uintptr_t max_hi_written = 0, max_hi_any = 0;
    bool have_w = false, have_any = false;
    for (const Range &x : r) {
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

}  // namespace

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
    if (flags & ~uint32_t(REDIST_MODE_MASK | REDIST_NO_OVERPARTITION | REDIST_COST_PERMUTE)) return REDIST_EINVAL;
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
    redist_plan_s *h = new (std::nothrow) redist_plan_s();
    if (!h) return REDIST_ENOMEM;
    try {
        Plan &p = h->p;
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
    } catch (const std::bad_alloc &) {
        rc = REDIST_ENOMEM;
    } catch (...) {
        rc = REDIST_EINTERNAL;
    }
    if (rc != REDIST_OK) {
        delete h;
        return rc;
    }
    *out = h;
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
    o.variant = L.geo.bulk == 2 ? 6 : L.geo.bulk ? 4 : (L.geo.mode == kModeZip ? 7 : L.geo.mode == kModeGather ? 5 : L.geo.mode == kModeRows ? 0 : L.geo.mode == kModeUnits ? 3 : (L.geo.aligned ? 1 : 2));
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
        const int N = p.n_devices;
        if (p.scratch_bytes > 0 && (!scratch || scratch_bytes < size_t(p.scratch_bytes))) return REDIST_ESCRATCH;
        const uintptr_t amask = uintptr_t(p.alignment) - 1;
        const i64 sb = p.local_src * p.elem_bytes, db = p.local_dst * p.elem_bytes;
        std::vector<Range> ranges;
        ranges.reserve(size_t(2 * N + 1));
        for (int d = 0; d < N; ++d) {
            if (!src_shards[d] || !dst_shards[d]) return REDIST_EINVAL;
            const uintptr_t s = uintptr_t(src_shards[d]), t = uintptr_t(dst_shards[d]);
            if ((s & amask) || (t & amask)) return REDIST_EALIGN;
            ranges.push_back(Range{s, s + uintptr_t(sb), 0});
            ranges.push_back(Range{t, t + uintptr_t(db), 1});
        }
        if (p.scratch_bytes > 0) {
            if (uintptr_t(scratch) & 255) return REDIST_EALIGN;
            ranges.push_back(Range{uintptr_t(scratch), uintptr_t(scratch) + uintptr_t(p.scratch_bytes), 1});
        }
        if (overlaps(ranges)) return REDIST_EOVERLAP;

        cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
        auto buffer = [&](BufKind kind, int32_t dev) -> char * {
            switch (kind) {
            case BUF_SRC: return static_cast<char *>(const_cast<void *>(src_shards[dev]));
            case BUF_DST: return static_cast<char *>(dst_shards[dev]);
            case BUF_SCRATCH0: return static_cast<char *>(scratch) + i64(dev) * p.slot_bytes;
            case BUF_SCRATCH1: return static_cast<char *>(scratch) + (i64(N) + dev) * p.slot_bytes;
            default: return static_cast<char *>(scratch);
            }
        };
        std::vector<const char *> stab;
        std::vector<char *> dtab;
        for (const Launch &L : p.launches) {
            stab.resize(L.src_holder.size());
            dtab.resize(L.dst_devs.size());
            for (size_t t = 0; t < stab.size(); ++t) stab[t] = buffer(L.from, L.src_holder[t] < 0 ? 0 : L.src_holder[t]);
            for (size_t t = 0; t < dtab.size(); ++t) dtab[t] = buffer(L.to, L.dst_devs[t] < 0 ? 0 : L.dst_devs[t]);
            if (L.geo.n_items == 0) continue;
            cudaError_t ce = launch_copy(L.kernel, L.geo, stab.data(), int(stab.size()), dtab.data(), int(dtab.size()),
                                         grid_for(L.geo), stream);
            if (ce != cudaSuccess) {
                tl_cuda_error = int(ce);
                return REDIST_ECUDA;
            }
        }
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

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
        std::vector<const void *> s(N);
        std::vector<void *> t(N);
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
        redist_status rc = redist_execute(plan, s.data(), t.data(), scratch, scratch_bytes, cuda_stream);
        if (rc != REDIST_OK) return rc;
        for (int d = 0; d < N; ++d) {
            cudaError_t ce = cudaMemcpyAsync(dst_host[d], t[d], size_t(db), cudaMemcpyDeviceToHost, stream);
            if (ce != cudaSuccess) {
                tl_cuda_error = int(ce);
                return REDIST_ECUDA;
            }
        }
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}

}  // extern "C"
