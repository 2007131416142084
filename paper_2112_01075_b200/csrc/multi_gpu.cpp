// Virtual devices spread over several GPUs: who would move how many bytes to whom.
//
// The paper runs its collectives between real devices (Section 8: eight of them) and its Discussion
// (Section 9) raises the alternative of individual device-to-device transfers computed from the base
// offset maps.  With the virtual devices of a plan assigned to G GPUs by a prefix of the mesh axes --
// device d lives on GPU d / (N / G), i.e. the leading mesh coordinates choose the GPU -- every launch of
// the plan splits into a part that stays inside a GPU and a part that crosses to a peer.  This file only
// does the accounting (host side, no CUDA): the matrix of bytes written, by the GPU that reads them and
// the GPU that receives them.  The data plane it describes: each GPU runs the launch restricted to the
// source tiles it holds and stores into its own or a peer's destination tiles; loads never leave the GPU.
// A replicated source tile is read from a replica on the receiving GPU when there is one.
#include <algorithm>

#include "plan.hpp"

using namespace redist;

extern "C" redist_status redist_plan_gpu_split(const redist_plan_t *plan, int32_t n_gpus, int32_t launch,
                                               int64_t *bytes)
{
    try {
        if (!plan || !bytes || n_gpus < 1 || launch < 0 || launch >= int32_t(plan->p.launches.size()))
            return REDIST_EINVAL;
        const Plan &p = plan->p;
        const int N = p.n_devices;
        // a prefix of the mesh axes: G = (sizes of the leading axes) * (a divisor of the next one)
        {
            i64 g = n_gpus;
            for (int a = 0; a < p.n_mesh_axes && g > 1; ++a) {
                const i64 k = p.mesh_shape[a];
                if (g >= k) {
                    if (g % k) return REDIST_EINVAL;
                    g /= k;
                } else {
                    if (k % g) return REDIST_EINVAL;
                    g = 1;
                }
            }
            if (g != 1) return REDIST_EINVAL;
        }
        const int per_gpu = N / n_gpus;
        auto gpu_of = [&](int d) { return d / per_gpu; };
        const Launch &L = p.launches[size_t(launch)];
        std::fill(bytes, bytes + size_t(n_gpus) * n_gpus, int64_t(0));
        // tile shapes and tile counts of the two layouts of this launch
        const int r = p.rank;
        std::vector<i64> c1(r), c2(r), n1(r), n2(r);
        for (int k = 0; k < r; ++k) {
            c1[k] = L.src_tile[size_t(k)];
            c2[k] = L.dst_tile[size_t(k)];
            n1[k] = p.global_shape[size_t(k)] / c1[k];
            n2[k] = p.global_shape[size_t(k)] / c2[k];
        }
        const i64 nt1 = i64(L.src_holder.size()), nt2 = i64(L.dst_devs.size()) / std::max<i64>(1, L.geo.fanout);
        // holders of every source tile, by GPU: holder_on[t1 * G + g] = a device of GPU g that holds t1, or -1
        std::vector<int32_t> holder_on(size_t(nt1) * n_gpus, -1);
        for (int d = N - 1; d >= 0; --d)
            if (L.src_tile_of[size_t(d)] >= 0) holder_on[size_t(L.src_tile_of[size_t(d)]) * n_gpus + gpu_of(d)] = d;
        std::vector<i64> i1(r), i2(r);
        for (i64 t2 = 0; t2 < nt2; ++t2) {
            i64 rem = t2;
            for (int k = r - 1; k >= 0; --k) {
                i2[k] = rem % n2[k];
                rem /= n2[k];
            }
            // source tiles that meet target tile t2: per dimension a range of tile indices
            std::vector<i64> lo(r), hi(r);
            for (int k = 0; k < r; ++k) {
                lo[k] = i2[k] * c2[k] / c1[k];
                hi[k] = ((i2[k] + 1) * c2[k] - 1) / c1[k];
            }
            i1 = lo;
            while (true) {
                i64 t1 = 0, vol = p.elem_bytes;
                for (int k = 0; k < r; ++k) {
                    t1 = t1 * n1[k] + i1[k];
                    const i64 a = std::max(i1[k] * c1[k], i2[k] * c2[k]);
                    const i64 b = std::min((i1[k] + 1) * c1[k], (i2[k] + 1) * c2[k]);
                    vol *= std::max<i64>(0, b - a);
                }
                for (uint32_t f = 0; f < L.geo.fanout; ++f) {
                    const int32_t dev = L.dst_devs[size_t(t2) * L.geo.fanout + f];
                    const int gd = dev < 0 ? 0 : gpu_of(dev);
                    int gs = gd;                                   // a replica on the receiving GPU, if any
                    if (L.src_holder[size_t(t1)] < 0) {
                        gs = 0;                                    // shared buffer of the naive baseline
                    } else if (holder_on[size_t(t1) * n_gpus + gd] < 0) {
                        gs = gpu_of(L.src_holder[size_t(t1)]);
                    }
                    bytes[size_t(gs) * n_gpus + gd] += vol;
                }
                int k = r - 1;
                while (k >= 0 && ++i1[k] > hi[k]) {
                    i1[k] = lo[k];
                    --k;
                }
                if (k < 0) break;
            }
        }
        return REDIST_OK;
    } catch (const std::bad_alloc &) {
        return REDIST_ENOMEM;
    } catch (...) {
        return REDIST_EINTERNAL;
    }
}
