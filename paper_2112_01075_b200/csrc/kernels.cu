// sm_100a copy kernels of the executor.
//
// Every collective of a redistribution moves bytes and never interprets them (Section 4.2: the
// meaning of a collective is how it changes the placement of tiles).  On one GPU, with every
// virtual device's tile in its own buffer, a collective -- or a fused run of them -- is therefore a
// strided gather/scatter between two layouts of the same global array, described by CopyGeometry
// (copy_params.h).  The work is bound by HBM bandwidth: every source byte is read once, with the
// widest access the strides allow (16 bytes in all benchmark shapes), and written once per target
// replica from registers (allgather stores the same registers `fanout` times instead of re-reading).
//
// Thread mapping: a block of 256 threads covers rows_per_pass rows of `lanes` vectors; a thread
// keeps its column and walks down the rows of its work item, issuing kUnroll independent loads
// before the matching stores.  All index decoding uses multiply-shift division by constants that
// the host precomputed; the per-item decode (box -> tiles and base offsets) is amortised over
// ~32 KiB of data.
#include <cuda_runtime.h>

#include "copy_params.h"
#include "kernels.h"

namespace redist {

namespace {

#ifndef REDIST_UNROLL
#define REDIST_UNROLL 4
#endif
constexpr int kUnroll = REDIST_UNROLL;

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv &f)
{
    return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

template <int VEC> struct VecType;
template <> struct VecType<16> { using T = uint4; };
template <> struct VecType<8> { using T = uint2; };
template <> struct VecType<4> { using T = uint32_t; };
template <> struct VecType<2> { using T = uint16_t; };
template <> struct VecType<1> { using T = uint8_t; };

// streaming accesses: the data is touched once (cache-streaming loads and stores)
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ uint2 ld_stream(const uint2 *p) { return __ldcs(p); }
__device__ __forceinline__ uint32_t ld_stream(const uint32_t *p) { return __ldcs(p); }
__device__ __forceinline__ uint16_t ld_stream(const uint16_t *p) { return __ldcs(p); }
__device__ __forceinline__ uint8_t ld_stream(const uint8_t *p) { return __ldcs(p); }

__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint2 *p, const uint2 &v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint32_t *p, uint32_t v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint16_t *p, uint16_t v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint8_t *p, uint8_t v) { __stcs(p, v); }

template <int VEC, int NT>
__device__ __forceinline__ void copy_body(const CopyParams<NT> &P)
{
    using T = typename VecType<VEC>::T;
    const CopyGeometry &g = P.g;
    const uint32_t tid = threadIdx.x;
    const uint32_t ty = fdiv(tid, g.lanes_div);
    const uint32_t tx = tid - ty * g.lanes;
    const bool active = ty < g.rows_per_pass;
    const uint32_t rpp = g.rows_per_pass;
    const uint32_t fanout = g.fanout;
    const int n_row = int(g.n_row);

    for (uint32_t item = blockIdx.x; item < g.n_items; item += gridDim.x) {
        const uint32_t box = fdiv(item, g.items_per_box);
        const uint32_t chunk = item - box * g.items_per_box.d;
        // box -> source tile / target tile and the byte offsets of the box inside them
        uint32_t t1 = 0, t2 = 0, rem = box;
        int64_t o1 = 0, o2 = 0;
        for (int u = int(g.n_unit) - 1; u >= 0; --u) {
            const uint32_t nxt = fdiv(rem, g.unit_n[u]);
            const uint32_t q = rem - nxt * g.unit_n[u].d;
            rem = nxt;
            const uint32_t a1 = fdiv(q, g.unit_m1[u]);
            const uint32_t a2 = fdiv(q, g.unit_m2[u]);
            t1 += a1 * g.unit_ts1[u];
            t2 += a2 * g.unit_ts2[u];
            o1 += int64_t(q - a1 * g.unit_m1[u].d) * g.unit_b1[u];
            o2 += int64_t(q - a2 * g.unit_m2[u].d) * g.unit_b2[u];
        }
        const char *sbase = P.src[t1] + o1 + int64_t(tx) * VEC;
        const int64_t dcol = o2 + int64_t(tx) * VEC;
        char *const *dtab = &P.dst[t2 * fanout];
        const uint32_t row0 = chunk * g.rows_per_item;
        const uint32_t row_end = min(row0 + g.rows_per_item, g.rows);

        for (uint32_t rb = row0; rb < row_end; rb += rpp * kUnroll) {
            T v[kUnroll];
            int64_t d2[kUnroll];
            bool ok[kUnroll];
#pragma unroll
            for (int k = 0; k < kUnroll; ++k) {
                const uint32_t row = rb + k * rpp + ty;
                ok[k] = active && row < row_end;
                int64_t s1 = 0, s2 = 0;
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
                d2[k] = s2;
                if (ok[k]) v[k] = ld_stream(reinterpret_cast<const T *>(sbase + s1));
            }
            for (uint32_t f = 0; f < fanout; ++f) {
                char *dbase = dtab[f] + dcol;
#pragma unroll
                for (int k = 0; k < kUnroll; ++k)
                    if (ok[k]) st_stream(reinterpret_cast<T *>(dbase + d2[k]), v[k]);
            }
        }
    }
}

// One entry per collective so that profiles name the step that ran.
#define REDIST_DEFINE_KERNEL(NAME)                                                               \
    template <int VEC, int NT>                                                                   \
    __global__ void __launch_bounds__(kBlockThreads) NAME(const __grid_constant__ CopyParams<NT> P) \
    {                                                                                            \
        copy_body<VEC, NT>(P);                                                                   \
    }

REDIST_DEFINE_KERNEL(redist_dynslice_kernel)
REDIST_DEFINE_KERNEL(redist_alltoall_kernel)
REDIST_DEFINE_KERNEL(redist_allgather_kernel)
REDIST_DEFINE_KERNEL(redist_allpermute_kernel)
REDIST_DEFINE_KERNEL(redist_fused_kernel)

template <int VEC, int NT>
cudaError_t launch_vec_nt(int kernel, const CopyParams<NT> &P, int grid, cudaStream_t stream)
{
    switch (kernel) {
    case 0: case 7: redist_dynslice_kernel<VEC, NT><<<grid, kBlockThreads, 0, stream>>>(P); break;
    case 1: redist_alltoall_kernel<VEC, NT><<<grid, kBlockThreads, 0, stream>>>(P); break;
    case 2: case 6: redist_allgather_kernel<VEC, NT><<<grid, kBlockThreads, 0, stream>>>(P); break;
    case 3: case 4: redist_allpermute_kernel<VEC, NT><<<grid, kBlockThreads, 0, stream>>>(P); break;
    default: redist_fused_kernel<VEC, NT><<<grid, kBlockThreads, 0, stream>>>(P); break;
    }
    return cudaGetLastError();
}

template <int NT>
cudaError_t launch_nt(int kernel, const CopyParams<NT> &P, int grid, cudaStream_t stream)
{
    switch (P.g.vec_bytes) {
    case 16: return launch_vec_nt<16, NT>(kernel, P, grid, stream);
    case 8: return launch_vec_nt<8, NT>(kernel, P, grid, stream);
    case 4: return launch_vec_nt<4, NT>(kernel, P, grid, stream);
    case 2: return launch_vec_nt<2, NT>(kernel, P, grid, stream);
    default: return launch_vec_nt<1, NT>(kernel, P, grid, stream);
    }
}

}  // namespace

cudaError_t launch_copy(int kernel, const CopyGeometry &geo, const char *const *src_tab, int n_src,
                        char *const *dst_tab, int n_dst, int grid, cudaStream_t stream)
{
    if (n_src <= kSmallTable && n_dst <= kSmallTable) {
        CopyParams<kSmallTable> P;
        P.g = geo;
        for (int i = 0; i < n_src; ++i) P.src[i] = src_tab[i];
        for (int i = 0; i < n_dst; ++i) P.dst[i] = dst_tab[i];
        return launch_nt<kSmallTable>(kernel, P, grid, stream);
    }
    if (n_src > kLargeTable || n_dst > kLargeTable) return cudaErrorInvalidValue;
    CopyParams<kLargeTable> P;
    P.g = geo;
    for (int i = 0; i < n_src; ++i) P.src[i] = src_tab[i];
    for (int i = 0; i < n_dst; ++i) P.dst[i] = dst_tab[i];
    return launch_nt<kLargeTable>(kernel, P, grid, stream);
}

}  // namespace redist
