/*
 * TEST INFRASTRUCTURE -- the CPU oracle for array redistribution.  Not part of the product:
 * only tests, the smoke check and the benchmark's CPU-baseline leg may build or call this file.
 * It shares no code, header or table with the CUDA library.
 *
 * What it computes is the *definition* of a redistribution, not the paper's algorithm:
 *   1. every device's base offset under a distributed type  (base offset maps D[[.]] and T[[.]],
 *      the figure "Semantics for distributed dimensions and types", part (a); axis order inside
 *      a dimension is minor-to-major, Section 2.1);
 *   2. the logical global array is assembled from the source tiles, tile of device d placed at
 *      its base offset (Section 4.1, "Semantics for distributed array types");
 *   3. every device's target tile is the slice of that global array at its base offset under the
 *      target type.  The data of the global array never changes during redistribution
 *      (Section 4.2), so exactly one result is correct.
 * There is no plan, no collective, no blocking beyond a row-wise memcpy of the last dimension.
 *
 * Conventions the paper leaves open (chosen once, the same on both sides): tiles are dense
 * row-major; a device id is the row-major index of its coordinates over mesh_shape (last mesh
 * axis fastest).
 *
 * Pins (tests, no GPU): the worked example [8{"x","y"}32] of Section 2.1; the lemma that the
 * image of D[[c{xs}n]] is all multiples of c below n; brute-force ownership enumeration written
 * separately in Python; the closed form for a linear-index fill; a numpy stack/transpose
 * formulation for 1-D meshes; A->B->A round trips.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_MAX_RANK 16
#define ORC_MAX_AXES 32

enum { ORC_OK = 0, ORC_EINVAL = 1, ORC_EILLFORMED = 2, ORC_ENOTDIV = 3, ORC_EMISMATCH = 4 };

static int g_threads = 1;

void orc_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int orc_get_threads(void) { return g_threads; }

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

static int64_t n_devices(int n_axes, const int64_t *mesh_shape)
{
    int64_t n = 1;
    for (int a = 0; a < n_axes; ++a) n *= mesh_shape[a];
    return n;
}

/*
 * Well-formedness (rules wf-dim and wf-type) and the tile sizes c_k = s_k / prod(axis sizes).
 */
static int check_type(int n_axes, const int64_t *mesh_shape, int rank, const int64_t *gshape,
                      const int32_t *axes_off, const int32_t *axes, int64_t *tile)
{
    int used[ORC_MAX_AXES] = {0};
    if (n_axes < 0 || n_axes > ORC_MAX_AXES || rank < 1 || rank > ORC_MAX_RANK) return ORC_EINVAL;
    for (int a = 0; a < n_axes; ++a)
        if (mesh_shape[a] < 1) return ORC_EINVAL;
    for (int k = 0; k < rank; ++k) {
        int64_t prod = 1;
        if (gshape[k] < 1) return ORC_EINVAL;
        for (int32_t p = axes_off[k]; p < axes_off[k + 1]; ++p) {
            int32_t a = axes[p];
            if (a < 0 || a >= n_axes) return ORC_EILLFORMED;   /* axis must exist in the mesh  */
            if (used[a]) return ORC_EILLFORMED;                /* distinct within and across dims */
            used[a] = 1;
            prod *= mesh_shape[a];
        }
        if (gshape[k] % prod != 0) return ORC_ENOTDIV;         /* c * prod(k_i) = n              */
        tile[k] = gshape[k] / prod;
    }
    return ORC_OK;
}

/*
 * Base offset of one device in one dimension:
 *   D[[c{}c]](i) = 0,   D[[c{x,xs}n]](i) = c*i_x + D[[(c*k){xs}n]](i),  k = size of axis x.
 * Written as the recursion unrolled from the minor-most (first listed) axis outwards.
 */
static int64_t dim_offset(const int64_t *mesh_shape, const int64_t *coord, int64_t c,
                          const int32_t *axes, int n)
{
    int64_t off = 0;
    for (int p = 0; p < n; ++p) {
        off += c * coord[axes[p]];
        c *= mesh_shape[axes[p]];
    }
    return off;
}

/* coordinates of device d: row-major unravel over mesh_shape, last axis fastest */
static void device_coord(int n_axes, const int64_t *mesh_shape, int64_t d, int64_t *coord)
{
    for (int a = n_axes - 1; a >= 0; --a) {
        coord[a] = d % mesh_shape[a];
        d /= mesh_shape[a];
    }
}

/*
 * tile_out[rank]        local tile shape (localtype)
 * off_out[N * rank]     base offset T[[tau]](d) for every device d
 */
int orc_base_offsets(int n_axes, const int64_t *mesh_shape, int rank, const int64_t *gshape,
                     const int32_t *axes_off, const int32_t *axes, int64_t *tile_out, int64_t *off_out)
{
    int64_t tile[ORC_MAX_RANK], coord[ORC_MAX_AXES];
    int rc = check_type(n_axes, mesh_shape, rank, gshape, axes_off, axes, tile);
    if (rc) return rc;
    int64_t N = n_devices(n_axes, mesh_shape);
    for (int k = 0; k < rank; ++k) tile_out[k] = tile[k];
    for (int64_t d = 0; d < N; ++d) {
        device_coord(n_axes, mesh_shape, d, coord);
        for (int k = 0; k < rank; ++k)
            off_out[d * rank + k] = dim_offset(mesh_shape, coord, tile[k], axes + axes_off[k],
                                               axes_off[k + 1] - axes_off[k]);
    }
    return ORC_OK;
}

/*
 * Copy rows [row_begin, row_end) of one tile between the tile buffer and the global array.
 * A "row" is one run of the last dimension; rows are numbered row-major over the leading
 * dimensions of the tile.  to_global != 0: tile -> G; otherwise G -> tile.
 * With compare != 0 nothing is written: returns 1 if any byte differs.
 */
static int tile_rows(int rank, const int64_t *gshape, const int64_t *tile, const int64_t *off, int e,
                     unsigned char *G, unsigned char *T, int to_global, int compare, int64_t row_begin,
                     int64_t row_end)
{
    int64_t idx[ORC_MAX_RANK];
    int64_t run = tile[rank - 1] * (int64_t)e;
    int diff = 0;
    for (int64_t row = row_begin; row < row_end; ++row) {
        int64_t r = row;
        for (int k = rank - 2; k >= 0; --k) {
            idx[k] = r % tile[k];
            r /= tile[k];
        }
        int64_t g = 0;                                   /* global linear element index of the row start */
        for (int k = 0; k < rank - 1; ++k) g = (g + off[k] + idx[k]) * gshape[k + 1];
        g += off[rank - 1];
        unsigned char *gp = G + g * (int64_t)e;
        unsigned char *tp = T + row * run;
        if (compare)
            diff |= memcmp(gp, tp, (size_t)run) != 0;
        else if (to_global)
            memcpy(gp, tp, (size_t)run);
        else
            memcpy(tp, gp, (size_t)run);
    }
    return diff;
}

static int64_t tile_row_count(int rank, const int64_t *tile)
{
    int64_t n = 1;
    for (int k = 0; k < rank - 1; ++k) n *= tile[k];
    return n;
}

/*
 * Assemble the global array G (row-major, prod(gshape)*elem_bytes bytes) from the source tiles.
 * Where several devices hold the same tile (replication: axes the type does not use), the lowest
 * device id writes; with check != 0 the others are compared and ORC_EMISMATCH is returned if a
 * replica differs.
 */
int orc_materialize(int n_axes, const int64_t *mesh_shape, int rank, const int64_t *gshape,
                    const int32_t *axes_off, const int32_t *axes, int elem_bytes,
                    const void *const *shards, void *G, int check)
{
    int64_t tile[ORC_MAX_RANK];
    int64_t N = n_devices(n_axes, mesh_shape);
    int64_t *off = (int64_t *)malloc((size_t)N * rank * sizeof(int64_t));
    char *first = (char *)malloc((size_t)N);
    if (!off || !first) { free(off); free(first); return ORC_EINVAL; }
    int rc = orc_base_offsets(n_axes, mesh_shape, rank, gshape, axes_off, axes, tile, off);
    if (rc) { free(off); free(first); return rc; }
    for (int64_t d = 0; d < N; ++d) {
        first[d] = 1;
        for (int64_t p = 0; p < d && first[d]; ++p)
            if (memcmp(off + p * rank, off + d * rank, (size_t)rank * sizeof(int64_t)) == 0) first[d] = 0;
    }
    int64_t rows = tile_row_count(rank, tile);
    int64_t chunk = rows < 64 ? rows : 64;
    int64_t nchunk = (rows + chunk - 1) / chunk;
    int mismatch = 0;
    for (int pass = 0; pass < (check ? 2 : 1); ++pass) {
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads) reduction(| : mismatch)
#endif
        for (int64_t w = 0; w < N * nchunk; ++w) {
            int64_t d = w / nchunk, c = w % nchunk;
            if ((pass == 0) != (first[d] != 0)) continue;
            int64_t rb = c * chunk, re = rb + chunk < rows ? rb + chunk : rows;
            mismatch |= tile_rows(rank, gshape, tile, off + d * rank, elem_bytes, (unsigned char *)G,
                                  (unsigned char *)shards[d], 1, pass == 1, rb, re);
        }
    }
    free(off);
    free(first);
    return mismatch ? ORC_EMISMATCH : ORC_OK;
}

/* Slice every device's tile out of the global array G under the given type. */
int orc_reslice(int n_axes, const int64_t *mesh_shape, int rank, const int64_t *gshape,
                const int32_t *axes_off, const int32_t *axes, int elem_bytes, const void *G,
                void *const *shards)
{
    int64_t tile[ORC_MAX_RANK];
    int64_t N = n_devices(n_axes, mesh_shape);
    int64_t *off = (int64_t *)malloc((size_t)N * rank * sizeof(int64_t));
    if (!off) return ORC_EINVAL;
    int rc = orc_base_offsets(n_axes, mesh_shape, rank, gshape, axes_off, axes, tile, off);
    if (rc) { free(off); return rc; }
    int64_t rows = tile_row_count(rank, tile);
    int64_t chunk = rows < 64 ? rows : 64;
    int64_t nchunk = (rows + chunk - 1) / chunk;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
    for (int64_t w = 0; w < N * nchunk; ++w) {
        int64_t d = w / nchunk, c = w % nchunk;
        int64_t rb = c * chunk, re = rb + chunk < rows ? rb + chunk : rows;
        tile_rows(rank, gshape, tile, off + d * rank, elem_bytes, (unsigned char *)G,
                  (unsigned char *)shards[d], 0, 0, rb, re);
    }
    free(off);
    return ORC_OK;
}
