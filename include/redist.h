/*
 * redist -- array redistribution over a logical device mesh, executed on one NVIDIA B200.
 *
 * The method is the one of "Memory-efficient array redistribution through portable collective
 * communication" (arXiv 2112.01075): a multi-dimensional array is partitioned over a logical mesh
 * under a source distributed type and must reach a target distributed type through a sequence of
 * the collectives allgather, alltoall, dynslice and allpermute.  Here the N mesh devices are
 * *virtual*: every device's tile is its own buffer in the memory of one GPU, and each collective
 * step (or a fused run of adjacent steps) is one CUDA kernel that moves the tiles of all virtual
 * devices at once.
 *
 * Conventions
 *   - A distributed type lists, per array dimension, the mesh axes that partition it, ordered
 *     minor-to-major: the first listed axis varies fastest (Section 2.1, "Distributed array
 *     types").  Tile size = global size / product of the listed axis sizes; it must divide
 *     (rule wf-dim).  Axes a type does not list replicate the data.
 *   - Virtual device id = row-major index of the device's mesh coordinates over mesh_shape
 *     (last mesh axis fastest).  The paper leaves this numbering to the runtime (Section 2.1).
 *   - A tile is dense, row-major, last dimension contiguous, without padding.
 *   - All functions return a redist_status; nothing throws, aborts or prints across this
 *     boundary.  Output arguments are untouched on failure.
 *   - "host" / "device" on a pointer argument says which memory it must point to.
 */
#ifndef REDIST_H_
#define REDIST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum redist_status {
    REDIST_OK = 0,
    REDIST_EINVAL = 1,       /* null pointer, bad rank / element size / flag / index                   */
    REDIST_EILLFORMED = 2,   /* rules wf-dim / wf-type: unknown axis, axis listed twice                */
    REDIST_ENOTDIV = 3,      /* tile size * product of axis sizes != global size (wf-dim)             */
    REDIST_EGLOBAL = 4,      /* source and target describe different global arrays (Section 2.5)      */
    REDIST_ESCRATCH = 5,     /* scratch buffer missing or smaller than redist_plan_scratch_bytes      */
    REDIST_EOVERLAP = 6,     /* destination / scratch ranges overlap each other or a source           */
    REDIST_EALIGN = 7,       /* a buffer is not aligned to redist_plan_alignment bytes                */
    REDIST_ENOMEM = 8,       /* host allocation failed                                                */
    REDIST_ECUDA = 9,        /* a CUDA call or kernel launch reported an error                        */
    REDIST_EUNSUPPORTED = 10,/* beyond a built-in limit (devices, rank, sizes); see redist_limits     */
    REDIST_EINTERNAL = 11    /* the synthesized plan failed its own end-state check (a bug)           */
} redist_status;

/*
 * A distributed type.  rank dimensions; global_shape[rank]; the axes of dimension k are
 * axes[axes_off[k] .. axes_off[k+1]) as indices into mesh_shape, minor-to-major.  All arrays are
 * host memory, read during the call only.
 */
typedef struct redist_type {
    int32_t rank;
    const int64_t *global_shape;
    const int32_t *axes_off;     /* rank + 1 entries, axes_off[0] == 0 */
    const int32_t *axes;         /* axes_off[rank] entries             */
} redist_type;

typedef struct redist_plan_s redist_plan_t;   /* opaque, host memory, immutable once created */

/* plan flags: exactly one execution mode, optionally or-ed with REDIST_NO_OVERPARTITION,
   REDIST_COST_PERMUTE and/or REDIST_NO_CACHE */
enum {
    REDIST_FUSE_ADJACENT = 0,    /* default: adjacent steps of the sequence run as one kernel wherever
                                    the fused copy keeps contiguous runs of at least 64 bytes         */
    REDIST_FUSE_NONE = 1,        /* one kernel per collective of the sequence; intermediates ping-pong
                                    between two scratch slots per virtual device                      */
    REDIST_FUSE_ALL = 2,         /* the whole sequence as a single kernel, no scratch                  */
    REDIST_NAIVE = 3,            /* comparison baseline only: gather the whole global array, then
                                    slice (the "easy" redistribution, Section 4.3)                    */
    REDIST_MODE_MASK = 3,
    REDIST_NO_OVERPARTITION = 16,/* forbid dynslice steps that partition the array over more mesh
                                    axes than the target type uses (over-partitioning, Section 7.2)  */
    REDIST_COST_PERMUTE = 32,    /* count the final allpermute when choosing the sequence.  The search
                                    of Section 7.3 weighs only dynslice / alltoall / allgather (the
                                    permutation carries no edge weight there) and appends the
                                    permutation afterwards; with this flag the sequences whose own cost
                                    lies below that plan's total are lowered too and the cheapest total
                                    (sequence plus permutation, cost model of Section 6.2) is kept.  The
                                    result never costs more than the default plan and obeys the same
                                    memory bound; planning takes longer.                              */
    REDIST_NO_CACHE = 64         /* synthesize afresh instead of consulting the plan cache             */
};

enum { REDIST_MAX_RANK = 8, REDIST_MAX_MESH_AXES = 16, REDIST_MAX_DEVICES = 1024 };

typedef enum redist_step_kind {
    REDIST_STEP_DYNSLICE = 0,
    REDIST_STEP_ALLTOALL = 1,
    REDIST_STEP_ALLGATHER = 2,
    REDIST_STEP_ALLPERMUTE = 3,
    REDIST_STEP_COPY = 4          /* only for an empty sequence (equal types): tiles are copied    */
} redist_step_kind;

/* One collective of the synthesized sequence (Sections 6 and 7). */
typedef struct redist_step_info {
    int32_t kind;                              /* redist_step_kind                                    */
    int32_t dim_i;                             /* dimension the axes leave (or are sliced into); -1   */
    int32_t dim_j;                             /* alltoall: dimension the axes move to; else -1       */
    int64_t factor;                            /* n = product of the sizes of the axes acted on       */
    int64_t local_before[REDIST_MAX_RANK];     /* localtype before the step                           */
    int64_t local_after[REDIST_MAX_RANK];      /* localtype after the step                            */
    int64_t cost;                              /* cost model of the paper, in elements per device     */
    int64_t localsize_after;                   /* elements per device after the step (for the height) */
} redist_step_info;

/* One kernel launch of the executor. */
typedef struct redist_launch_info {
    int32_t first_step, n_steps;   /* the collectives this launch covers                               */
    int32_t kernel;                /* 0 dynslice, 1 alltoall, 2 allgather, 3 allpermute, 4 copy,
                                      5 fused sequence, 6 naive gather, 7 naive slice                  */
    int32_t vector_bytes;          /* bytes per global memory access                                   */
    int64_t run_bytes;             /* shortest contiguous run                                          */
    int64_t bytes_read;            /* HBM bytes the launch reads (every source element once)          */
    int64_t bytes_written;         /* HBM bytes the launch writes                                      */
    int64_t n_items;               /* work items (thread-block sized pieces)                           */
    int32_t fanout;                /* destination replicas stored per element read                     */
    int32_t variant;               /* kernel variant: 0 rows, 1 chunks, 2 ragged chunks, 3 units (register
                                      kernels), 4 TMA bulk copies, 5 gather walk, 6 ragged rows loaded by
                                      TMA bulk copies, 7 zip through shared memory, 8 super-boxes through
                                      shared memory; the kernel is named
                                      redist_<collective>[_bulk|_gather|_ragged_bulk|_zip|_box]_kernel
                                      (variants 5, 7 and 8 on units of 1 or 2 bytes: redist_fused_..._kernel
                                      whatever the collective)                                        */
} redist_launch_info;

/*
 * redist_plan -- synthesize the sequence of collectives from src to dst (host only, no CUDA call).
 *
 * Follows Section 7: decompose the mesh into prime-sized axes (Principle 1, Section 3), search the
 * graph of weak types (nodes: local types with localsize <= max(localsize src, localsize dst);
 * edges: multi-axes dynslice / alltoall / allgather weighted by the cost model) for a shortest
 * path, lower it to device-map collectives (Lowering Theorem, Section 6.1), and append at most one
 * allpermute, placed before any trailing allgathers (Section 7.3).
 *
 *   n_mesh_axes, mesh_shape[n_mesh_axes]   host; the logical mesh, sizes >= 1
 *   src, dst                               host; distributed types over that mesh
 *   elem_bytes                             1, 2, 4, 8 or 16; elements are copied, never interpreted
 *   flags                                  see above
 *   out                                    host; receives the plan, owned by the caller until
 *                                          redist_plan_destroy
 * Plans are cached (the evaluation of Section 8 asks how long synthesis takes; a runtime asks for the
 * same few redistributions over and over): a second request for the same mesh, types, element size,
 * flags and tuning values returns a handle to the same immutable plan without searching again.  The
 * cache keeps the 256 most recently created plans; every handle must still be destroyed.
 * Errors: EINVAL, EILLFORMED, ENOTDIV, EGLOBAL, EUNSUPPORTED, ENOMEM, EINTERNAL.
 */
redist_status redist_plan(int32_t n_mesh_axes, const int64_t *mesh_shape, const redist_type *src,
                          const redist_type *dst, int32_t elem_bytes, uint32_t flags, redist_plan_t **out);

void redist_plan_destroy(redist_plan_t *plan);

/* Plan cache counters since the library was loaded or the cache was last cleared (any may be NULL). */
void redist_plan_cache_stats(int64_t *hits, int64_t *misses, int64_t *entries);
void redist_plan_cache_clear(void);

/*
 * Tuning values -- process-wide, copied into every plan created afterwards (existing plans keep theirs).
 * Defaults are the measured optima.  Names and ranges:
 *   "bulk"               0/1    1: aligned runs of 512 bytes and more move by TMA bulk copies (default);
 *                               0: register kernels only
 *   "gather"             0..2   gather walk: never / where measured faster (default 1) / wherever it applies
 *   "zip"                0..2   zip kernels: never / only where the gather walk is not chosen / wherever
 *                               they apply (default 2)
 *   "box"                0..2   super-box kernels (several interleaving dimensions staged through shared
 *                               memory at once): never / where the other short-run paths do badly
 *                               (default 1) / wherever they apply
 *   "box_width"          0..256 lanes that share one target range in the super-box kernels (a power of two; other
 *                               values are ignored); 0 (default): a warp or more as a rule, fewer where the units of
 *                               one range would fall into a few shared-memory banks
 *   "zip_walks"          0..7   chunk-to-unit maps the zip kernels may use: 1 periodic + 2 by range +
 *                               4 tabulated (default 7; the flat walk is always available)
 *   "zip_by_range_slots" >= 1   fewest chunk slots of a range for the by-range walk (default 256)
 *   "item_kb"            0..1024 KiB read per work item; 0 (default) = 32 / 16 / 8 by fan-out, and 20 / 12 / 6
 *                               in the bulk-copy kernels
 *   "l2_hint"            0..4   bulk copies of the plain bulk-copy kernels that carry an L2 evict-first policy: none /
 *                               loads / stores / both / stores where every segment goes to four or more replicas
 *                               (default 4)
 *   "piece"              0/1    1 (default): on units of 1 or 2 bytes and runs of 64 bytes and more the super-box
 *                               kernels read a chunk that lies inside one run as one unaligned 16-byte piece; 0: unit by unit
 *   "pdl"                0/1    1: kernels use programmatic dependent launch (default); 0: plain stream order
 *   "nvtx"               0/1    1: redist_execute and redist_execute_static wrap every kernel launch in an NVTX
 *                               range named after the collective, for timeline profilers (default 0)
 *   "step_latency"       >= 0   elements added to the cost of every collective while searching: small
 *                               transfers are bound by per-step latency, not by bytes (Section 8, the
 *                               third research question); 0 (default) is the paper's cost model
 *   "wait_polls"         >= 1   mbarrier polls before a bulk-copy block gives up (default 2^18)
 *   "test_extra_tx"      >= 0   test only: makes every bounded wait run out (see redist_bulk_timeouts)
 *   "test_shrink_tiles"  >= 0   test only: the checked build takes every tile to be that many bytes shorter
 *                               (see redist_debug_bounds_report); no effect on the normal build
 * Errors: EINVAL for an unknown name or a value out of range.
 */
redist_status redist_tuning_set(const char *name, int64_t value);
redist_status redist_tuning_get(const char *name, int64_t *value);
void redist_tuning_reset(void);

/*
 * redist_execute -- run the plan on the GPU (asynchronous on `stream`).
 *
 * Executes the collectives of the plan (typing rules T-AllGather, T-DynSlice, T-AllToAll and
 * T-Permute; low-level forms of Section 6) as strided copy kernels over all virtual devices.  The
 * result on every device is the tile its target type prescribes; data values never change.
 *
 *   src_shards[N]   host array of DEVICE pointers; src_shards[d] holds localsize(src)*elem_bytes
 *                   bytes.  Devices that replicate a tile must hold identical bytes (not checked);
 *                   source pointers may alias each other.  Read only.  When the tile size is not a
 *                   multiple of 16 bytes the kernels may read (never write) up to the next 16-byte
 *                   boundary past the tile's end -- always inside the allocation granule of any
 *                   CUDA allocator, and, as tiles start on 16-byte boundaries, never a byte of
 *                   another tile.
 *   dst_shards[N]   host array of DEVICE pointers; dst_shards[d] receives localsize(dst)*elem_bytes
 *                   bytes.  Every destination is written completely.
 *   scratch         DEVICE pointer to at least redist_plan_scratch_bytes(plan) bytes, or NULL when
 *                   that is 0.  Contents are undefined afterwards.
 *   cuda_stream     a cudaStream_t (NULL = default stream) on the current device
 * Ownership: all buffers and the stream belong to the caller.  The call allocates nothing, on the
 * host or on the device (pointer tables and the kernel parameter block live on the call's stack:
 * about 8 KiB for plans of up to 64 virtual devices, about 100 KiB beyond), copies no table to the device (tables travel as kernel parameters) and does not
 * synchronize.  A plan may be executed from several host threads at once on different streams and
 * buffers.
 * Errors: EINVAL, ESCRATCH, EALIGN (pointers must be multiples of redist_plan_alignment),
 * EOVERLAP (destination and scratch ranges must be disjoint from each other and from every
 * source; checked on the host), ECUDA (launch error; see redist_last_cuda_error).
 */
redist_status redist_execute(const redist_plan_t *plan, const void *const *src_shards,
                             void *const *dst_shards, void *scratch, size_t scratch_bytes,
                             void *cuda_stream);

/*
 * redist_bind / redist_bound_execute -- the same execution split in two for callers that run one
 * redistribution on the same buffers many times (every step of a training loop): binding validates
 * the buffers exactly as redist_execute does and prepares every kernel launch once (entry point,
 * launch shape, parameter block with both pointer tables); executing the bound plan is then the
 * kernel launches and nothing else -- no checks, no table building, no allocation.
 *
 *   redist_bind            arguments as redist_execute; *out receives the bound plan (host memory,
 *                          owned by the caller until redist_bound_destroy; it keeps the plan alive).
 *                          The buffers must stay valid and in place while the bound plan is used.
 *   redist_bound_execute   asynchronous on `cuda_stream`; may be called from several threads at once
 *                          (but the launches of all calls write the same buffers: order them)
 * Errors: redist_bind as redist_execute plus ENOMEM; redist_bound_execute EINVAL, ECUDA.
 */
typedef struct redist_bound_s redist_bound_t;
redist_status redist_bind(const redist_plan_t *plan, const void *const *src_shards, void *const *dst_shards,
                          void *scratch, size_t scratch_bytes, redist_bound_t **out);
redist_status redist_bound_execute(const redist_bound_t *bound, void *cuda_stream);
void redist_bound_destroy(redist_bound_t *bound);

/*
 * redist_execute_host -- the same redistribution for tiles that live in HOST memory.
 *
 * Copies every source tile to dev_src (one cudaMemcpyAsync per tile), runs redist_execute on the
 * staged tiles and copies every result tile back, all on `stream`; returns without synchronizing.
 *
 *   src_host[N], dst_host[N]   host arrays of HOST pointers (pinned memory gives true async copies)
 *   dev_src, dev_dst           DEVICE staging buffers of at least redist_plan_staging_bytes(plan, 0)
 *                              and (plan, 1) bytes: N tiles, each rounded up to 256 bytes
 *   scratch                    as for redist_execute
 * Errors: as redist_execute, plus ESCRATCH for staging buffers that are too small.
 */
redist_status redist_execute_host(const redist_plan_t *plan, const void *const *src_host,
                                  void *const *dst_host, void *dev_src, size_t dev_src_bytes,
                                  void *dev_dst, size_t dev_dst_bytes, void *scratch,
                                  size_t scratch_bytes, void *cuda_stream);

/*
 * redist_execute_static -- redist_execute for callers that cannot supply scratch memory.
 * (The paper has no counterpart: it is a property of this library, not of the method.)
 *
 * Some callers have tiles but no way to allocate: a plug-in inside a server that handed all device
 * memory to a pool at start-up and forbids cudaMalloc afterwards, or a latency-bound path on which
 * an allocation may fail or stall.  For them the ping-pong buffers of an unfused plan come from a
 * fixed array of REDIST_STATIC_SCRATCH_BYTES bytes built into the library image (every GPU that
 * loads the library holds those bytes until the process exits).  The call allocates nothing on
 * the device or the host and calls no allocating routine.
 *
 *   plan            any plan with redist_plan_scratch_bytes(plan) <= REDIST_STATIC_SCRATCH_BYTES;
 *                   a larger plan is refused with REDIST_ESCRATCH and nothing runs
 *   src_shards[N], dst_shards[N], cuda_stream    exactly as for redist_execute
 * Set-up: the first call on each device (with that device current) looks up the device address of
 * the built-in array; make that first call before any stream capture begins.  The address is kept
 * for the life of the process: it does not survive a cudaDeviceReset.
 * Sharing: all calls on a device use the same array.  It keeps whatever the previous call left;
 * nothing in it has to start at zero, because every byte a step reads from it was written by an
 * earlier step of the same call.  Two calls whose kernels may overlap on the GPU (different
 * streams without an ordering between them) race on the array: order them.
 * Errors: EINVAL, ESCRATCH (plan too large), EALIGN, EOVERLAP, EUNSUPPORTED (device index >= 64),
 * ECUDA.  Results are identical to redist_execute with a caller-provided scratch buffer.
 */
#define REDIST_STATIC_SCRATCH_BYTES (8u << 20)
redist_status redist_execute_static(const redist_plan_t *plan, const void *const *src_shards,
                                    void *const *dst_shards, void *cuda_stream);

/* ---- queries (host only) -------------------------------------------------------------------- */

int32_t redist_plan_num_devices(const redist_plan_t *plan);               /* N                        */
int32_t redist_plan_rank(const redist_plan_t *plan);
int64_t redist_plan_local_elems(const redist_plan_t *plan, int32_t which); /* 0: source, 1: target    */
size_t  redist_plan_scratch_bytes(const redist_plan_t *plan);             /* total to pass to execute */
size_t  redist_plan_scratch_bytes_per_device(const redist_plan_t *plan);  /* the per-virtual-device
                                               share; for REDIST_NAIVE the size of the global array,
                                               which the literal method would hold on every device   */
size_t  redist_plan_staging_bytes(const redist_plan_t *plan, int32_t which);
int32_t redist_plan_alignment(const redist_plan_t *plan);                 /* required pointer alignment */
int64_t redist_plan_height(const redist_plan_t *plan);   /* max localsize over the sequence (elements);
                                               the memory bound of Section 4.3 says
                                               height <= max(localsize src, localsize dst)            */
int64_t redist_plan_cost(const redist_plan_t *plan);     /* summed cost of the sequence (elements)    */
int32_t redist_plan_num_steps(const redist_plan_t *plan);    /* collectives in the sequence           */
int32_t redist_plan_num_launches(const redist_plan_t *plan); /* kernels redist_execute launches       */
redist_status redist_plan_step_info(const redist_plan_t *plan, int32_t step, redist_step_info *out);
redist_status redist_plan_launch_info(const redist_plan_t *plan, int32_t launch, redist_launch_info *out);

/*
 * redist_plan_describe -- the typed sequence and the launch descriptors as JSON (prime mesh, every
 * step with the axes acted on, the type and the device map after it, costs, and per launch the copy
 * descriptor the kernel receives).  Writes at most cap bytes including the terminating NUL and
 * returns the length the full text needs (excluding the NUL); call with cap = 0 to size a buffer.
 */
size_t redist_plan_describe(const redist_plan_t *plan, char *buf, size_t cap);

/*
 * redist_base_offsets -- base offset map T[[type]] (figure "Semantics for distributed dimensions
 * and types", part (a)): out_offsets[d*rank + k] is the lowest global index in dimension k of the
 * tile held by virtual device d; out_tile[rank] is the local tile shape.  Host only.
 */
redist_status redist_base_offsets(int32_t n_mesh_axes, const int64_t *mesh_shape, const redist_type *type,
                                  int64_t *out_tile, int64_t *out_offsets);

/*
 * redist_plan_gpu_split -- byte accounting for running the plan with its virtual devices spread over
 * several GPUs (host only; nothing in this library moves data between GPUs).  The paper executes its
 * collectives between real devices (Section 8) and discusses individual device-to-device transfers
 * derived from the base offset maps as the alternative (Section 9); this is that derivation for one
 * launch.  Virtual device d is placed on GPU d / (N / n_gpus): the leading mesh coordinates choose the
 * GPU, so n_gpus must be the product of the leading mesh axis sizes times a divisor of the next one.
 *
 *   launch          index of a kernel launch of the plan (redist_plan_num_launches)
 *   bytes           host; receives n_gpus * n_gpus numbers, row-major: bytes[s * n_gpus + t] = bytes that
 *                   GPU s reads from tiles it holds and writes into tiles that live on GPU t (a replicated
 *                   source tile is read on the receiving GPU when that GPU holds a replica, else from the
 *                   lowest-numbered holder).  The diagonal stays inside a GPU; the sum over the matrix is
 *                   the launch's bytes_written; with n_gpus = 1 it is that single number.
 * Errors: EINVAL (also for an n_gpus that is no prefix of the mesh), ENOMEM.
 */
redist_status redist_plan_gpu_split(const redist_plan_t *plan, int32_t n_gpus, int32_t launch, int64_t *bytes);

const char *redist_status_string(redist_status status);

/* The last CUDA error code (cudaError_t as int) seen by the calling thread inside this library. */
int32_t redist_last_cuda_error(void);

/*
 * redist_bulk_timeouts -- health counter of the bulk-copy kernels (not part of the paper's method).
 * Runs are staged in shared memory by TMA bulk copies whose completion a thread block awaits on an
 * mbarrier with a bounded number of polls ("wait_polls").  A block whose wait runs out stores
 * nothing, counts itself here, keeps polling (sleeping up to 256 ns between polls) for as many polls
 * again so that copies still in flight can land in shared memory it still owns, and returns: a
 * faulty copy engine shows up as a non-zero count and unwritten output instead of a hang.  Returns
 * the count for the current device since the library was loaded (0 in a healthy run), or -1 on a
 * CUDA error.  Synchronizes the device.  A non-zero count means the outputs of the run are invalid.
 * The tuning value "test_extra_tx" exists to test this path: it makes every block announce that
 * many bytes more than its copies deliver, so every copy lands but no wait ever completes.
 */
int64_t redist_bulk_timeouts(void);

/*
 * redist_debug_bounds_report -- checked build only (the library compiled with -DREDIST_BOUNDS, which
 * the tests load in place of the normal one).  There every global access of the kernels is tested
 * against the tiles of the launch and every dynamic shared-memory access against the launch's
 * shared-memory size; a failing access is skipped, not performed.  out[0] = number of failed tests
 * since the last call, out[1..4] = source line, thread block, side (1 read, 2 write, 3 shared memory)
 * and distance from the nearest tile base of the first one.  The call resets the record.
 * Synchronizes the device.  The normal build returns EUNSUPPORTED.
 */
redist_status redist_debug_bounds_report(int64_t out[5]);

#ifdef __cplusplus
}
#endif
#endif /* REDIST_H_ */
