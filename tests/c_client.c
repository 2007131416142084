/*
 * A client of the library written in plain C99: what a caller without Python sees of the boundary.
 *
 *   c_client <in.bin> <out.bin>
 *
 * Problem (fixed): the smallest benchmark configuration, uint32 [256, 256] on a 2 x 2 mesh,
 * {d0: x, d1: y} -> {d0: y, d1: x}, forward and back.
 *   in.bin    the four source tiles, one after the other (4 * 65536 bytes)
 *   out.bin   receives the four tiles of the target type after the forward redistribution
 * The program also runs the way back and checks that the source tiles return bit for bit, then times
 *   - the host side of redist_bound_execute and of redist_execute (calls queued in batches of 500,
 *     the wait for the GPU between batches is not timed), and
 *   - forward + back on the device with CUDA events,
 * and prints one line of JSON.  Exit status 0 only if every call succeeded and the round trip is exact.
 */
#define _POSIX_C_SOURCE 199309L
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include "redist.h"

enum { N = 4, TILE_BYTES = 128 * 128 * 4, BATCH = 500, BATCHES = 20, PAIRS = 2000 };

#define CHECK_RD(call)                                                                          \
    do {                                                                                        \
        redist_status rc_ = (call);                                                             \
        if (rc_ != REDIST_OK) {                                                                 \
            fprintf(stderr, "%s: %s\n", #call, redist_status_string(rc_));                      \
            return 1;                                                                           \
        }                                                                                       \
    } while (0)

#define CHECK_CU(call)                                                                          \
    do {                                                                                        \
        cudaError_t e_ = (call);                                                                \
        if (e_ != cudaSuccess) {                                                                \
            fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));                         \
            return 1;                                                                           \
        }                                                                                       \
    } while (0)

static double now_s(void)
{
    struct timespec t;
    clock_gettime(CLOCK_MONOTONIC, &t);
    return (double)t.tv_sec + 1e-9 * (double)t.tv_nsec;
}

int main(int argc, char **argv)
{
    if (argc != 3) {
        fprintf(stderr, "usage: %s in.bin out.bin\n", argv[0]);
        return 2;
    }
    /* the two types: dimension k lists its mesh axes minor to major */
    const int64_t mesh[2] = {2, 2};
    const int64_t shape[2] = {256, 256};
    const int32_t off[3] = {0, 1, 2};
    const int32_t axes_a[2] = {0, 1}, axes_b[2] = {1, 0};
    const redist_type type_a = {2, shape, off, axes_a}, type_b = {2, shape, off, axes_b};

    redist_plan_t *fwd = NULL, *back = NULL;
    CHECK_RD(redist_plan(2, mesh, &type_a, &type_b, 4, REDIST_FUSE_ADJACENT, &fwd));
    CHECK_RD(redist_plan(2, mesh, &type_b, &type_a, 4, REDIST_FUSE_ADJACENT, &back));
    if (redist_plan_num_devices(fwd) != N || redist_plan_local_elems(fwd, 0) * 4 != TILE_BYTES ||
        redist_plan_local_elems(fwd, 1) * 4 != TILE_BYTES || redist_plan_scratch_bytes(fwd) != 0 ||
        redist_plan_scratch_bytes(back) != 0) {
        fprintf(stderr, "unexpected plan\n");
        return 1;
    }

    static unsigned char host_in[N * TILE_BYTES], host_out[N * TILE_BYTES];
    FILE *f = fopen(argv[1], "rb");
    if (!f || fread(host_in, 1, sizeof host_in, f) != sizeof host_in) {
        fprintf(stderr, "cannot read %s\n", argv[1]);
        return 1;
    }
    fclose(f);

    void *a[N], *b[N], *a2[N];
    const void *a_src[N], *b_src[N];
    for (int d = 0; d < N; ++d) {
        CHECK_CU(cudaMalloc(&a[d], TILE_BYTES));
        CHECK_CU(cudaMalloc(&b[d], TILE_BYTES));
        CHECK_CU(cudaMalloc(&a2[d], TILE_BYTES));
        CHECK_CU(cudaMemcpy(a[d], host_in + (size_t)d * TILE_BYTES, TILE_BYTES, cudaMemcpyHostToDevice));
        CHECK_CU(cudaMemset(b[d], 0xEE, TILE_BYTES));
        CHECK_CU(cudaMemset(a2[d], 0xEE, TILE_BYTES));
        a_src[d] = a[d];
        b_src[d] = b[d];
    }
    cudaStream_t stream;
    CHECK_CU(cudaStreamCreate(&stream));

    /* forward, written out for the caller to compare; back, compared here */
    CHECK_RD(redist_execute(fwd, a_src, b, NULL, 0, stream));
    CHECK_RD(redist_execute(back, b_src, a2, NULL, 0, stream));
    CHECK_CU(cudaStreamSynchronize(stream));
    for (int d = 0; d < N; ++d)
        CHECK_CU(cudaMemcpy(host_out + (size_t)d * TILE_BYTES, b[d], TILE_BYTES, cudaMemcpyDeviceToHost));
    f = fopen(argv[2], "wb");
    if (!f || fwrite(host_out, 1, sizeof host_out, f) != sizeof host_out) {
        fprintf(stderr, "cannot write %s\n", argv[2]);
        return 1;
    }
    fclose(f);
    for (int d = 0; d < N; ++d) {
        CHECK_CU(cudaMemcpy(host_out, a2[d], TILE_BYTES, cudaMemcpyDeviceToHost));
        if (memcmp(host_out, host_in + (size_t)d * TILE_BYTES, TILE_BYTES) != 0) {
            fprintf(stderr, "round trip differs on tile %d\n", d);
            return 1;
        }
    }

    /* bound forms: checks and parameter blocks once */
    redist_bound_t *bf = NULL, *bb = NULL;
    CHECK_RD(redist_bind(fwd, a_src, b, NULL, 0, &bf));
    CHECK_RD(redist_bind(back, b_src, a2, NULL, 0, &bb));
    for (int i = 0; i < 50; ++i) {
        CHECK_RD(redist_bound_execute(bf, stream));
        CHECK_RD(redist_bound_execute(bb, stream));
    }
    CHECK_CU(cudaStreamSynchronize(stream));

    double host_bound = 0.0, host_plain = 0.0;
    for (int k = 0; k < BATCHES; ++k) {
        double t0 = now_s();
        for (int i = 0; i < BATCH / 2; ++i) {
            if (redist_bound_execute(bf, stream) != REDIST_OK || redist_bound_execute(bb, stream) != REDIST_OK) return 1;
        }
        host_bound += now_s() - t0;
        CHECK_CU(cudaStreamSynchronize(stream));
        t0 = now_s();
        for (int i = 0; i < BATCH / 2; ++i) {
            if (redist_execute(fwd, a_src, b, NULL, 0, stream) != REDIST_OK ||
                redist_execute(back, b_src, a2, NULL, 0, stream) != REDIST_OK)
                return 1;
        }
        host_plain += now_s() - t0;
        CHECK_CU(cudaStreamSynchronize(stream));
    }

    cudaEvent_t e0, e1;
    CHECK_CU(cudaEventCreate(&e0));
    CHECK_CU(cudaEventCreate(&e1));
    float ms_best = 1e30f;
    for (int rep = 0; rep < 5; ++rep) {
        CHECK_CU(cudaEventRecord(e0, stream));
        for (int i = 0; i < PAIRS; ++i) {
            if (redist_bound_execute(bf, stream) != REDIST_OK || redist_bound_execute(bb, stream) != REDIST_OK) return 1;
        }
        CHECK_CU(cudaEventRecord(e1, stream));
        CHECK_CU(cudaEventSynchronize(e1));
        float ms = 0.f;
        CHECK_CU(cudaEventElapsedTime(&ms, e0, e1));
        if (ms < ms_best) ms_best = ms;
    }
    /* the timed loops must have left the data as the first round trip did */
    for (int d = 0; d < N; ++d) {
        CHECK_CU(cudaMemcpy(host_out, a2[d], TILE_BYTES, cudaMemcpyDeviceToHost));
        if (memcmp(host_out, host_in + (size_t)d * TILE_BYTES, TILE_BYTES) != 0) {
            fprintf(stderr, "round trip differs on tile %d after the timed loops\n", d);
            return 1;
        }
    }
    printf("{\"calls\": %d, \"host_us_per_bound_call\": %.3f, \"host_us_per_execute_call\": %.3f, "
           "\"device_us_forward_and_back\": %.3f, \"bulk_timeouts\": %ld}\n",
           BATCH * BATCHES, 1e6 * host_bound / (BATCH * BATCHES), 1e6 * host_plain / (BATCH * BATCHES),
           1e3 * ms_best / PAIRS, (long)redist_bulk_timeouts());

    redist_bound_destroy(bf);
    redist_bound_destroy(bb);
    redist_plan_destroy(fwd);
    redist_plan_destroy(back);
    for (int d = 0; d < N; ++d) {
        cudaFree(a[d]);
        cudaFree(b[d]);
        cudaFree(a2[d]);
    }
    cudaStreamDestroy(stream);
    return 0;
}
