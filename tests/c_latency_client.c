/* Per-update latency of the small configurations (89,578 parameters) driven straight from C, without the
 * Python interpreter between the calls: a plain C99 client of include/softsync_ps.h plus the CUDA runtime
 * for device memory.  Prints microseconds per weight update for
 *   - one update per kernel pass, ordinary launches and programmatic dependent launches,
 *   - PS_OPT_FUSE_T = 16 updates per pass, with c = 1 (lambda = n = 30) and c = 4 (lambda = 4, n = 1).
 * Every pull, push and apply of the protocol is inside the timed loop; gradients are device buffers that
 * exist before it starts.  Usage: c_latency_client [updates]  (default 20000). */
#define _POSIX_C_SOURCE 199309L
#include "softsync_ps.h"

#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>
#include <time.h>

#define N_PARAMS 89578
#define POOL 64

#define CHECK(cond) do { if (!(cond)) { printf("failed: %s (line %d)\n", #cond, __LINE__); return -1.0; } } while (0)

static double now_us(void)
{
    struct timespec t;
    clock_gettime(CLOCK_MONOTONIC, &t);
    return t.tv_sec * 1e6 + t.tv_nsec * 1e-3;
}

/* microseconds per update, or a negative number on failure */
static double run(int lambda, int n, int fuse_t, int overlap, long updates, float *w, float *v, float **grads)
{
    ps_t *ps = NULL;
    int64_t ts = 0;
    const int c = lambda / n;
    long pushes = 0, applied = 0, pending = 0;
    double t0, t1;
    static float w0[N_PARAMS];

    CHECK(ps_create(&ps, N_PARAMS, lambda, n, 0.001f, 0.9f, 5e-4f, PS_MOD_INV_STALENESS) == PS_OK);
    CHECK(ps_bind_state(ps, w, v) == PS_OK);
    CHECK(ps_set_option(ps, PS_OPT_FUSE_T, fuse_t) == PS_OK);
    CHECK(ps_set_option(ps, PS_OPT_OVERLAP_LAUNCH, overlap) == PS_OK);
    CHECK(ps_init_weights(ps, w0, 1) == PS_OK);
    for (int phase = 0; phase < 2; ++phase) {                 /* phase 0 warms up, phase 1 is timed */
        const long want = phase == 0 ? 200 : updates;
        CHECK(ps_synchronize(ps) == PS_OK);
        t0 = now_us();
        applied = 0;
        while (applied < want) {
            const int learner = (int)(pushes % lambda);
            int rc;
            CHECK(ps_pull_weights(ps, NULL, &ts) == PS_OK);
            rc = ps_push_gradient(ps, learner, grads[pushes % POOL], ts);
            CHECK(rc == PS_OK || rc == PS_READY);
            ++pushes;
            pending += rc == PS_READY;
            if (pending >= fuse_t) {
                rc = ps_apply_update(ps);
                CHECK(rc >= 1);
                applied += rc;
                pending -= rc;
            }
        }
        CHECK(ps_synchronize(ps) == PS_OK);
        t1 = now_us();
    }
    CHECK(c >= 1 && ps_destroy(ps) == PS_OK);
    return (t1 - t0) / (double)applied;
}

int main(int argc, char **argv)
{
    const long updates = argc > 1 ? atol(argv[1]) : 20000;
    float *w = NULL, *v = NULL, *grads[POOL];
    double us;
    int ok = 1;

    if (cudaMalloc((void **)&w, N_PARAMS * sizeof(float)) != cudaSuccess) { printf("no device memory\n"); return 1; }
    if (cudaMalloc((void **)&v, N_PARAMS * sizeof(float)) != cudaSuccess) return 1;
    for (int i = 0; i < POOL; ++i) {
        if (cudaMalloc((void **)&grads[i], N_PARAMS * sizeof(float)) != cudaSuccess) return 1;
        if (cudaMemset(grads[i], 0, N_PARAMS * sizeof(float)) != cudaSuccess) return 1;
    }
    us = run(30, 30, 1, 0, updates, w, v, grads);  ok &= us > 0;
    printf("c=1  T=1  ordinary launches              %8.3f us per update\n", us);
    us = run(30, 30, 1, 1, updates, w, v, grads);  ok &= us > 0;
    printf("c=1  T=1  programmatic dependent launches %8.3f us per update\n", us);
    us = run(4, 1, 1, 1, updates, w, v, grads);    ok &= us > 0;
    printf("c=4  T=1  programmatic dependent launches %8.3f us per update\n", us);
    us = run(30, 30, 16, 1, updates, w, v, grads); ok &= us > 0;
    printf("c=1  T=16 programmatic dependent launches %8.3f us per update\n", us);
    us = run(4, 1, 16, 1, updates, w, v, grads);   ok &= us > 0;
    printf("c=4  T=16 programmatic dependent launches %8.3f us per update\n", us);
    for (int i = 0; i < POOL; ++i) cudaFree(grads[i]);
    cudaFree(w); cudaFree(v);
    printf(ok ? "c latency client ok\n" : "c latency client FAILED\n");
    return ok ? 0 : 1;
}
