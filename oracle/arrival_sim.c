/* TEST INFRASTRUCTURE: reference implementation, not part of the product path.
 *
 * The reference's own seeded learner-arrival simulator.  Every learner runs
 * the loop of Section 2.1 (pullWeights, calcGradient, pushGradient) against a
 * server that handles one blocking call at a time (Section 2.3): a learner
 * pushes, and pulls again before anybody else is served.  The simulator draws
 * how long each calcGradient takes and emits the resulting order of events;
 * together with oracle_ps_* (softsync_oracle.c) that yields timestamps and
 * staleness.
 *
 * Models:
 *   0 rounds     each round is one Fisher-Yates permutation of the learners
 *   1 exp        compute time ~ Exp(1) i.i.d.
 *   2 uniform    compute time ~ U[0.9, 1.1] i.i.d.: the homogeneous, similar-
 *                speed learners of Section 2.3
 *   3 lognormal  persistent per-learner speed exp(0.5 z), z ~ N(0,1), times a
 *                per-iteration jitter U[0.95, 1.05]
 *
 * Pins (tests/test_oracle_arrivals.py): with lambda = 30 homogeneous learners
 * the paper measures tau in {0,1,2} for 1-softsync and a mean staleness close
 * to n with nothing beyond 2n for n = 15, 30 (Section 2.4, Fig. 1); with
 * Exp(1) times and c = 1 the staleness is geometric with mean lambda - 1; the
 * log-normal model's per-learner mean duration has log-standard-deviation 0.5 and
 * its durations spread +-5 % around that mean (checked on the simulated times).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#define EV_PULL 0
#define EV_PUSH 1

/* SplitMix64 (Steele, Lea, Flood 2014) as a sequential generator. */
static uint64_t next_u64(uint64_t *state)
{
    uint64_t z = (*state += 0x9E3779B97F4A7C15ULL);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* uniform in (0, 1): 53 random bits, never 0 */
static double next_unit(uint64_t *state)
{
    return ((double)(next_u64(state) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

static double next_normal(uint64_t *state)
{
    const double u1 = next_unit(state), u2 = next_unit(state);
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);   /* Box-Muller */
}

static double draw_duration(int model, double speed, uint64_t *state)
{
    switch (model) {
    case 1: return -log(next_unit(state));
    case 2: return 0.9 + 0.2 * next_unit(state);
    default: return speed * (0.95 + 0.1 * next_unit(state));
    }
}

/* Writes events to kind[]/learner[] (capacity cap) and returns their number,
 * or -1 if cap is too small / arguments are invalid.  The trace opens with a
 * pull by every learner and ends with the pull that follows push number
 * num_pushes. */
static int64_t simulate(int model, int lambda, int64_t num_pushes, uint64_t seed,
                        int32_t *kind, int32_t *learner, double *when, int64_t cap)
{
    if (lambda < 1 || num_pushes < 0 || model < 0 || model > 3) return -1;
    if (cap < lambda + 2 * num_pushes) return -1;
    uint64_t state = seed;
    int64_t ne = 0, pushes = 0;
    for (int l = 0; l < lambda; ++l) { kind[ne] = EV_PULL; learner[ne] = l; if (when) when[ne] = 0.0; ++ne; }

    if (model == 0) {
        int *perm = malloc(sizeof(int) * lambda);
        while (pushes < num_pushes) {
            for (int l = 0; l < lambda; ++l) perm[l] = l;
            for (int a = lambda - 1; a > 0; --a) {        /* Fisher-Yates */
                int b = (int)(next_u64(&state) % (uint64_t)(a + 1));
                int t = perm[a]; perm[a] = perm[b]; perm[b] = t;
            }
            for (int a = 0; a < lambda && pushes < num_pushes; ++a, ++pushes) {
                kind[ne] = EV_PUSH; learner[ne] = perm[a]; if (when) when[ne] = (double)pushes; ++ne;
                kind[ne] = EV_PULL; learner[ne] = perm[a]; if (when) when[ne] = (double)pushes; ++ne;
            }
        }
        free(perm);
        return ne;
    }

    double *done = malloc(sizeof(double) * lambda);       /* when each learner's gradient is ready */
    double *speed = malloc(sizeof(double) * lambda);
    for (int l = 0; l < lambda; ++l) speed[l] = model == 3 ? exp(0.5 * next_normal(&state)) : 1.0;
    for (int l = 0; l < lambda; ++l) done[l] = draw_duration(model, speed[l], &state);
    for (; pushes < num_pushes; ++pushes) {
        int first = 0;                                    /* earliest finisher, lowest id on ties */
        for (int l = 1; l < lambda; ++l) if (done[l] < done[first]) first = l;
        kind[ne] = EV_PUSH; learner[ne] = first; if (when) when[ne] = done[first]; ++ne;
        kind[ne] = EV_PULL; learner[ne] = first; if (when) when[ne] = done[first]; ++ne;
        done[first] += draw_duration(model, speed[first], &state);
    }
    free(done); free(speed);
    return ne;
}

int64_t oracle_simulate_arrivals(int model, int lambda, int64_t num_pushes, uint64_t seed,
                                 int32_t *kind, int32_t *learner, int64_t cap)
{
    return simulate(model, lambda, num_pushes, seed, kind, learner, NULL, cap);
}

/* The same trace together with the simulated time of every event (for checking the duration laws). */
int64_t oracle_simulate_arrivals_timed(int model, int lambda, int64_t num_pushes, uint64_t seed,
                                       int32_t *kind, int32_t *learner, double *when, int64_t cap)
{
    return simulate(model, lambda, num_pushes, seed, kind, learner, when, cap);
}
