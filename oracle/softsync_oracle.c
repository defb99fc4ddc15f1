/* TEST INFRASTRUCTURE: reference implementation, not part of the product path.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 * It shares no code with the CUDA library and neither includes the other.
 *
 * A plain, slow, single-threaded model of the paper's parameter server running
 * the n-softsync protocol (Section 2.1, 2.2, 2.4):
 *
 *   - a scalar clock i starts at 0 and goes up by exactly 1 per weight update
 *     (Section 2.1, "Timestamp");
 *   - a learner pulls the weights together with the clock value, and the
 *     gradient it later pushes carries that value j (Section 2.1);
 *   - the staleness of a pushed gradient is tau = i - j >= 0 (Section 2.1);
 *   - the server updates the weights once c = floor(lambda / n) gradients
 *     have arrived from any learners (Section 2.2, Eq. 2);
 *   - each gradient is scaled by alpha0 / tau when tau > 0 (Eq. 3) or by the
 *     constant alpha0 (the control experiment of Section 4.3).
 *
 * Readings where the paper is silent:
 *   - tau = 0 is given the full alpha0: sigma = max(tau, 1).  Eq. 1 (hardsync,
 *     tau = 0) uses the full learning rate.
 *   - an update takes exactly c gradients, first come first grouped.
 *   - tau is taken when the gradient arrives, so all c members of update i
 *     see the same server clock i (the footnote to Eq. 5 counts staleness so).
 *   - inside a group the gradients are summed in ascending (learner, push
 *     index) order, left to right.
 *   - the update runs inside the push that completes the group; a pull that
 *     follows sees the new clock.
 *   - momentum and weight decay: see update_rule.inc.
 *   - exponential penalty (the earlier proposal that Section 1 sets the 1/tau rule against; the
 *     paper gives no formula for it): alpha = alpha0 * rho^tau with a base 0 < rho <= 1, so a fresh
 *     gradient (tau = 0) gets alpha0; the log's sigma field then holds tau itself.
 *   - per-layer multipliers: see update_rule.inc.
 *   - the base rate alpha0 may be changed between calls (the step schedules of
 *     Section 4.3); a gradient is scaled with the alpha0 in force when it arrived,
 *     since Section 2.4 (Eq. 3) fixes the rate per gradient as it comes in.
 *
 * Parity pins: tests/test_oracle_*.py (hand-worked examples under
 * tests/golden/, closed forms, reductions to plain SGD, invariants).
 * Convergence/accuracy behaviour of the method is not modelled here:
 * parity unpinned for it (it needs the paper's datasets).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_C 4096

#define ORACLE_MOD_CONSTANT 0
#define ORACLE_MOD_INV_STALENESS 1
#define ORACLE_MOD_EXP_STALENESS 2

#define ORACLE_GRAD_FP32 0
#define ORACLE_GRAD_BF16 1

/* ---- the update rule in both precisions -------------------------------- */
#define REAL float
#define FN(name) name##_f32
#define ROUND_SCALE(x) ((float)(x))
#include "update_rule.inc"
#undef REAL
#undef FN
#undef ROUND_SCALE

#define REAL double
#define FN(name) name##_f64
#define ROUND_SCALE(x) ((double)(x))
#include "update_rule.inc"
#undef REAL
#undef FN
#undef ROUND_SCALE

/* ---- protocol state ----------------------------------------------------- */
typedef struct {
    int64_t update;      /* clock value i before this update                */
    int64_t push_index;  /* how many pushes this learner had made before    */
    int64_t ts_grad;     /* j: clock value the learner pulled               */
    int64_t tau;         /* i - j                                           */
    int64_t sigma;       /* staleness used in the learning rate (>= 1)      */
    int32_t learner;
    int32_t position;    /* place in the summation order, 0 .. c-1          */
    double scale;        /* s_l = alpha0 / (c sigma_l), in working precision */
    double decay;        /* d = wd * sum_l s_l, in working precision        */
} oracle_log_entry;

typedef struct {
    int32_t learner;
    int64_t push_index, ts_grad, tau, sigma;
    double alpha0;       /* base rate in force at arrival */
    void *grad;          /* N values widened to the working precision */
} pending_t;

typedef struct oracle_ps {
    int64_t N;
    int lambda, n, c, modulation, precision;
    int hardsync;                    /* 1: the hardsync protocol of Section 2.2 (barrier, staleness 0) */
    double alpha0, momentum, wd;     /* exact widenings of the fp32 parameters */
    double rho;                      /* base of the exponential staleness penalty */
    float *lm, *dm;                  /* per-element rate / decay multipliers, NULL = all 1 */
    void *w, *v;
    int64_t ts;
    int64_t *pulled_ts;              /* -1: has not pulled yet */
    int64_t *push_count;
    pending_t *pending;
    int npending;
    oracle_log_entry *log;
    int64_t log_size, log_cap;
} oracle_ps;

static size_t real_size(const oracle_ps *ps) { return ps->precision == 32 ? sizeof(float) : sizeof(double); }

oracle_ps *oracle_ps_create(int64_t N, int lambda, int n, float alpha0, float momentum,
                            float weight_decay, int modulation, int precision)
{
    if (N < 0 || lambda < 1 || n < 1 || n > lambda) return NULL;
    if (precision != 32 && precision != 64) return NULL;
    if (modulation < ORACLE_MOD_CONSTANT || modulation > ORACLE_MOD_EXP_STALENESS) return NULL;
    if (lambda / n > ORACLE_MAX_C) return NULL;
    oracle_ps *ps = calloc(1, sizeof *ps);
    ps->N = N; ps->lambda = lambda; ps->n = n;
    ps->c = lambda / n;                                   /* Eq. 2: c = floor(lambda/n) */
    ps->alpha0 = alpha0; ps->momentum = momentum; ps->wd = weight_decay;
    ps->modulation = modulation; ps->precision = precision;
    ps->rho = 0.5;
    ps->w = calloc((size_t)(N ? N : 1), real_size(ps));
    ps->v = calloc((size_t)(N ? N : 1), real_size(ps));
    ps->pulled_ts = malloc(sizeof(int64_t) * lambda);
    ps->push_count = calloc(lambda, sizeof(int64_t));
    for (int l = 0; l < lambda; ++l) ps->pulled_ts[l] = -1;
    ps->pending = calloc(ps->c, sizeof(pending_t));
    for (int l = 0; l < ps->c; ++l) ps->pending[l].grad = malloc((size_t)(N ? N : 1) * real_size(ps));
    return ps;
}

void oracle_ps_destroy(oracle_ps *ps)
{
    if (!ps) return;
    for (int l = 0; l < ps->c; ++l) free(ps->pending[l].grad);
    free(ps->pending); free(ps->w); free(ps->v);
    free(ps->pulled_ts); free(ps->push_count); free(ps->log); free(ps->lm); free(ps->dm); free(ps);
}

/* theta_0 = w0, velocity 0, clock 0 (Section 2.1). */
void oracle_ps_set_weights(oracle_ps *ps, const float *w0)
{
    for (int64_t k = 0; k < ps->N; ++k) {
        if (ps->precision == 32) { ((float *)ps->w)[k] = w0[k]; ((float *)ps->v)[k] = 0.0f; }
        else { ((double *)ps->w)[k] = (double)w0[k]; ((double *)ps->v)[k] = 0.0; }
    }
    ps->ts = 0;
}

/* Hardsync protocol (Section 2.2, Eq. 1): the server waits for one gradient from every learner, all
 * computed on the current weights, averages them and updates; needs n = 1 so that c = lambda.
 * Returns 0, or -1 if n != 1 or gradients are pending. */
int oracle_ps_set_hardsync(oracle_ps *ps, int on)
{
    if (on && ps->n != 1) return -1;
    if (ps->npending) return -1;
    ps->hardsync = on ? 1 : 0;
    return 0;
}

/* Base rho of the exponential staleness penalty alpha0 * rho^tau (0 < rho <= 1); used only when the
 * server was created with ORACLE_MOD_EXP_STALENESS.  Returns 0, or -1 for a base outside (0, 1]. */
int oracle_ps_set_penalty_base(oracle_ps *ps, float rho)
{
    if (!(rho > 0.0f) || rho > 1.0f) return -1;
    ps->rho = rho;
    return 0;
}

/* Per-layer multipliers: layer q covers elements [bounds[q], bounds[q+1]) (bounds[0] = 0,
 * bounds[nseg] = N, ascending) and scales the learning rate by lr_mult[q] and the weight decay by
 * wd_mult[q].  nseg = 0 removes them.  Returns 0, or -1 if the bounds do not tile [0, N). */
int oracle_ps_set_layer_multipliers(oracle_ps *ps, int nseg, const int64_t *bounds,
                                    const float *lr_mult, const float *wd_mult)
{
    if (nseg < 0) return -1;
    if (nseg == 0) { free(ps->lm); free(ps->dm); ps->lm = ps->dm = NULL; return 0; }
    if (bounds[0] != 0 || bounds[nseg] != ps->N) return -1;
    for (int q = 0; q < nseg; ++q) if (bounds[q] > bounds[q + 1]) return -1;
    free(ps->lm); free(ps->dm);
    ps->lm = malloc(sizeof(float) * (size_t)(ps->N ? ps->N : 1));
    ps->dm = malloc(sizeof(float) * (size_t)(ps->N ? ps->N : 1));
    for (int q = 0; q < nseg; ++q)
        for (int64_t k = bounds[q]; k < bounds[q + 1]; ++k) { ps->lm[k] = lr_mult[q]; ps->dm[k] = wd_mult[q]; }
    return 0;
}

/* Learning-rate schedule: the base rate for gradients that arrive from now on (Section 4.3). */
void oracle_ps_set_alpha0(oracle_ps *ps, float alpha0) { ps->alpha0 = alpha0; }

int64_t oracle_ps_timestamp(const oracle_ps *ps) { return ps->ts; }
int oracle_ps_group_size(const oracle_ps *ps) { return ps->c; }

/* pullWeights: the learner receives theta_i and the clock value i. */
int64_t oracle_ps_pull(oracle_ps *ps, int learner)
{
    if (learner < 0 || learner >= ps->lambda) return -1;
    ps->pulled_ts[learner] = ps->ts;
    return ps->ts;
}

static float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;       /* bf16 is the upper half of an fp32 */
    float f; memcpy(&f, &u, sizeof f); return f;
}

static void log_append(oracle_ps *ps, const oracle_log_entry *e)
{
    if (ps->log_size == ps->log_cap) {
        ps->log_cap = ps->log_cap ? 2 * ps->log_cap : 1024;
        ps->log = realloc(ps->log, sizeof(oracle_log_entry) * (size_t)ps->log_cap);
    }
    ps->log[ps->log_size++] = *e;
}

/* (learner, push index) ascending: the fixed summation order of a group. */
static int before(const pending_t *a, const pending_t *b)
{
    if (a->learner != b->learner) return a->learner < b->learner;
    return a->push_index < b->push_index;
}

static void apply_pending(oracle_ps *ps)
{
    const int c = ps->c;
    int order[ORACLE_MAX_C];
    for (int l = 0; l < c; ++l) order[l] = l;
    for (int a = 1; a < c; ++a) {                       /* insertion sort */
        int x = order[a], b = a - 1;
        while (b >= 0 && before(&ps->pending[x], &ps->pending[order[b]])) { order[b + 1] = order[b]; --b; }
        order[b + 1] = x;
    }
    const void *grads[ORACLE_MAX_C];
    int64_t sigma[ORACLE_MAX_C], tau[ORACLE_MAX_C];
    double scale[ORACLE_MAX_C], alpha0[ORACLE_MAX_C];
    for (int l = 0; l < c; ++l) {
        grads[l] = ps->pending[order[l]].grad; sigma[l] = ps->pending[order[l]].sigma;
        tau[l] = ps->pending[order[l]].tau;
        alpha0[l] = ps->pending[order[l]].alpha0;
    }
    const int exp_penalty = ps->modulation == ORACLE_MOD_EXP_STALENESS;

    double d;
    if (ps->precision == 32)
        d = apply_group_f32(ps->w, ps->v, ps->N, c, (const float *const *)grads, sigma, tau,
                            alpha0, exp_penalty, ps->rho, ps->momentum, ps->wd, ps->lm, ps->dm, scale);
    else
        d = apply_group_f64(ps->w, ps->v, ps->N, c, (const double *const *)grads, sigma, tau,
                            alpha0, exp_penalty, ps->rho, ps->momentum, ps->wd, ps->lm, ps->dm, scale);

    for (int l = 0; l < c; ++l) {
        const pending_t *p = &ps->pending[order[l]];
        oracle_log_entry e = { ps->ts, p->push_index, p->ts_grad, p->tau, p->sigma,
                               p->learner, l, scale[l], d };
        log_append(ps, &e);
    }
    ps->ts += 1;                                         /* each update advances the clock by 1 */
    ps->npending = 0;
}

/* pushGradient + sumGradients (+ applyUpdate when the group is complete), with the gradient's
 * timestamp j given by the caller: "a learner pushes gradient with timestamp j to the parameter
 * server of timestamp i, where i >= j" (Section 2.1).
 * Returns 1 if this push triggered a weight update, 0 if not, < 0 on misuse. */
int oracle_ps_push_with_timestamp(oracle_ps *ps, int learner, const void *grad, int grad_dtype, int64_t j)
{
    if (learner < 0 || learner >= ps->lambda) return -1;
    if (j < 0) return -2;
    const int64_t tau = ps->ts - j;                      /* staleness, Section 2.1 */
    if (tau < 0) return -3;
    if (ps->hardsync) {
        if (tau != 0) return -3;                         /* "ensures that the gradient staleness is 0" */
        for (int q = 0; q < ps->npending; ++q)           /* one contribution per learner and round */
            if (ps->pending[q].learner == learner) return -4;
    }
    int64_t sigma = 1;
    if (ps->modulation == ORACLE_MOD_INV_STALENESS)
        sigma = tau > 0 ? tau : 1;                       /* Eq. 3, and alpha0 itself at tau = 0 */
    if (ps->modulation == ORACLE_MOD_EXP_STALENESS)
        sigma = tau;                                     /* the penalty's exponent */

    pending_t *p = &ps->pending[ps->npending++];
    p->learner = learner; p->push_index = ps->push_count[learner]++;
    p->ts_grad = j; p->tau = tau; p->sigma = sigma; p->alpha0 = ps->alpha0;
    for (int64_t k = 0; k < ps->N; ++k) {
        const float g = grad_dtype == ORACLE_GRAD_BF16 ? bf16_to_f32(((const uint16_t *)grad)[k])
                                                       : ((const float *)grad)[k];
        if (ps->precision == 32) ((float *)p->grad)[k] = g; else ((double *)p->grad)[k] = (double)g;
    }
    if (ps->npending == ps->c) { apply_pending(ps); return 1; }
    return 0;
}

/* The usual case: the gradient carries the timestamp of the learner's latest pull (Section 2.1). */
int oracle_ps_push(oracle_ps *ps, int learner, const void *grad, int grad_dtype)
{
    if (learner < 0 || learner >= ps->lambda) return -1;
    return oracle_ps_push_with_timestamp(ps, learner, grad, grad_dtype, ps->pulled_ts[learner]);
}

void oracle_ps_get_state(const oracle_ps *ps, double *w_out, double *v_out)
{
    for (int64_t k = 0; k < ps->N; ++k) {
        w_out[k] = ps->precision == 32 ? (double)((float *)ps->w)[k] : ((double *)ps->w)[k];
        v_out[k] = ps->precision == 32 ? (double)((float *)ps->v)[k] : ((double *)ps->v)[k];
    }
}

/* fp32 -> bf16, round to nearest, ties to even: bf16 keeps the upper 16 bits of the fp32 pattern, so add
 * half of the dropped part (0x7FFF plus the lowest kept bit) and truncate.  NaN maps to 0x7FFF. */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u; memcpy(&u, &f, sizeof u);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FFF;
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* The weights as a bf16 learner would pull them (an extension: the paper's weights are 4-byte).
 * Defined for the fp32 server state only. */
int oracle_ps_get_weights_bf16(const oracle_ps *ps, uint16_t *out)
{
    if (ps->precision != 32) return -1;
    for (int64_t k = 0; k < ps->N; ++k) out[k] = f32_to_bf16_rne(((const float *)ps->w)[k]);
    return 0;
}

/* The same rounding on caller-supplied values (so that it can be pinned on its own). */
void oracle_round_to_bf16(const float *in, uint16_t *out, int64_t n)
{
    for (int64_t k = 0; k < n; ++k) out[k] = f32_to_bf16_rne(in[k]);
}

int64_t oracle_ps_log_size(const oracle_ps *ps) { return ps->log_size; }

void oracle_ps_get_log(const oracle_ps *ps, oracle_log_entry *out)
{
    memcpy(out, ps->log, sizeof(oracle_log_entry) * (size_t)ps->log_size);
}
