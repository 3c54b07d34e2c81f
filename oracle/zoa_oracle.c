/*
 * CPU oracle for the 0/1 Adam optimizer step (arXiv 2202.06009).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * nothing in the product may call it: only the test-suite, the smoke check
 * and the benchmark's CPU-baseline leg do.
 *
 * What it follows, in the paper's order and notation:
 *   Algorithm 1 (proposed 0/1 Adam)            -> zo_alg1_half_step, zo_alg1_sync,
 *                                                 zo_alg1_variance, zo_alg1_step
 *   Algorithm 2 (frozen-variance 1-bit framework,
 *                1-bit Adam as a special case)  -> zo_alg2_step
 *   Algorithm 3 (error-feedback 1bit-AllReduce) -> zo_onebit_allreduce
 *   Algorithm 4 (AllReduce, plain mean)         -> zo_allreduce
 *   Eq. 3       (1-bit compressor C[a])         -> zo_compress
 *
 * The file is compiled twice: once with ZO_REAL=float (suffix _f32) and once
 * with ZO_REAL=double (suffix _f64).  In the float build every elementwise
 * operation is ONE IEEE-754 binary32 round-to-nearest operation (build with
 * -ffp-contract=off so that no multiply-add is fused, and without
 * -ffast-math so that subnormals are kept); the double build is the same text
 * with real = double and is used for the algebraic pins.  In both builds the
 * three reductions of the method (the l1 norm of a chunk, the mean over
 * workers of the compressed buffers, the mean over workers of the gradients)
 * accumulate in double, in index / worker order, and are rounded to `real`
 * once at the end.
 *
 * Readings taken where the paper is silent, ambiguous or misprinted:
 *  R1  The model and buffer updates of Algorithm 1 print m_t, the momentum before
 *      the momentum update.  Read literally with a sync at every step, the
 *      momentum approximation of the sync branch overwrites m_{t+1} with the
 *      mean of m_t, so the gradient never enters m and the model never moves.
 *      The derivation in Section 4 (u_t = sum_k gamma_k m_k with m_k the
 *      momentum of step k) and the non-sync branch m_{t+1} = m_{t+1/2} need
 *      m_{t+1/2}.  We use m_{t+1/2}; `literal_momentum` = 1 selects the printed
 *      form so that a test can show it is degenerate.
 *  R2  The divisor of the momentum approximation, sum_{h=t'}^{t} gamma_h, is taken as the sum of
 *      the gamma_h that were actually accumulated into u since u was last
 *      reset (the inclusive printed range would count gamma_{t'} twice).
 *  R3  x_{t'} in the model sync is the model produced by the sync at step t' (x_0
 *      before the first sync).
 *  R4  The server step of Algorithm 3 prints \hat z_{t+1} inside C[.] and
 *      \hat z_t in the error update; both are the buffers just received.
 *  R5  C[.] is applied per chunk of `chunk` consecutive coordinates of the flat
 *      vector, the last chunk dividing by its true length.  chunk >= d gives
 *      Eq. 3 verbatim.
 *  R6  sign(a) is carried by one bit: bit = (a >= 0), so +0 and -0 both map to
 *      +scale and NaN maps to -scale.
 *  R7  Wire format: coordinate j is bit (j mod 32), least significant first,
 *      of 32-bit word floor(j/32); unused bits of the last word are 0; one
 *      scale per chunk.
 *  R8  The model sync uses v_t; the variance update assigns v_{t+1} afterwards.
 *  R9  Algorithm 2 also prints m_t in its model update.  It is introduced as the
 *      special case of Algorithm 1 without local steps, so it takes the same
 *      convention as R1: the momentum just computed.  (With the identity
 *      compressor both algorithms are then the same Adam; `literal_momentum`
 *      selects the printed, one-step-delayed form here too.)  Its model update
 *      reads v_t, so the variance of a T_v step is assigned after it.
 *
 * Pins (tests/test_oracle_pins.py, none of which re-types these formulas):
 *  zo_compress          hand-worked fixtures; z = zhat + err; l1 preserved;
 *                       closed-form error energy |z|_2^2 - |z|_1^2/len; the
 *                       scale minimises the l2 error by brute-force scan;
 *                       Gaussian error ratio 1 - 2/pi; numpy.packbits layout.
 *  zo_onebit_allreduce  hand-worked two-worker fixture; telescoping identity
 *                       of the error feedback (no mass is lost, only delayed);
 *                       invariance under permutation of the workers.
 *  zo_allreduce         numpy mean.
 *  zo_alg1_*            identity compressor with T_u = T_v = all steps equals
 *                       the closed (unrolled) form of Adam's recurrences;
 *                       frozen v equals damped momentum SGD (torch.optim.SGD);
 *                       x = x_{t'} - u / sqrt(v + eps) between syncs;
 *                       hand-worked power-of-two fixture of one sync step;
 *                       sign and scale symmetries; a noisy quadratic is minimised.
 *  zo_alg2_step        identity compressor equals the closed form of Adam and
 *                       equals zo_alg1_step with T_u = all steps; T_v = the first
 *                       T0 steps is Adam for T0 steps and then keeps v; hand-worked
 *                       compressed step; the received gradients telescope.
 *  The paper prints no worked numbers, so the values of a long trajectory are
 *  fixed only by these pins together.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#ifndef ZO_REAL
#error "compile with -DZO_REAL=float -DZO_SUFFIX=_f32 or -DZO_REAL=double -DZO_SUFFIX=_f64"
#endif

typedef ZO_REAL real;

#define ZO_CAT2(a, b) a##b
#define ZO_CAT(a, b) ZO_CAT2(a, b)
#define ZO(name) ZO_CAT(name, ZO_SUFFIX)

enum { ZO_COMPRESSOR_ONEBIT = 0, ZO_COMPRESSOR_IDENTITY = 1 };

/* square root in the working precision (correctly rounded in both) */
static real ZO(zo_sqrt)(real a) { return sizeof(real) == sizeof(float) ? (real)sqrtf((float)a) : (real)sqrt((double)a); }

/* All arrays are owned by the caller.  Per-worker arrays are [n][d] row-major
 * (n = number of workers, d = model dimension, the paper's letters). */
typedef struct {
    int64_t d;                /* model dimension */
    int32_t n;                /* number of workers */
    int64_t chunk;            /* coordinates sharing one scale (R5) */
    real beta1, beta2, eps;
    int32_t compressor;       /* ZO_COMPRESSOR_* */
    int32_t literal_momentum; /* R1: 1 = use m_t in the model and buffer updates, as printed */
    real *x;                  /* [n][d] local models x^(i) */
    real *m;                  /* [n][d] momentum m^(i) */
    real *u;                  /* [n][d] auxiliary buffer u^(i) */
    real *delta;              /* [n][d] worker compression error delta^(i) */
    real *v;                  /* [d]    variance */
    real *delta_bar;          /* [d]    server compression error */
    real *x_sync;             /* [d]    x_{t'} (R3) */
    real *z_hat;              /* [n][d] scratch: compressed worker buffers */
    real *u_bar;              /* [d]    scratch: output of the 1-bit AllReduce */
    uint32_t *words_worker;   /* [n][ceil(d/32)] sign bits sent by the workers (R7) */
    real *scales_worker;      /* [n][ceil(d/chunk)] */
    uint32_t *words_server;   /* [ceil(d/32)] sign bits sent by the server */
    real *scales_server;      /* [ceil(d/chunk)] */
    double gamma_sum;         /* sum of gamma_h accumulated into u (R2) */
    int64_t t_sync;           /* t' */
} ZO(zo_state);

/* Eq. 3, per chunk (R5): a_hat = (|a_c|_1 / len_c) * sign(a), and the wire
 * form of it.  `words` / `scales` may be NULL. */
void ZO(zo_compress)(const real *a, int64_t d, int64_t chunk, real *a_hat,
                     uint32_t *words, real *scales)
{
    if (words)
        for (int64_t w = 0; w < (d + 31) / 32; ++w) words[w] = 0u;
    for (int64_t c0 = 0, c = 0; c0 < d; c0 += chunk, ++c) {
        int64_t c1 = c0 + chunk < d ? c0 + chunk : d;
        double l1 = 0.0;
        for (int64_t j = c0; j < c1; ++j) l1 += fabs((double)a[j]);
        real scale = (real)(l1 / (double)(c1 - c0));
        for (int64_t j = c0; j < c1; ++j) {
            int bit = a[j] >= (real)0; /* R6 */
            a_hat[j] = bit ? scale : -scale;
            if (words && bit) words[j / 32] |= 1u << (j % 32);
        }
        if (scales) scales[c] = scale;
    }
}

static void ZO(zo_identity)(const real *a, int64_t d, real *a_hat)
{
    for (int64_t j = 0; j < d; ++j) a_hat[j] = a[j];
}

/* Algorithm 3.  z is [n][d]; on return st->u_bar holds \bar z, st->delta and
 * st->delta_bar hold the new errors and the wire buffers hold what was sent. */
void ZO(zo_onebit_allreduce)(ZO(zo_state) *st, const real *z)
{
    const int64_t d = st->d;
    const int64_t n_words = (d + 31) / 32;
    const int64_t n_chunks = (d + st->chunk - 1) / st->chunk;
    /* (on the i-th node) compress z + delta, keep what compression lost */
    for (int i = 0; i < st->n; ++i) {
        real *delta = st->delta + (size_t)i * d;
        real *z_hat = st->z_hat + (size_t)i * d;
        for (int64_t j = 0; j < d; ++j) delta[j] = z[(size_t)i * d + j] + delta[j];
        if (st->compressor == ZO_COMPRESSOR_IDENTITY)
            ZO(zo_identity)(delta, d, z_hat);
        else
            ZO(zo_compress)(delta, d, st->chunk, z_hat,
                            st->words_worker ? st->words_worker + (size_t)i * n_words : NULL,
                            st->scales_worker ? st->scales_worker + (size_t)i * n_chunks : NULL);
        for (int64_t j = 0; j < d; ++j) delta[j] = delta[j] - z_hat[j];
    }
    /* (on the server) average, add the server error, compress again (R4) */
    for (int64_t j = 0; j < d; ++j) {
        double sum = 0.0;
        for (int i = 0; i < st->n; ++i) sum += (double)st->z_hat[(size_t)i * d + j];
        st->delta_bar[j] = (real)(sum / (double)st->n + (double)st->delta_bar[j]);
    }
    if (st->compressor == ZO_COMPRESSOR_IDENTITY)
        ZO(zo_identity)(st->delta_bar, d, st->u_bar);
    else
        ZO(zo_compress)(st->delta_bar, d, st->chunk, st->u_bar, st->words_server,
                        st->scales_server);
    for (int64_t j = 0; j < d; ++j) st->delta_bar[j] = st->delta_bar[j] - st->u_bar[j];
}

/* Algorithm 4: g_bar = (1/n) sum_i g^(i). */
void ZO(zo_allreduce)(const real *g, int32_t n, int64_t d, real *g_bar)
{
    for (int64_t j = 0; j < d; ++j) {
        double sum = 0.0;
        for (int i = 0; i < n; ++i) sum += (double)g[(size_t)i * d + j];
        g_bar[j] = (real)(sum / (double)n);
    }
}

/* Algorithm 1, first half of an iteration: momentum update, local model update, buffer update. */
void ZO(zo_alg1_half_step)(ZO(zo_state) *st, const real *g, real gamma)
{
    const real one_minus_beta1 = (real)1 - st->beta1;
    for (int i = 0; i < st->n; ++i)
        for (int64_t j = 0; j < st->d; ++j) {
            size_t k = (size_t)i * st->d + j;
            real m_prev = st->m[k];
            real m_half = st->beta1 * m_prev + one_minus_beta1 * g[k];     /* momentum update */
            real m_used = st->literal_momentum ? m_prev : m_half;          /* R1 */
            real step = gamma * m_used;
            st->x[k] = st->x[k] - step / ZO(zo_sqrt)(st->v[j] + st->eps);    /* model update */
            st->u[k] = st->u[k] + step;                                    /* buffer update */
            st->m[k] = m_half;
        }
    st->gamma_sum += (double)gamma;                                        /* R2 */
}

/* Algorithm 1, the sync branch (t in T_u).  Returns 0, or -1 when nothing was accumulated
 * since the last sync (the divisor of the momentum approximation would be zero). */
int ZO(zo_alg1_sync)(ZO(zo_state) *st, int64_t t)
{
    if (!(st->gamma_sum > 0.0)) return -1;
    const real gamma_sum = (real)st->gamma_sum;
    ZO(zo_onebit_allreduce)(st, st->u);                                    /* 1-bit AllReduce */
    for (int64_t j = 0; j < st->d; ++j) {
        real m_next = st->u_bar[j] / gamma_sum;                            /* momentum approximation */
        real x_next = st->x_sync[j] - st->u_bar[j] / ZO(zo_sqrt)(st->v[j] + st->eps); /* model sync */
        for (int i = 0; i < st->n; ++i) {
            size_t k = (size_t)i * st->d + j;
            st->m[k] = m_next;
            st->x[k] = x_next;
            st->u[k] = (real)0;                                            /* buffer reset */
        }
        st->x_sync[j] = x_next;                                            /* R3 */
    }
    st->gamma_sum = 0.0;
    st->t_sync = t;                                                        /* t' = t */
    return 0;
}

/* Algorithm 1, the variance branch (t in T_v). */
void ZO(zo_alg1_variance)(ZO(zo_state) *st, const real *g, real *g_bar_scratch)
{
    const real one_minus_beta2 = (real)1 - st->beta2;
    ZO(zo_allreduce)(g, st->n, st->d, g_bar_scratch);                      /* full-precision AllReduce */
    for (int64_t j = 0; j < st->d; ++j) {
        real g_bar = g_bar_scratch[j];
        st->v[j] = st->beta2 * st->v[j] + one_minus_beta2 * (g_bar * g_bar); /* variance update */
    }
}

/* One whole iteration t of Algorithm 1 given the gradients g^(i)_t.
 * g_bar_scratch is [d]. */
int ZO(zo_alg1_step)(ZO(zo_state) *st, const real *g, real gamma, int64_t t,
                     int in_T_u, int in_T_v, real *g_bar_scratch)
{
    int rc = 0;
    ZO(zo_alg1_half_step)(st, g, gamma);
    if (in_T_u) rc = ZO(zo_alg1_sync)(st, t);   /* else: keep the half-step values */
    if (in_T_v) ZO(zo_alg1_variance)(st, g, g_bar_scratch); /* else: v stays (R8) */
    return rc;
}

/* One whole iteration t of Algorithm 2.  On a T_v step the workers
 * exchange full-precision gradients (Algorithm 4) and the variance moves; on
 * any other step they exchange 1-bit compressed gradients (Algorithm 3).
 * Momentum and model are the same on every worker; they are kept per worker
 * like the rest of the state.  g_bar_scratch is [d]. */
void ZO(zo_alg2_step)(ZO(zo_state) *st, const real *g, real gamma, int in_T_v, real *g_bar_scratch)
{
    const real one_minus_beta1 = (real)1 - st->beta1, one_minus_beta2 = (real)1 - st->beta2;
    const real *g_bar = g_bar_scratch;
    if (in_T_v) {
        ZO(zo_allreduce)(g, st->n, st->d, g_bar_scratch);                  /* AllReduce (t in T_v) */
    } else {
        ZO(zo_onebit_allreduce)(st, g);                                    /* Compressed-AllReduce (Algorithm 3) */
        g_bar = st->u_bar;
    }
    for (int i = 0; i < st->n; ++i)
        for (int64_t j = 0; j < st->d; ++j) {
            size_t k = (size_t)i * st->d + j;
            real m_prev = st->m[k];
            real m_next = st->beta1 * m_prev + one_minus_beta1 * g_bar[j]; /* Update momentum */
            real m_used = st->literal_momentum ? m_prev : m_next;          /* R9 */
            st->x[k] = st->x[k] - (gamma * m_used) / ZO(zo_sqrt)(st->v[j] + st->eps); /* Update model (reads v_t) */
            st->m[k] = m_next;
        }
    if (in_T_v)
        for (int64_t j = 0; j < st->d; ++j)
            st->v[j] = st->beta2 * st->v[j] + one_minus_beta2 * (g_bar[j] * g_bar[j]); /* Set v_{t+1} (else v_{t+1} = v_t) */
}
