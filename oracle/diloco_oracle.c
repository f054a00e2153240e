/*
 * CPU oracle for the DiLoCo outer-optimisation step (standard, naive delayed,
 * eager) and the inner AdamW step.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * index-by-index restatement of Algorithms 1-3 of the paper, used only by the
 * test-suite, by the smoke check and by the benchmark's CPU-baseline leg.  It
 * shares no code with the CUDA library and the CUDA library never calls it.
 *
 * The file is compiled twice into one shared object:
 *     -DREAL=float  -DSFX=f32   one IEEE round-to-nearest per written operation
 *                               (build with -ffp-contract=off: no FMA fusion);
 *                               this is the parity target of the GPU kernels
 *     -DREAL=double -DSFX=f64   the same steps in double, the "truth" used for
 *                               tolerance checks and closed-form pins
 *
 * Notation follows the paper: M replicas, theta_m current parameters of
 * replica m, s_m = theta_m^(t-H) the start-of-phase ("outer") parameters,
 * Delta_m the local outer gradient, Delta the all-reduced mean, b_m the
 * momentum buffer of OuterOpt, eta / mu the outer learning rate / momentum.
 *
 * Readings of points the paper leaves open (each is a choice, listed in the
 * design notes of the repository):
 *   - OuterOpt = SGD with Nesterov momentum (Section 2.1) in the form
 *         b <- mu*b + g ;  theta <- theta - eta*(g + mu*b),  b initially 0.
 *   - OuterOpt state (s_m, b_m) is per replica for every variant: the call
 *     sits inside the "parallel for m" loop with per-replica arguments.
 *   - 1/M is a division by (REAL)M; the sum over m runs left to right.
 *   - InnerOpt = AdamW with decoupled weight decay, bias correction,
 *     eps added after the square root.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py
 * (hand-worked dyadic example, exact rational brute force, closed forms,
 * torch.optim library routines, invariants); nothing is "parity unpinned"
 * except the readings above themselves, which the paper cannot settle.
 *
 * Layout: every [M, stride] buffer is replica-major, element (m, i) at
 * m*stride + i, only i < P is touched.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifndef REAL
#error "compile with -DREAL=float -DSFX=f32 or -DREAL=double -DSFX=f64"
#endif

#define CAT2(a, b) a##_##b
#define CAT(a, b) CAT2(a, b)
#define FN(name) CAT(name, SFX)

enum { VAR_STANDARD = 0, VAR_DELAYED = 1, VAR_EAGER = 2 };
/* storage of theta: native REAL; bf16 only; REAL master + bf16 working copy */
enum { THETA_NATIVE = 0, THETA_BF16 = 1, THETA_MASTER_BF16 = 2 };
enum { GRAD_NATIVE = 0, GRAD_BF16 = 1 };

/* bf16 <-> fp32: bf16 is the upper 16 bits of an IEEE binary32. */
static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even on the 16 discarded bits; NaN stays NaN (quiet). */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

static REAL load_theta(int kind, const void *theta, const REAL *master, size_t at)
{
    if (kind == THETA_NATIVE) return ((const REAL *)theta)[at];
    if (kind == THETA_BF16) return (REAL)bf16_to_f32(((const uint16_t *)theta)[at]);
    return master[at]; /* THETA_MASTER_BF16: the master copy is the value */
}

static void store_theta(int kind, void *theta, REAL *master, size_t at, REAL x)
{
    if (kind == THETA_NATIVE) {
        ((REAL *)theta)[at] = x;
    } else if (kind == THETA_BF16) {
        ((uint16_t *)theta)[at] = f32_to_bf16_rne((float)x);
    } else {
        master[at] = x;
        ((uint16_t *)theta)[at] = f32_to_bf16_rne((float)x);
    }
}

/*
 * One outer step at index range [0, P) for all M replicas.
 *
 *   variant    VAR_STANDARD  Algorithm 1, lines 7-10
 *              VAR_DELAYED   Algorithm 2, lines 7-11
 *              VAR_EAGER     Algorithm 3, lines 7-12
 *   bootstrap  1 = this is the first outer step (t = H) of a delayed / eager
 *              run: the "if t > H" branch is not taken, nothing is applied;
 *              the local gradients and their mean are recorded and the
 *              current theta_m becomes the next start point.
 *
 * Buffers (REAL unless noted): theta [M,stride] (storage per theta_kind),
 * master [M,stride] or NULL, start [M,stride], delta_prev_local [M,stride]
 * (eager only), delta_prev_avg [stride] (delayed, eager), outer_mom
 * [M,stride].  All updated in place.  Returns 0, or -1 on a bad argument.
 */
int FN(oracle_outer_step)(int variant, int bootstrap, int M, int64_t P, int64_t stride,
                          REAL eta, REAL mu, int theta_kind,
                          void *theta, REAL *master, REAL *start,
                          REAL *delta_prev_local, REAL *delta_prev_avg, REAL *outer_mom,
                          int nthreads)
{
    if (M < 1 || M > 64 || P < 0 || stride < P) return -1;
    if (variant < VAR_STANDARD || variant > VAR_EAGER) return -1;
    if (variant == VAR_STANDARD && bootstrap) return -1;
    (void)nthreads;
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
    for (int64_t i = 0; i < P; ++i) {
        REAL d[64];
        /* Alg. 1-3 line 7: Delta_m = theta_m^(t-H) - theta_m^(t) */
        for (int m = 0; m < M; ++m) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            REAL x = load_theta(theta_kind, theta, master, at);
            d[m] = start[at] - x;
        }
        /* line 8: Delta = (1/M) sum_m Delta_m, summed m = 1..M in order */
        REAL acc = d[0];
        for (int m = 1; m < M; ++m) acc = acc + d[m];
        REAL D_new = acc / (REAL)M;

        if (bootstrap) {
            /* t = H: "if t > H" fails, no OuterOpt call */
            for (int m = 0; m < M; ++m) {
                size_t at = (size_t)m * (size_t)stride + (size_t)i;
                REAL x = load_theta(theta_kind, theta, master, at);
                if (variant == VAR_EAGER) delta_prev_local[at] = d[m];
                start[at] = x;
            }
            delta_prev_avg[i] = D_new;
            continue;
        }

        /* the all-reduce started one phase ago has landed (block-receive) */
        REAL D_old = (variant == VAR_STANDARD) ? (REAL)0 : delta_prev_avg[i];

        for (int m = 0; m < M; ++m) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            REAL g;
            if (variant == VAR_STANDARD) {
                g = D_new;                              /* Alg. 1 line 10 */
            } else if (variant == VAR_DELAYED) {
                g = D_old;                              /* Alg. 2 line 11 */
            } else {
                /* Alg. 3 line 11: (1/M)(Delta_m^(t) - Delta_m^(t-H)) + Delta^(t-H) */
                REAL e = d[m] - delta_prev_local[at];
                e = e / (REAL)M;
                g = e + D_old;
            }
            /* OuterOpt(theta_m^(t-H), g): SGD with Nesterov momentum */
            REAL b = mu * outer_mom[at];
            b = b + g;
            REAL u = mu * b;
            u = g + u;
            u = eta * u;
            REAL n = start[at] - u;
            outer_mom[at] = b;
            start[at] = n;                              /* next phase's theta^(t-H) */
            store_theta(theta_kind, theta, master, at, n);
            if (variant == VAR_EAGER) delta_prev_local[at] = d[m];
        }
        if (variant != VAR_STANDARD) delta_prev_avg[i] = D_new; /* now in flight */
    }
    return 0;
}

/*
 * The eager outer gradient in the paper's second, equivalent form (Section
 * 2.3 prose): tilde Delta_m = (1/M) (Delta_m^(t) + sum_{m' != m} Delta_{m'}^(t-H)).
 * A real worker cannot evaluate it (it needs every stale local gradient);
 * it exists only to cross-check line 11 of Algorithm 3.  out [M,stride].
 */
int FN(oracle_eager_gradient_form_b)(int M, int64_t P, int64_t stride, int theta_kind,
                                     const void *theta, const REAL *master, const REAL *start,
                                     const REAL *delta_prev_local, REAL *out)
{
    if (M < 1 || M > 64 || P < 0 || stride < P) return -1;
    for (int64_t i = 0; i < P; ++i) {
        for (int m = 0; m < M; ++m) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            REAL x = load_theta(theta_kind, theta, master, at);
            REAL acc = start[at] - x;
            for (int q = 0; q < M; ++q) {
                if (q == m) continue;
                acc = acc + delta_prev_local[(size_t)q * (size_t)stride + (size_t)i];
            }
            out[at] = acc / (REAL)M;
        }
    }
    return 0;
}

/* Same for line 11 itself, without applying it.  out [M,stride]. */
int FN(oracle_eager_gradient_form_a)(int M, int64_t P, int64_t stride, int theta_kind,
                                     const void *theta, const REAL *master, const REAL *start,
                                     const REAL *delta_prev_local, const REAL *delta_prev_avg,
                                     REAL *out)
{
    if (M < 1 || M > 64 || P < 0 || stride < P) return -1;
    for (int64_t i = 0; i < P; ++i) {
        for (int m = 0; m < M; ++m) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            REAL x = load_theta(theta_kind, theta, master, at);
            REAL e = (start[at] - x) - delta_prev_local[at];
            e = e / (REAL)M;
            out[at] = e + delta_prev_avg[i];
        }
    }
    return 0;
}

/*
 * One inner AdamW step, number k >= 1 since the moments were zero, for all M
 * replicas (Alg. 1-3 line 5 with InnerOpt = AdamW).
 *
 *   m <- beta1 m + (1-beta1) g            v <- beta2 v + (1-beta2) g g
 *   mhat = m / (1 - beta1^k)              vhat = v / (1 - beta2^k)
 *   theta <- theta - lr * ( mhat / (sqrt(vhat) + eps) + wd * theta )
 *
 * The bias corrections and (1-beta) are formed once, outside the loop; the
 * corrections in double and then rounded to REAL.  grads [M,gstride] in REAL
 * or bf16.  Moments are REAL.  Returns 0, or -1 on a bad argument.
 */
int FN(oracle_inner_adamw)(int M, int64_t P, int64_t stride, int64_t gstride,
                           REAL lr, REAL beta1, REAL beta2, REAL eps, REAL wd, int64_t k,
                           int theta_kind, int grad_kind,
                           void *theta, REAL *master, const void *grads,
                           REAL *adam_m, REAL *adam_v, int nthreads)
{
    if (M < 1 || P < 0 || stride < P || gstride < P || k < 1) return -1;
    const REAL c1 = (REAL)(1.0 - pow((double)beta1, (double)k));
    const REAL c2 = (REAL)(1.0 - pow((double)beta2, (double)k));
    const REAL omb1 = (REAL)1 - beta1;
    const REAL omb2 = (REAL)1 - beta2;
    (void)nthreads;
    for (int m = 0; m < M; ++m) {
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
        for (int64_t i = 0; i < P; ++i) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            size_t gat = (size_t)m * (size_t)gstride + (size_t)i;
            REAL g = (grad_kind == GRAD_NATIVE)
                         ? ((const REAL *)grads)[gat]
                         : (REAL)bf16_to_f32(((const uint16_t *)grads)[gat]);
            REAL x = load_theta(theta_kind, theta, master, at);
            REAL t1 = beta1 * adam_m[at];
            REAL t2 = omb1 * g;
            REAL m1 = t1 + t2;
            REAL t3 = beta2 * adam_v[at];
            REAL t4 = omb2 * g;
            t4 = t4 * g;
            REAL v1 = t3 + t4;
            REAL mh = m1 / c1;
            REAL vh = v1 / c2;
#if defined(ORACLE_REAL_IS_DOUBLE)
            REAL den = sqrt(vh) + eps;
#else
            REAL den = sqrtf(vh) + eps;
#endif
            REAL a = mh / den;
            REAL w = wd * x;
            REAL upd = a + w;
            upd = lr * upd;
            REAL x1 = x - upd;
            adam_m[at] = m1;
            adam_v[at] = v1;
            store_theta(theta_kind, theta, master, at, x1);
        }
    }
    return 0;
}

/* exported so that tests can pin the bf16 rounding on its own */
uint16_t FN(oracle_f32_to_bf16)(float f) { return f32_to_bf16_rne(f); }
float FN(oracle_bf16_to_f32)(uint16_t h) { return bf16_to_f32(h); }
