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
 *   - Quantised communication (Section 3, "Quantized Communication": outer
 *     gradients sent as float32, bfloat16, float8 or float4 "using EXMY"): the
 *     operand of the all-reduce, and only it, is rounded: Delta = (1/M) sum_m
 *     Q_m(Delta_m); every local use of Delta_m (line 11's fresh and stale
 *     terms) stays in full precision.  The paper fixes no bit layout, so EXMY
 *     is read as: 1 sign bit, X exponent bits, Y mantissa bits, bias
 *     2^(X-1)-1, subnormals, every code a finite number (no inf/NaN codes),
 *     round to nearest with ties to the even code, saturating; each replica's
 *     vector is scaled so that its largest magnitude maps to the format's
 *     largest value (one fp32 scale per replica per outer step; the maximum
 *     propagates NaN and a scale that is zero or underflows to zero is
 *     replaced by 1, see amax_update / amax_to_scale).  PARITY
 *     UNPINNED against the paper for the EXMY layout and scaling (nothing is
 *     printed to pin them to); the rounding itself is pinned by brute force
 *     over every code, the E2M1 value table and a library's float8 casts.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py
 * (hand-worked dyadic example, exact rational brute force, closed forms,
 * torch.optim library routines, invariants).  "Parity unpinned" applies only
 * to readings that fill gaps the paper leaves open: the EXMY wire format
 * above, and overlaps of more than one outer step (the ring logic in
 * __init__.py: outer_step_overlap), for which the paper prints no formula.
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

/* communication format of the outer gradients */
enum { COMM_F32 = 0, COMM_BF16 = 1, COMM_EXMY = 2 };

/* largest finite EXMY value: top exponent code, all mantissa bits set */
static double exmy_max(int X, int Y)
{
    int bias = (1 << (X - 1)) - 1;
    int emax = (1 << X) - 1 - bias;
    return ldexp(2.0 - ldexp(1.0, -Y), emax);
}

/* the (X+Y)-bit code of a non-negative representable value v: exponent field << Y | mantissa */
static int exmy_code(double v, int X, int Y)
{
    int bias = (1 << (X - 1)) - 1;
    if (v < ldexp(1.0, 1 - bias)) return (int)(v / ldexp(1.0, 1 - bias - Y));   /* subnormal: field 0 */
    int e2;
    double f = frexp(v, &e2);           /* v = f * 2^e2, 0.5 <= f < 1 */
    int E = e2 - 1;
    int mant = (int)((2.0 * f - 1.0) * (double)(1 << Y));
    (void)X;
    return ((E + bias) << Y) | mant;
}

/*
 * Nearest EXMY(X, Y) number to y, ties to the even code, saturating.  Within
 * the binade 2^E <= |y| < 2^(E+1) the representable numbers are the multiples
 * of 2^(E-Y); below the smallest normal 2^(1-bias) the spacing stays
 * 2^(1-bias-Y) (subnormals).  The two neighbours are lo = floor(|y|/spacing) *
 * spacing and hi = lo + spacing (2^(E+1) when lo is the binade's last number);
 * all of this is exact in double.
 */
static double exmy_round(double y, int X, int Y)
{
    double a = fabs(y);
    if (a == 0.0 || a != a) return y;  /* zero keeps its sign; NaN stays NaN */
    if (isinf(a)) return y < 0 ? -exmy_max(X, Y) : exmy_max(X, Y); /* saturating, like any |y| > max */
    int bias = (1 << (X - 1)) - 1;
    int e2;
    (void)frexp(a, &e2);               /* a = f * 2^e2, 0.5 <= f < 1  =>  2^(e2-1) <= a */
    int E = e2 - 1;
    if (E < 1 - bias) E = 1 - bias;
    double spacing = ldexp(1.0, E - Y);
    double lo = floor(a / spacing) * spacing;
    double hi = lo + spacing;
    double q;
    if (a - lo < hi - a) q = lo;
    else if (a - lo > hi - a) q = hi;
    else q = (exmy_code(lo, X, Y) % 2 == 0) ? lo : hi;
    double top = exmy_max(X, Y);
    if (q > top) q = top;
    return y < 0 ? -q : q;
}

/*
 * Per-replica scale of the EXMY wire format.  amax = max_i |Delta_m[i]| where the maximum
 * PROPAGATES NaN (as IEEE 754-2019 `maximum` does): one NaN element makes amax NaN.
 * scale = amax / max(EXMY), except that a scale of zero (the replica did not move, or moved
 * so little that the quotient underflows to zero in REAL) is replaced by 1.  Consequences,
 * all by plain IEEE arithmetic in the lines below: a replica whose outer gradient holds a NaN
 * or an infinity has a NaN or infinite scale, and EVERY element it puts on the wire decodes
 * to NaN (x / NaN, 0 * inf): a non-finite outer gradient poisons that replica's whole
 * contribution instead of being silently clamped to the format's largest value.  (A reading:
 * the paper does not discuss non-finite values.  With the bf16 wire there is no scale and
 * NaN / infinity travel element by element.)
 */
static REAL amax_update(REAL amax, REAL d)
{
    REAL ab = d < 0 ? -d : d;
    if (ab != ab) return ab;            /* NaN enters ... */
    if (amax != amax) return amax;      /* ... and stays */
    return ab > amax ? ab : amax;
}

static REAL amax_to_scale(REAL amax, int X, int Y)
{
    REAL scale = amax / (REAL)exmy_max(X, Y);
    if (scale == (REAL)0) scale = (REAL)1;
    return scale;
}

/* what the wire carries for one element of replica m's outer gradient */
static REAL comm_round(REAL d, int comm, int X, int Y, REAL scale)
{
    if (comm == COMM_F32) return d;
    if (comm == COMM_BF16) return (REAL)bf16_to_f32(f32_to_bf16_rne((float)d));
    REAL y = d / scale;
    REAL q = (REAL)exmy_round((double)y, X, Y);
    return q * scale;
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
int FN(oracle_outer_step_comm)(int variant, int bootstrap, int M, int64_t P, int64_t stride,
                               REAL eta, REAL mu, int theta_kind,
                               void *theta, REAL *master, REAL *start,
                               REAL *delta_prev_local, REAL *delta_prev_avg, REAL *outer_mom,
                               int comm, int X, int Y, REAL *scales_out, int nthreads)
{
    if (M < 1 || M > 64 || P < 0 || stride < P) return -1;
    if (variant < VAR_STANDARD || variant > VAR_EAGER) return -1;
    if (variant == VAR_STANDARD && bootstrap) return -1;
    if (comm < COMM_F32 || comm > COMM_EXMY) return -1;
    if (comm == COMM_EXMY && (X < 1 || X > 5 || Y < 0 || X + Y > 7)) return -1;
    (void)nthreads;
    /* per-replica scale: largest |Delta_m| maps to the largest EXMY value */
    REAL scale[64];
    for (int m = 0; m < M; ++m) scale[m] = (REAL)1;
    if (comm == COMM_EXMY) {
        for (int m = 0; m < M; ++m) {
            REAL amax = (REAL)0;
            for (int64_t i = 0; i < P; ++i) {
                size_t at = (size_t)m * (size_t)stride + (size_t)i;
                REAL dm = start[at] - load_theta(theta_kind, theta, master, at);
                amax = amax_update(amax, dm);
            }
            scale[m] = amax_to_scale(amax, X, Y);
            if (scales_out) scales_out[m] = scale[m];
        }
    }
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
    for (int64_t i = 0; i < P; ++i) {
        REAL d[64];
        /* Alg. 1-3 line 7: Delta_m = theta_m^(t-H) - theta_m^(t) */
        for (int m = 0; m < M; ++m) {
            size_t at = (size_t)m * (size_t)stride + (size_t)i;
            REAL x = load_theta(theta_kind, theta, master, at);
            d[m] = start[at] - x;
        }
        /* line 8: Delta = (1/M) sum_m Delta_m, summed m = 1..M in order; what is summed is
           what each worker put on the wire */
        REAL acc = comm_round(d[0], comm, X, Y, scale[0]);
        for (int m = 1; m < M; ++m) acc = acc + comm_round(d[m], comm, X, Y, scale[m]);
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

/* full-precision communication (the three algorithms as printed) */
int FN(oracle_outer_step)(int variant, int bootstrap, int M, int64_t P, int64_t stride,
                          REAL eta, REAL mu, int theta_kind,
                          void *theta, REAL *master, REAL *start,
                          REAL *delta_prev_local, REAL *delta_prev_avg, REAL *outer_mom,
                          int nthreads)
{
    return FN(oracle_outer_step_comm)(variant, bootstrap, M, P, stride, eta, mu, theta_kind, theta, master, start,
                                      delta_prev_local, delta_prev_avg, outer_mom, COMM_F32, 0, 0, NULL, nthreads);
}

/* exported so that tests can pin the EXMY rounding on its own */
double FN(oracle_exmy_round)(double y, int X, int Y) { return exmy_round(y, X, Y); }
double FN(oracle_exmy_max)(int X, int Y) { return exmy_max(X, Y); }

/*
 * Wire format of one worker's quantised outer gradient (the bytes an EXMY all-gather would
 * carry; a reading, like EXMY itself: the paper prints none).  Each element is the code
 * sign << (X+Y) | exponent field << Y | mantissa of R(d / scale), scale = amax / max(EXMY)
 * (1 if amax = 0), amax = max |d|.  Codes of at most 4 bits are packed two per byte
 * (element 2j in bits 0-3, element 2j+1 in bits 4-7), wider codes take one byte each.
 */
static int wire_packed(int X, int Y) { return X + Y + 1 <= 4; }

int FN(oracle_wire_encode)(int64_t P, const REAL *d, int X, int Y, uint8_t *payload, REAL *amax_out)
{
    if (P < 0 || X < 1 || X > 5 || Y < 0 || X + Y > 7) return -1;
    REAL amax = (REAL)0;
    for (int64_t i = 0; i < P; ++i) amax = amax_update(amax, d[i]);
    REAL scale = amax_to_scale(amax, X, Y);
    const int packed = wire_packed(X, Y);
    if (packed) memset(payload, 0, (size_t)((P + 1) / 2));
    for (int64_t i = 0; i < P; ++i) {
        REAL y = d[i] / scale;
        double q = exmy_round((double)y, X, Y);
        /* every code is a finite number, so NaN has none.  y is NaN only when this worker's
           scale is NaN or infinite; it then travels as code 0 (+0), which the receiver's
           value(code) * scale turns back into NaN (0 * NaN, 0 * inf): same result as the fused step */
        int code = (q != q) ? 0 : exmy_code(fabs(q), X, Y) | ((signbit(q) ? 1 : 0) << (X + Y));
        if (packed) payload[i / 2] |= (uint8_t)(code << (4 * (i & 1)));
        else payload[i] = (uint8_t)code;
    }
    *amax_out = amax;
    return 0;
}

/* value of a code, from the definition of the format */
static double exmy_decode(int code, int X, int Y)
{
    int bias = (1 << (X - 1)) - 1;
    int sign = (code >> (X + Y)) & 1;
    int e = (code >> Y) & ((1 << X) - 1);
    int m = code & ((1 << Y) - 1);
    double v = e == 0 ? ldexp((double)m, 1 - bias - Y) : ldexp((double)((1 << Y) + m), e - bias - Y);
    return sign ? -v : v;
}

/* sum_out[i] = sum over workers m = 0 .. M-1, in order, of scale_m * value(code_m[i]) */
int FN(oracle_wire_decode_sum)(int M, int64_t P, int64_t payload_stride, const uint8_t *payloads,
                               const REAL *amaxes, int X, int Y, REAL *sum_out)
{
    if (M < 1 || P < 0 || X < 1 || X > 5 || Y < 0 || X + Y > 7) return -1;
    const int packed = wire_packed(X, Y);
    for (int64_t i = 0; i < P; ++i) {
        REAL acc = (REAL)0;
        for (int m = 0; m < M; ++m) {
            const uint8_t *row = payloads + (size_t)m * (size_t)payload_stride;
            int code = packed ? (row[i / 2] >> (4 * (i & 1))) & 15 : row[i];
            REAL scale = amax_to_scale(amaxes[m], X, Y);
            REAL w = (REAL)exmy_decode(code, X, Y) * scale;
            acc = (m == 0) ? w : acc + w;
        }
        sum_out[i] = acc;
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
