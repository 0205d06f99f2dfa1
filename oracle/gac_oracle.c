/*
 * gac_oracle.c -- CPU oracle for the Gradient Alignment Control (GAC) hot path.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64
 * restatement of what the paper defines, used only to check the CUDA library
 * and to be timed as a CPU baseline.  It shares no code, header, table or
 * helper with the CUDA path and must never be called from it.
 *
 * What it computes (paper passages):
 *   - the three inner products <g,d>, <g,g>, <d,d> over the flattened
 *     concatenation of all gradient tensors         (App. A.1, the two
 *     displayed triples of inner products; Eq. 1)
 *   - c = <g,d> / (sqrt(<g,g> <d,d>) + eps)          (App. A.1, cosine with eps)
 *   - the three regimes on |c|                       (Sec. 4.2; Algorithm 1)
 *   - alpha = c_low/|c|, beta = 1                    (Eq. 5; App. A.2)
 *   - g' = beta g + (alpha-beta) <g,u> u, u = d/|d|  (Eq. 2-3; App. A.2 rank-one form)
 *   - the stored direction becomes the raw gradient  (App. A.2 "Memory footprint";
 *     App. A.1 "Evaluation protocol"; Algorithm 1 compares with g_{t-1})
 *
 * Every pin that ties these functions to the paper and to mathematics lives in
 * tests/test_oracle_*.py; nothing here is "parity unpinned".
 *
 * Element types: 0 = IEEE binary32, 1 = bfloat16 (upper 16 bits of a binary32).
 * All pointers are host pointers.  Nothing here allocates.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

#define ORC_SAFE 0
#define ORC_PROJECT 1
#define ORC_VIOLATION 2

#define ORC_MODE_ADAPTIVE 0
#define ORC_MODE_FIXED 1

#define ORC_STATE_RAW 0
#define ORC_STATE_PROJECTED 1
#define ORC_STATE_HOLD 2

/* ---- element access ----------------------------------------------------- */

static double elem_as_double(const void *p, int dt, uint64_t i)
{
    if (dt == ORC_F32)
        return (double)((const float *)p)[i];
    /* bfloat16: the 16 stored bits are the top half of a binary32 pattern */
    uint32_t w = (uint32_t)((const uint16_t *)p)[i] << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bfloat16 (ties to even), directly, with no
 * intermediate binary32 rounding.  bfloat16 has 8 significant bits, minimum
 * normal exponent 2^-126, subnormal spacing 2^-133, largest finite value
 * (2 - 2^-7) 2^127. */
static uint16_t double_to_bf16_bits(double x)
{
    if (isnan(x))
        return 0x7FC0;
    double ax = fabs(x);
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    if (isinf(x))
        return (uint16_t)(sign | 0x7F80);
    if (ax == 0.0)
        return sign;
    int e;
    (void)frexp(ax, &e);               /* ax = m 2^e, m in [0.5,1) */
    int qexp = e - 8;                  /* spacing of 8-significant-bit values */
    if (qexp < -133)
        qexp = -133;                   /* subnormal range: fixed spacing */
    double q = nearbyint(ldexp(ax, -qexp)); /* default mode: nearest, ties to even */
    double r = ldexp(q, qexp);         /* exactly a bfloat16 value or 2^128 */
    if (r > 0x1.FEp127)
        return (uint16_t)(sign | 0x7F80);
    float f = (float)r;                /* exact: r has at most 8 significant bits */
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    return (uint16_t)(sign | (uint16_t)(w >> 16));
}

void orc_round_to_bf16(const double *x, uint16_t *out, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i)
        out[i] = double_to_bf16_bits(x[i]);
}

static void store_rounded(void *p, int dt, uint64_t i, double v)
{
    if (dt == ORC_F32)
        ((float *)p)[i] = (float)v;    /* C conversion: nearest, ties to even */
    else
        ((uint16_t *)p)[i] = double_to_bf16_bits(v);
}

/* ---- step 1: the three inner products (App. A.1) ------------------------ */

/* Running Neumaier-compensated sums for dot, gg, dd, so that a list of
 * tensors is accumulated as ONE sum over the logical concatenation. */
typedef struct {
    double sum[3];
    double comp[3];
} orc_acc;

void orc_acc_init(orc_acc *a)
{
    for (int k = 0; k < 3; ++k) {
        a->sum[k] = 0.0;
        a->comp[k] = 0.0;
    }
}

static void neumaier_add(double *sum, double *comp, double x)
{
    double t = *sum + x;
    if (fabs(*sum) >= fabs(x))
        *comp += (*sum - t) + x;
    else
        *comp += (x - t) + *sum;
    *sum = t;
}

/* Adds elements [0,n) of one tensor pair.  d_is_zero != 0 means the stored
 * direction is the all-zero vector g_0 of Algorithm 1 (first step): d is not
 * read at all and contributes nothing to dot and dd. */
void orc_stats_accumulate(orc_acc *a, const void *g, int g_dt, const void *d, int d_dt,
                          uint64_t n, int d_is_zero)
{
    for (uint64_t i = 0; i < n; ++i) {
        double gi = elem_as_double(g, g_dt, i);
        neumaier_add(&a->sum[1], &a->comp[1], gi * gi);
        if (!d_is_zero) {
            double di = elem_as_double(d, d_dt, i);
            neumaier_add(&a->sum[0], &a->comp[0], gi * di);
            neumaier_add(&a->sum[2], &a->comp[2], di * di);
        }
    }
}

void orc_acc_value(const orc_acc *a, double out[3])
{
    for (int k = 0; k < 3; ++k)
        out[k] = a->sum[k] + a->comp[k];
}

/* Merge b into a (used when fixed ranges were accumulated separately). */
void orc_acc_merge(orc_acc *a, const orc_acc *b)
{
    for (int k = 0; k < 3; ++k) {
        neumaier_add(&a->sum[k], &a->comp[k], b->sum[k]);
        neumaier_add(&a->sum[k], &a->comp[k], b->comp[k]);
    }
}

/* Second, independent summation order: recursive pairwise halves. */
static void pairwise(const void *g, int g_dt, const void *d, int d_dt, uint64_t lo, uint64_t hi,
                     double out[3])
{
    if (hi - lo <= 8) {
        out[0] = out[1] = out[2] = 0.0;
        for (uint64_t i = lo; i < hi; ++i) {
            double gi = elem_as_double(g, g_dt, i);
            double di = elem_as_double(d, d_dt, i);
            out[0] += gi * di;
            out[1] += gi * gi;
            out[2] += di * di;
        }
        return;
    }
    uint64_t mid = lo + (hi - lo) / 2;
    double l[3], r[3];
    pairwise(g, g_dt, d, d_dt, lo, mid, l);
    pairwise(g, g_dt, d, d_dt, mid, hi, r);
    for (int k = 0; k < 3; ++k)
        out[k] = l[k] + r[k];
}

void orc_stats_pairwise(const void *g, int g_dt, const void *d, int d_dt, uint64_t n, double out[3])
{
    pairwise(g, g_dt, d, d_dt, 0, n, out);
}

/* ---- steps 2-4: cosine, regime, gains (App. A.1; Algorithm 1; Eq. 5) ----- */

typedef struct {
    double c_low, c_high;     /* Algorithm 1 inputs, 0 < c_low < c_high            */
    double eps;               /* App. A.1 cosine denominator term, 1e-8 in the paper */
    double beta;              /* orthogonal gain, 1 in the paper (App. A.2)         */
    int32_t mode;             /* ORC_MODE_ADAPTIVE: Eq. 5; ORC_MODE_FIXED: Eq. 3    */
    int32_t state_mode;       /* ORC_STATE_RAW is the paper's rule                  */
    double alpha_fixed;       /* parallel gain used when mode == FIXED              */
    int32_t zero_on_violation;
    int32_t reserved;
    double clip_max_norm;     /* > 0: global-norm clipping of the outgoing gradient (Table 2:
                                 "Gradient clipping True"), applied after the GAC rule; 0 = off */
    double clip_eps;          /* added to the norm in the clip factor, 1e-6 as in torch's
                                 clip_grad_norm_ */
} orc_hparams;

typedef struct {
    double dot, gg, dd;
    double cosine;
    double alpha;             /* parallel gain actually used (1 when nothing is changed) */
    double coef64;            /* (alpha - beta) <g,d>/<d,d>, multiplies d in the rank-one form */
    float coef;               /* coef64 rounded once to binary32: the number both sides share */
    int32_t regime;
    int32_t nonfinite;
    int32_t reserved;
} orc_decision;

void orc_decide(const double sums[3], const orc_hparams *hp, int first_step, orc_decision *o)
{
    double dot = sums[0], gg = sums[1], dd = sums[2];
    if (first_step) {                  /* Algorithm 1: g_0 = 0 */
        dot = 0.0;
        dd = 0.0;
    }
    o->dot = dot;
    o->gg = gg;
    o->dd = dd;
    o->alpha = 1.0;
    o->coef64 = 0.0;
    o->coef = 0.0f;
    o->reserved = 0;
    o->nonfinite = !(isfinite(dot) && isfinite(gg) && isfinite(dd));
    if (o->nonfinite) {
        /* The paper is silent on NaN/Inf gradients.  Reading taken: report
         * them, treat the step as a violation (skip), leave g and d alone. */
        o->cosine = NAN;
        o->regime = ORC_VIOLATION;
        return;
    }
    /* Zero reference or zero gradient: u = 0 and the projector is the
     * identity (App. F, definition of u_{t-1} and first line of the proof),
     * so the step is safe and nothing is divided by <d,d>. */
    if (gg == 0.0 || dd == 0.0) {
        o->cosine = 0.0;
        o->regime = ORC_SAFE;
        return;
    }
    o->cosine = dot / (sqrt(gg * dd) + hp->eps);   /* App. A.1: eps outside the root */
    double ac = fabs(o->cosine);

    if (hp->mode == ORC_MODE_FIXED) {
        /* Eq. 3 with caller-given gains, applied on every step */
        o->regime = ORC_PROJECT;
        o->alpha = hp->alpha_fixed;
    } else if (ac <= hp->c_low) {      /* Algorithm 1, first branch (inclusive) */
        o->regime = ORC_SAFE;
        return;
    } else if (ac >= hp->c_high) {     /* Algorithm 1, second branch (inclusive) */
        o->regime = ORC_VIOLATION;
        return;
    } else {
        o->regime = ORC_PROJECT;
        o->alpha = hp->c_low / ac;     /* Eq. 5 */
    }
    /* App. A.2: g' = beta g + (alpha-beta) <g,u> u with u = d/|d|, i.e. the
     * multiplier of d is (alpha-beta) <g,d>/<d,d>.  eps does not enter here. */
    o->coef64 = (o->alpha - hp->beta) * dot / dd;
    o->coef = (float)o->coef64;
}

/* ---- steps 5-6: in-place rank-one update and state refresh (App. A.2) ---- */

/* Squared Euclidean norm of the gradient that the rule sends on, before any
 * clipping and before rounding: sum over i of (beta g_i + coef d_i)^2 in the
 * projection regime, of g_i^2 in the safe regime.  Accumulated into a->sum[0]
 * with Neumaier compensation so that a list can be fed tensor by tensor. */
void orc_outgoing_sqnorm(orc_acc *a, const void *g, int g_dt, const void *d, int d_dt, uint64_t n,
                         const orc_hparams *hp, int regime, float coef, int d_is_zero)
{
    for (uint64_t i = 0; i < n; ++i) {
        double gi = elem_as_double(g, g_dt, i);
        double out = gi;
        if (regime == ORC_PROJECT) {
            double di = d_is_zero ? 0.0 : elem_as_double(d, d_dt, i);
            out = hp->beta * gi + (double)coef * di;
        }
        neumaier_add(&a->sum[0], &a->comp[0], out * out);
    }
}

/* Global-norm clip factor: min(1, max_norm / (norm + clip_eps)). */
double orc_clip_scale(double sqnorm, const orc_hparams *hp)
{
    if (!(hp->clip_max_norm > 0.0))
        return 1.0;
    double f = hp->clip_max_norm / (sqrt(sqnorm) + hp->clip_eps);
    return f < 1.0 ? f : 1.0;
}

/* g (type g_dt) and d (binary32) are updated in place over n elements, given
 * the decision.  d is binary32, or bfloat16 when g is bfloat16 (a snapshot of
 * half the size).  coef is the shared binary32 coefficient.  d_is_zero: d holds
 * no valid data on the first step and is only written.  clip_scale (1 = none)
 * multiplies the outgoing gradient of a safe or projection step; a skipped
 * step sends nothing on, so it is not scaled. */
void orc_project(void *g, int g_dt, void *d, int d_dt, uint64_t n, const orc_hparams *hp, int regime,
                 int nonfinite, float coef, int d_is_zero, double clip_scale)
{
    if (nonfinite)
        return;                        /* reading above: touch nothing */
    for (uint64_t i = 0; i < n; ++i) {
        double gi = elem_as_double(g, g_dt, i);
        double gout = gi;
        int write_g = 0;
        if (regime == ORC_PROJECT) {
            double di = d_is_zero ? 0.0 : elem_as_double(d, d_dt, i);
            gout = hp->beta * gi + (double)coef * di;
            write_g = 1;
        } else if (regime == ORC_VIOLATION && hp->zero_on_violation) {
            gout = 0.0;
            write_g = 1;
        }
        if (clip_scale != 1.0 && regime != ORC_VIOLATION) {
            gout = clip_scale * gout;
            write_g = 1;
        }
        if (write_g)
            store_rounded(g, g_dt, i, gout);
        if (hp->state_mode == ORC_STATE_RAW) {
            store_rounded(d, d_dt, i, gi);   /* exact whenever d is at least as wide as g */
        } else if (hp->state_mode == ORC_STATE_PROJECTED) {
            store_rounded(d, d_dt, i, elem_as_double(g, g_dt, i));
        }                              /* ORC_STATE_HOLD: d unchanged */
    }
}

/* ---- the step after the path: GAC output consumed by AdamW --------------- */

/* Algorithm 1 hands the (safe or projected) gradient to the optimizer; the
 * paper trains with AdamW (Table 2: lr 1e-6, betas (0.9, 0.999), eps 1e-8,
 * weight decay 1e-2).  This is the decoupled-weight-decay Adam of Loshchilov
 * and Hutter as commonly implemented:
 *     p <- p (1 - lr wd)
 *     m <- b1 m + (1 - b1) g'          v <- b2 v + (1 - b2) g'^2
 *     p <- p - (lr / (1 - b1^t)) m / (sqrt(v) / sqrt(1 - b2^t) + eps)
 * with t the number of updates applied so far including this one, fed with the
 * UNROUNDED g' = clip_scale (beta g + coef d) (projection) or clip_scale g
 * (safe).  A skipped step (violation) leaves p, m, v alone: theta_t = theta_{t-1}.
 * g itself is not written.  d is refreshed as in orc_project.  p, m, v are binary32. */
typedef struct {
    double lr, beta1, beta2, eps, weight_decay;
} orc_adamw;

void orc_project_adamw(const void *g, int g_dt, void *d, int d_dt, float *p, float *m, float *v, uint64_t n,
                       const orc_hparams *hp, int regime, int nonfinite, float coef, int d_is_zero,
                       double clip_scale, const orc_adamw *o, uint64_t t)
{
    if (nonfinite)
        return;
    double bc1 = 1.0 - pow(o->beta1, (double)t);
    double bc2 = 1.0 - pow(o->beta2, (double)t);
    double step_size = o->lr / bc1;
    double sqrt_bc2 = sqrt(bc2);
    for (uint64_t i = 0; i < n; ++i) {
        double gi = elem_as_double(g, g_dt, i);
        if (regime != ORC_VIOLATION) {
            double gout = gi;
            if (regime == ORC_PROJECT) {
                double di = d_is_zero ? 0.0 : elem_as_double(d, d_dt, i);
                gout = hp->beta * gi + (double)coef * di;
            }
            if (clip_scale != 1.0)
                gout = clip_scale * gout;
            double pi = (double)p[i] * (1.0 - o->lr * o->weight_decay);
            double mi = o->beta1 * (double)m[i] + (1.0 - o->beta1) * gout;
            double vi = o->beta2 * (double)v[i] + (1.0 - o->beta2) * gout * gout;
            double denom = sqrt(vi) / sqrt_bc2 + o->eps;
            pi = pi - step_size * (mi / denom);
            p[i] = (float)pi;
            m[i] = (float)mi;
            v[i] = (float)vi;
        }
        if (hp->state_mode == ORC_STATE_RAW)
            store_rounded(d, d_dt, i, gi);
        /* other state modes are not offered by the fused form */
    }
}
