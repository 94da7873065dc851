/*
 * ampq_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, double-precision CPU statement of the loss-MSE sensitivity
 * pass of "Automatic mixed precision for optimizing gained time with
 * constrained loss mean-squared-error based on model partition to sequential
 * sub-graphs" (Sec. 2.1-2.2, Algorithm 1 steps 2 and 4).  It exists so that the
 * CUDA library can be compared with something written independently from the
 * paper.  It shares no code, header, table or constant generator with the CUDA
 * path and nothing in the product may call it.  Only the tests, the smoke check
 * and the bench's CPU-baseline leg load it.
 *
 * What is fixed by the paper and what is a reading of it:
 *   - sensitivity  s_l^r = || z_l^r (.) dg/dz_l^r ||^2          (Sec. 2.2, the
 *     equation that defines the per-sample sensitivity) -> orc_score_segment,
 *     accumulator S;
 *   - mean sensitivity s_l = (1/R) sum_r s_l^r, d_{l,f} = s_l alpha_f, with
 *     alpha_f = 2^(-2 m_f) / 12 (Sec. 2.2, noise-variance equation) ->
 *     orc_layer_combine, orc_alpha;
 *   - group loss-MSE d_{j,p} = sum_l s_{l_{j,l}} alpha_{Q_j[l,p]} (Sec. 2.2,
 *     last equation) -> orc_group_costs;
 *   - the integer program of Sec. 2.1 (maximise sum c subject to sum d <=
 *     budget, one configuration per group) -> orc_select_bruteforce,
 *     orc_select_bnb (plain depth-first search), orc_select_dp_integer (the
 *     textbook dynamic program, for integer-valued d);
 *   - budget tau^2 E[g^2] (Sec. 2.1; E[g^2] is the mean-square loss of
 *     Algorithm 1 step 2) -> orc_budget_from_tau.
 *   - The paper only models the quantisation error; the measured error term
 *     D_f = sum_k (g_k * (Q_f(z_k) - z_k))^2 realises the same expectation
 *     E[g~^2] = sum_k g_k^2 E[z~_k^2] with the actual FP8 rounding.  The FP8
 *     formats (E4M3: 4 exponent / 3 mantissa bits as in Sec. 3.1, finite
 *     maximum 448; E5M2: maximum 57344), per-tensor amax scaling and
 *     round-to-nearest-even saturating cast are readings, listed in the design
 *     notes of the repository.
 *
 * Parity pins (see tests/test_oracle_*.py): the FP8 grid against its closed
 * form, encode against a brute-force nearest-grid-point search, zero error for
 * on-grid tensors, the closed-form quantisation-noise variance ulp^2/12, the
 * Gaussian expectation of S, exact power-of-two scaling laws, pure-Python
 * rational-arithmetic re-computation on tiny inputs, and exhaustive
 * enumeration for the selection.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_FMT_BASE = 0, ORC_FMT_E4M3 = 1, ORC_FMT_E5M2 = 2 };

/* ------------------------------------------------------------------------- */
/* FP8 formats, from their definition: 1 sign bit, ebits exponent bits with a
 * bias, mbits mantissa bits, gradual underflow.  E4M3 has no infinity and one
 * NaN mantissa pattern (exponent field 15, mantissa 7), so its largest finite
 * value is 1.75 * 2^8 = 448.  E5M2 follows the IEEE layout: exponent field 31
 * is Inf/NaN and the largest finite value is 1.75 * 2^15 = 57344. */
typedef struct {
    int ebits, mbits, bias;
    int ieee_specials; /* 1: top exponent is Inf/NaN; 0: only E=max,M=max is NaN */
    double fmax;
} orc_fmt;

static int orc_get_fmt(int fmt, orc_fmt *o) {
    if (fmt == ORC_FMT_E4M3) {
        o->ebits = 4; o->mbits = 3; o->bias = 7; o->ieee_specials = 0; o->fmax = 448.0;
        return 0;
    }
    if (fmt == ORC_FMT_E5M2) {
        o->ebits = 5; o->mbits = 2; o->bias = 15; o->ieee_specials = 1; o->fmax = 57344.0;
        return 0;
    }
    return -1;
}

double orc_fmax(int fmt) {
    orc_fmt f;
    if (orc_get_fmt(fmt, &f)) return NAN;
    return f.fmax;
}

int orc_mantissa_bits(int fmt) {
    orc_fmt f;
    if (fmt == ORC_FMT_BASE) return 7; /* BF16 */
    if (orc_get_fmt(fmt, &f)) return -1;
    return f.mbits;
}

/* alpha_f = 2^(-2 m_f) / 12: variance of |z| 2^-m U[-1/2,1/2] divided by z^2
 * (Sec. 2.2, noise model). */
double orc_alpha(int mantissa_bits) {
    return ldexp(1.0, -2 * mantissa_bits) / 12.0;
}

/* Value of an 8-bit code. */
double orc_fp8_decode(int fmt, unsigned code) {
    orc_fmt f;
    if (orc_get_fmt(fmt, &f)) return NAN;
    int sign = (code >> 7) & 1;
    int E = (code >> f.mbits) & ((1 << f.ebits) - 1);
    int M = code & ((1 << f.mbits) - 1);
    int Emax = (1 << f.ebits) - 1;
    double v;
    if (f.ieee_specials && E == Emax) {
        v = (M == 0) ? INFINITY : NAN;
    } else if (!f.ieee_specials && E == Emax && M == (1 << f.mbits) - 1) {
        v = NAN;
    } else if (E == 0) {
        v = ldexp((double)M, 1 - f.bias - f.mbits);                 /* subnormal */
    } else {
        v = ldexp((double)((1 << f.mbits) + M), E - f.bias - f.mbits); /* normal */
    }
    return sign ? -v : v;
}

/* Round-to-nearest-even, saturate-to-finite cast of an fp32 value to a code.
 * The spacing of the grid around |y| is 2^(e-m) with e = floor(log2|y|),
 * never below the subnormal spacing 2^(1-bias-m); |y|/spacing is rounded to
 * an integer with ties to even, which is ties-to-even-code because adjacent
 * codes alternate parity of that integer.  Results above fmax (and Inf)
 * become +-fmax; the sign of zero is kept; NaN gives 0x7F. */
unsigned orc_fp8_encode(int fmt, float y) {
    orc_fmt f;
    if (orc_get_fmt(fmt, &f)) return 0xFFu;
    if (y != y) return 0x7Fu;
    unsigned sign = signbit(y) ? 0x80u : 0u;
    double a = fabs((double)y);
    int emin = 1 - f.bias;
    unsigned mag;
    double n;
    int e;
    if (a == 0.0) return sign;
    if (isinf(a)) {
        a = f.fmax;
    }
    {
        int ex;
        (void)frexp(a, &ex); /* a = frac * 2^ex, frac in [0.5,1) -> floor(log2 a) = ex-1 */
        e = ex - 1;
    }
    if (e < emin) e = emin;
    /* a / 2^(e-m) is exact (power-of-two scaling of a double holding an fp32). */
    n = nearbyint(ldexp(a, f.mbits - e)); /* default rounding mode: ties to even */
    if (n >= (double)(2 << f.mbits)) {    /* rounded up into the next binade */
        n = (double)(1 << f.mbits);
        e += 1;
    }
    if (ldexp(n, e - f.mbits) > f.fmax) {
        /* saturate: code of fmax */
        double fm = f.fmax;
        int ex;
        (void)frexp(fm, &ex);
        e = ex - 1;
        n = ldexp(fm, f.mbits - e);
    }
    if (n < (double)(1 << f.mbits)) {
        mag = (unsigned)n; /* subnormal (e == emin): exponent field 0 */
    } else {
        mag = ((unsigned)(e + f.bias) << f.mbits) | ((unsigned)n - (1u << f.mbits));
    }
    return sign | mag;
}

/* ------------------------------------------------------------------------- */
/* element access: fp32 or bf16 (upper 16 bits of an fp32) -> exact double   */
static inline float orc_load_f(int dtype, const void *p, long long k) {
    if (dtype == ORC_F32) return ((const float *)p)[k];
    uint32_t b = (uint32_t)((const uint16_t *)p)[k] << 16;
    float f;
    memcpy(&f, &b, 4);
    return f;
}

/* Step 1: amax_t = max_k |z_k| over the whole tensor.  NaN makes the result
 * NaN (a contract violation the library reports as an error). */
float orc_amax(int dtype, const void *values, long long n) {
    float m = 0.0f;
    int saw_nan = 0;
    for (long long k = 0; k < n; ++k) {
        float a = fabsf(orc_load_f(dtype, values, k));
        if (a != a) saw_nan = 1;
        if (a > m) m = a;
    }
    return saw_nan ? NAN : m;
}

/* Step 2: scale = fl32(amax / fmax), inv_scale = fl32(fmax / amax).  The
 * quotient of two fp32 values taken in double and rounded once to fp32 is the
 * IEEE fp32 quotient.  amax = 0, or an amax so small that fmax/amax is not a
 * finite fp32, gives the neutral pair (1, 1). */
void orc_scales(int fmt, float amax, float *scale, float *inv_scale) {
    double fmax = orc_fmax(fmt);
    float s = 1.0f, inv = 1.0f;
    if (amax > 0.0f) {
        float i = (float)(fmax / (double)amax);
        if (isfinite(i)) {
            inv = i;
            s = (float)((double)amax / fmax);
        }
    }
    *scale = s;
    *inv_scale = inv;
}

/* Power-of-two scaling: the smallest power of two p with fmax * p >= amax, so
 * that nothing saturates and z * (1/p) is exact; inv_scale = 1/p.  The neutral
 * pair (1, 1) when amax = 0 or p (or 1/p) is not a normal fp32. */
void orc_scales_pow2(int fmt, float amax, float *scale, float *inv_scale) {
    double fmax = orc_fmax(fmt);
    *scale = 1.0f;
    *inv_scale = 1.0f;
    if (!(amax > 0.0f) || isinf(amax)) return;
    int k = -200;
    while (ldexp(fmax, k) < (double)amax) ++k; /* plain search: exact comparisons in double */
    if (k < -126 || k > 126) return;
    *scale = (float)ldexp(1.0, k);
    *inv_scale = (float)ldexp(1.0, -k);
}

/* Step 3 (codes only): q_k = encode_f( fl32( z_k * inv_scale ) ). */
void orc_codes(int dtype, const void *values, long long n, int fmt, float inv_scale,
               unsigned char *codes) {
    for (long long k = 0; k < n; ++k) {
        double z = (double)orc_load_f(dtype, values, k);
        float y = (float)(z * (double)inv_scale); /* exact product, one rounding */
        codes[k] = (unsigned char)orc_fp8_encode(fmt, y);
    }
}

/* Storing an fp32 value as bf16: round to nearest, ties to even, on the upper
 * 16 bits (finite inputs only). */
static inline uint16_t orc_f32_to_bf16(float f) {
    uint32_t b;
    memcpy(&b, &f, 4);
    uint32_t lsb = (b >> 16) & 1u;
    b += 0x7FFFu + lsb;
    return (uint16_t)(b >> 16);
}

/* The quantised operand itself, z^ = z + z~ (Sec. 2.2): z^_k = decode_f(q_k) * scale
 * evaluated as one fp32 product (the exact product rounded once), then stored
 * in the operand's own type (fp32 as is, bf16 by round-to-nearest-even).  This
 * is what a model run "in format f" feeds to the layer. */
void orc_fake_quant(int dtype, const void *values, long long n, int fmt, float scale,
                    float inv_scale, void *out) {
    for (long long k = 0; k < n; ++k) {
        double z = (double)orc_load_f(dtype, values, k);
        float y = (float)(z * (double)inv_scale);
        unsigned q = orc_fp8_encode(fmt, y);
        float zh = (float)(orc_fp8_decode(fmt, q) * (double)scale);
        if (dtype == ORC_F32) ((float *)out)[k] = zh;
        else ((uint16_t *)out)[k] = orc_f32_to_bf16(zh);
    }
}

/* Steps 3-4 for one segment (one tensor, one sample): over its n elements
 *   S    = sum_k (z_k g_k)^2                     (the paper's sensitivity term)
 *   D_f  = sum_k (g_k e_k)^2,  e_k = decode_f(q_k) * scale_f - z_k
 * for each of the nfmt low-precision formats.  out = [S, D_0, ..., D_{nfmt-1}].
 * Plain left-to-right double accumulation. */
void orc_score_segment(int dtype, const void *values, const void *grads, long long n,
                       int nfmt, const int *fmts, const float *scales,
                       const float *inv_scales, double *out) {
    double S = 0.0;
    double D[8];
    if (nfmt > 8) nfmt = 8;
    for (int f = 0; f < nfmt; ++f) D[f] = 0.0;
    for (long long k = 0; k < n; ++k) {
        double z = (double)orc_load_f(dtype, values, k);
        double g = (double)orc_load_f(dtype, grads, k);
        double zg = z * g;
        S += zg * zg;
        for (int f = 0; f < nfmt; ++f) {
            float y = (float)(z * (double)inv_scales[f]);
            unsigned q = orc_fp8_encode(fmts[f], y);
            double zh = orc_fp8_decode(fmts[f], q) * (double)scales[f];
            double e = zh - z;
            double ge = g * e;
            D[f] += ge * ge;
        }
    }
    out[0] = S;
    for (int f = 0; f < nfmt; ++f) out[1 + f] = D[f];
}

/* Step 5, one layer.  seg0 / seg1: [R][1+nlow] doubles for operand 0 / 1 (the
 * output of orc_score_segment per sample).  F = 1 + nlow formats, format 0 is
 * the high-precision baseline whose loss-MSE contribution is 0 by definition
 * of the loss MSE relative to the unquantised loss (Sec. 2.1).
 *   s_r[r]        = S(op0,r) + S(op1,r)       (extended input holds both)
 *   s_mean        = (1/R) sum_r s_r
 *   d_model[f]    = alpha_f * s_mean ; d_model[0] = 0
 *   d_meas_r[r,f] = D_f(op0,r) + D_f(op1,r) ; column 0 = 0
 *   d_meas[f]     = (1/R) sum_r d_meas_r[r,f]
 * mbits[f] = mantissa bits of format f (f >= 1). */
void orc_layer_combine(int R, int F, const int *mbits, const double *seg0, const double *seg1,
                       double *s_r, double *s_mean, double *d_meas_r, double *d_model,
                       double *d_meas) {
    int nacc = F; /* 1 + nlow */
    double acc = 0.0;
    for (int r = 0; r < R; ++r) {
        s_r[r] = seg0[r * nacc] + seg1[r * nacc];
        acc += s_r[r];
    }
    *s_mean = acc / (double)R;
    d_model[0] = 0.0;
    d_meas[0] = 0.0;
    for (int f = 1; f < F; ++f) {
        double a = 0.0;
        d_model[f] = orc_alpha(mbits[f]) * (*s_mean);
        for (int r = 0; r < R; ++r) {
            double v = seg0[r * nacc + f] + seg1[r * nacc + f];
            d_meas_r[r * F + f] = v;
            a += v;
        }
        d_meas[f] = a / (double)R;
    }
    for (int r = 0; r < R; ++r) d_meas_r[r * F] = 0.0;
}

/* Step 6: d_{j,p} = sum_{l=0}^{Lj-1} d_layer[ layer_ids[l] ][ Q[l + Lj*p] ],
 * left fold in l.  d_layer is [L][F]. */
void orc_group_costs(int Lj, int Pj, int F, const int *layer_ids, const unsigned char *Q,
                     const double *d_layer, double *d_out) {
    for (int p = 0; p < Pj; ++p) {
        double d = 0.0;
        for (int l = 0; l < Lj; ++l) d += d_layer[(long long)layer_ids[l] * F + Q[l + Lj * p]];
        d_out[p] = d;
    }
}

/* budget = tau^2 * (1/R) sum_r (g^r)^2. */
double orc_budget_from_tau(double tau, const double *losses, int R) {
    double a = 0.0;
    for (int r = 0; r < R; ++r) a += losses[r] * losses[r];
    return tau * tau * (a / (double)R);
}

/* ------------------------------------------------------------------------- */
/* Selection.  Tables are flattened: group j owns entries off[j]..off[j]+P[j]-1
 * of c[] and d[].  An assignment p = (p_0..p_{J-1}) has
 *   d(p) = (((0 + d_{0,p0}) + d_{1,p1}) + ...),  c(p) likewise (left folds),
 * is feasible iff d(p) <= budget, and assignments are ordered: larger c, then
 * smaller d, then lexicographically smaller p.  Returns 0 and the best
 * feasible assignment, or 1 if none is feasible. */
static int orc_better(int J, double c, double d, const int *p, double bc, double bd,
                      const int *bp, int have_best) {
    if (!have_best) return 1;
    if (c != bc) return c > bc;
    if (d != bd) return d < bd;
    for (int j = 0; j < J; ++j)
        if (p[j] != bp[j]) return p[j] < bp[j];
    return 0;
}

int orc_select_bruteforce(int J, const int *P, const long long *off, const double *c,
                          const double *d, double budget, int *p_out, double *c_out,
                          double *d_out) {
    int *p = (int *)calloc((size_t)(J > 0 ? J : 1), sizeof(int));
    int have = 0;
    double bc = 0.0, bd = 0.0;
    for (;;) {
        double cs = 0.0, ds = 0.0;
        for (int j = 0; j < J; ++j) {
            ds += d[off[j] + p[j]];
            cs += c[off[j] + p[j]];
        }
        if (ds <= budget && orc_better(J, cs, ds, p, bc, bd, p_out, have)) {
            have = 1; bc = cs; bd = ds;
            memcpy(p_out, p, sizeof(int) * (size_t)J);
        }
        /* odometer, p_0 slowest */
        int j = J - 1;
        while (j >= 0) {
            if (++p[j] < P[j]) break;
            p[j] = 0;
            --j;
        }
        if (j < 0) break;
    }
    free(p);
    if (!have) return 1;
    *c_out = bc; *d_out = bd;
    return 0;
}

/* Depth-first branch and bound for problems too large to enumerate (Sec. 2.1,
 * the integer program).  Groups are taken in order j = 0..J-1 and configurations
 * in order p = 0..P_j-1, so leaves are met in lexicographic order and carry
 * exactly the left-fold sums of the enumeration.  Below a node with partial
 * sums (cs, ds) over groups < j, a leaf's sums are those partial sums with one
 * term per remaining group folded on.  Floating-point addition is monotone in
 * each argument, so folding on, group by group, the smallest d of each
 * remaining group gives a value no leaf below can undercut, and folding on the
 * largest c of each gives a value no leaf below can exceed.  A node is cut
 *   (i)  when that smallest reachable d is above the budget, or
 *   (ii) when that largest reachable c is strictly below the best c so far;
 * nothing else is cut and no tolerance is involved, so the result is the
 * enumeration's.  This is slow when the budget admits many assignments; the
 * tests use it where it is not (tight budgets, moderate J) and
 * orc_select_dp_integer for large J. */
typedef struct {
    int J;
    const int *P;
    const long long *off;
    const double *c, *d;
    double budget;
    double *min_d, *max_c;   /* per group */
    int *p, *bp; int have; double bc, bd;
    long long nodes, node_limit;
} orc_bnb;

static void orc_bnb_rec(orc_bnb *s, int j, double cs, double ds) {
    if (s->nodes++ > s->node_limit) return;
    if (j == s->J) {
        if (ds <= s->budget && orc_better(s->J, cs, ds, s->p, s->bc, s->bd, s->bp, s->have)) {
            s->have = 1; s->bc = cs; s->bd = ds;
            memcpy(s->bp, s->p, sizeof(int) * (size_t)s->J);
        }
        return;
    }
    {
        double lo_d = ds, hi_c = cs;
        for (int k = j; k < s->J; ++k) { lo_d += s->min_d[k]; hi_c += s->max_c[k]; }
        if (lo_d > s->budget) return;            /* (i)  */
        if (s->have && hi_c < s->bc) return;     /* (ii) */
    }
    for (int p = 0; p < s->P[j]; ++p) {
        s->p[j] = p;
        orc_bnb_rec(s, j + 1, cs + s->c[s->off[j] + p], ds + s->d[s->off[j] + p]);
    }
}

/* returns 0 ok, 1 infeasible, 2 node limit hit (result not proven optimal) */
int orc_select_bnb(int J, const int *P, const long long *off, const double *c, const double *d,
                   double budget, long long node_limit, int *p_out, double *c_out,
                   double *d_out) {
    orc_bnb s;
    int rc;
    memset(&s, 0, sizeof s);
    s.J = J; s.P = P; s.off = off; s.c = c; s.d = d; s.budget = budget;
    s.node_limit = node_limit > 0 ? node_limit : 2000000000LL;
    s.min_d = (double *)calloc((size_t)J + 1, sizeof(double));
    s.max_c = (double *)calloc((size_t)J + 1, sizeof(double));
    s.p = (int *)calloc((size_t)J + 1, sizeof(int));
    s.bp = (int *)calloc((size_t)J + 1, sizeof(int));
    for (int j = 0; j < J; ++j) {
        s.min_d[j] = d[off[j]]; s.max_c[j] = c[off[j]];
        for (int p = 1; p < P[j]; ++p) {
            if (d[off[j] + p] < s.min_d[j]) s.min_d[j] = d[off[j] + p];
            if (c[off[j] + p] > s.max_c[j]) s.max_c[j] = c[off[j] + p];
        }
    }
    orc_bnb_rec(&s, 0, 0.0, 0.0);
    if (s.nodes > s.node_limit) rc = 2;
    else rc = s.have ? 0 : 1;
    if (s.have) {
        memcpy(p_out, s.bp, sizeof(int) * (size_t)J);
        *c_out = s.bc; *d_out = s.bd;
    }
    free(s.min_d); free(s.max_c); free(s.p); free(s.bp);
    return rc;
}

/* The same integer program when every d is a non-negative integer: the
 * textbook dynamic program of the multiple-choice knapsack over the integer
 * budget.  best[w] after group j = the largest left-fold c over assignments of
 * groups 0..j whose d sums to exactly w (integers: that sum has no rounding and
 * no order).  best[w] + c_{j,p} is the left fold of the extended assignment,
 * and because floating-point addition is monotone the largest prefix value
 * gives the largest extended value, so the table holds true maxima of left
 * folds.  Answer: the largest best[w] over w <= budget, the smallest such w,
 * and one assignment that attains them (which one, among several with the same
 * (c, d), is not specified).  Returns 0 ok, 1 infeasible, 3 too large. */
int orc_select_dp_integer(int J, const int *P, const long long *off, const double *c,
                          const long long *d, long long budget, int *p_out, double *c_out,
                          long long *d_out) {
    if (budget < 0) return 1;
    if (budget > 50000000LL || (double)(budget + 1) * (double)(J + 1) > 4e8) return 3;
    const size_t W = (size_t)budget + 1;
    double *best = (double *)malloc(W * sizeof(double));
    double *next = (double *)malloc(W * sizeof(double));
    char *ok = (char *)calloc(W, 1), *nok = (char *)calloc(W, 1);
    int *choice = (int *)malloc(W * (size_t)(J > 0 ? J : 1) * sizeof(int)); /* [j][w]: p that gave next[w] */
    ok[0] = 1; best[0] = 0.0;
    for (int j = 0; j < J; ++j) {
        memset(nok, 0, W);
        for (size_t w = 0; w < W; ++w) {
            if (!ok[w]) continue;
            for (int p = 0; p < P[j]; ++p) {
                long long dv = d[off[j] + p];
                if (dv < 0 || (long long)w + dv > budget) continue;
                size_t w2 = w + (size_t)dv;
                double v = best[w] + c[off[j] + p];
                if (!nok[w2] || v > next[w2]) { nok[w2] = 1; next[w2] = v; choice[(size_t)j * W + w2] = p; }
            }
        }
        { double *t = best; best = next; next = t; char *u = ok; ok = nok; nok = u; }
    }
    int have = 0; size_t bw = 0;
    for (size_t w = 0; w < W; ++w)
        if (ok[w] && (!have || best[w] > best[bw])) { have = 1; bw = w; }
    if (have) {
        *c_out = best[bw]; *d_out = (long long)bw;
        size_t w = bw;
        for (int j = J - 1; j >= 0; --j) {
            int p = choice[(size_t)j * W + w];
            p_out[j] = p;
            w -= (size_t)d[off[j] + p];
        }
    }
    free(best); free(next); free(ok); free(nok); free(choice);
    return have ? 0 : 1;
}
