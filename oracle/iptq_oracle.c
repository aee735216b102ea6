/*
 * CPU oracle for the integer-only non-linear path of IPTQ-ViT (see the header).
 * TEST INFRASTRUCTURE ONLY: plain C, int64 intermediates, one element at a
 * time, in the paper's order and notation.  No blocking, fusion or SIMD.
 * OpenMP is used only to spread independent rows / problems over host cores.
 */
#include "iptq_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------- small integer helpers -------------------------------------- */

/* floor(x / 2^k): arithmetic shift written out so that it does not depend on
 * the compiler's treatment of ">>" on negative values. */
static int64_t fshr(int64_t x, int k)
{
    if (k <= 0) return x;
    if (k >= 63) return x < 0 ? -1 : 0;
    int64_t d = (int64_t)1 << k;
    int64_t q = x / d;            /* truncates toward zero */
    if ((x % d) != 0 && x < 0) q -= 1;
    return q;
}

/* position of the top set bit + 1 (bitlen(0) = 0) */
static int bitlen_u64(uint64_t v)
{
    int n = 0;
    while (v) { n++; v >>= 1; }
    return n;
}

static int64_t clamp64(int64_t v, int64_t lo, int64_t hi) { return v < lo ? lo : (v > hi ? hi : v); }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------- R: dyadic requantisation ----------------------------------- */
/*
 * The paper has no requantisation formula; integer-only pipelines it builds on
 * (Sec. 2) use a dyadic multiplier.  reading: R(y) = clamp(((hi32(y*mult) +
 * 2^(shift-1)) >> shift) + zp, qmin, qmax), hi32(p) = floor(p / 2^32) of the
 * exact 64-bit product.  The double rounding (floor, then round-half-up) is
 * the definition.
 */
int oracle_requant_prepare(double ratio, int32_t zp, int32_t qmin, int32_t qmax, oracle_requant_t* out)
{
    if (!out) return ORACLE_ERR_ARG;
    if (!(ratio > 0.0) || !(ratio < 0.25)) return ORACLE_ERR_RANGE;
    int ex;
    double m = frexp(ratio, &ex);          /* ratio = m * 2^ex, m in [0.5, 1) */
    (void)m;
    int e = ex - 1;                        /* floor(log2 ratio) */
    double scaled = ldexp(ratio, 30 - e);  /* in [2^30, 2^31) */
    int64_t mult = (int64_t)floor(scaled + 0.5);
    if (mult >= ((int64_t)1 << 31)) { mult = (int64_t)1 << 30; e += 1; }
    int shift = -e - 2;
    if (shift < 1 || shift > 31) return ORACLE_ERR_RANGE;
    out->mult = (int32_t)mult;
    out->shift = shift;
    out->zp = zp;
    out->qmin = qmin;
    out->qmax = qmax;
    return ORACLE_OK;
}

static int64_t requant_noclamp(int64_t y, int64_t mult, int shift)
{
    int64_t hi = fshr(y * mult, 32);
    return fshr(hi + ((int64_t)1 << (shift - 1)), shift);
}

int32_t oracle_requant(int32_t y, const oracle_requant_t* rq)
{
    int64_t v = requant_noclamp(y, rq->mult, rq->shift) + rq->zp;
    return (int32_t)clamp64(v, rq->qmin, rq->qmax);
}

/* ---------- Softmax (Sec. 3.4, Eqs. (6)-(15)) --------------------------- */

int oracle_softmax_prepare(double in_scale, int row_len, int out_bits, int variant, oracle_softmax_consts_t* out)
{
    if (!out) return ORACLE_ERR_ARG;
    if (row_len < 1 || out_bits < 4 || out_bits > 8) return ORACLE_ERR_ARG;
    if (variant != ORACLE_SM_BITEXP && variant != ORACLE_SM_SHIFTMAX && variant != ORACLE_SM_POLY &&
        variant != ORACLE_SM_LOG2) return ORACLE_ERR_ARG;
    if (variant == ORACLE_SM_LOG2 && out_bits != 4) return ORACLE_ERR_ARG;   /* 4-bit log2 codes */
    if (!(in_scale > 0.0)) return ORACLE_ERR_RANGE;
    memset(out, 0, sizeof(*out));
    /* Eq. (14): the integer that stands for 1.0 is floor(1 / S_delta). */
    double inv = floor(1.0 / in_scale);
    if (!(inv >= 8.0) || !(inv < 16777216.0)) return ORACLE_ERR_RANGE;   /* 8 <= x0 < 2^24 */
    int64_t x0 = (int64_t)inv;
    out->variant = variant;
    out->out_bits = out_bits;
    out->row_len = row_len;
    out->x0 = (int32_t)x0;
    /* reading: beyond 34 * x0 the exponential is zero anyway; clamping keeps every step in 32 bits. */
    out->dcap = (int32_t)(34 * x0);

    int64_t unit;  /* value of the exponential at distance 0 */
    if (variant == ORACLE_SM_POLY || variant == ORACLE_SM_LOG2) {
        /* reading: second-order exp polynomial of the cited polynomial method,
         * exp(p) ~ a (p + b)^2 + c on p in (-ln2, 0]; a is absorbed in the scale. */
        const double a = 0.3585, b = 1.353, cc = 0.344;
        double qln2 = floor(log(2.0) / in_scale);
        double qb = floor(b / in_scale);
        double qc = floor(cc / (a * in_scale * in_scale));
        if (qln2 < 1.0 || qb >= 32768.0 || qc >= 1073741824.0) return ORACLE_ERR_RANGE;
        out->qln2 = (int32_t)qln2;
        out->qb = (int32_t)qb;
        out->qc = (int32_t)qc;
        int64_t E0 = (int64_t)qb * (int64_t)qb + (int64_t)qc;
        int w = bitlen_u64((uint64_t)E0);
        out->norm_l = w <= 14 ? 14 - w : 0;     /* bring E0 into [2^13, 2^14) */
        out->norm_r = w > 14 ? w - 14 : 0;
        unit = fshr(E0 << out->norm_l, out->norm_r);
        out->nsh = 0;
    } else {
        /* reading: Eq. (9) needs a left shift so that ">> q" keeps bits: x0 << N in [2^13, 2^14) when x0 < 2^13. */
        int w = bitlen_u64((uint64_t)x0);
        out->nsh = w < 14 ? 14 - w : 0;
        unit = x0 << out->nsh;
    }
    /* the row sum must fit 31 bits (contract of the 32-bit implementations) */
    if ((int64_t)row_len * unit >= ((int64_t)1 << 31)) return ORACLE_ERR_RANGE;
    /* reading: "M is a large integer" (Eq. (15)): keep >= 16 significant bits in floor(2^M / sum). */
    int wsum = bitlen_u64((uint64_t)((int64_t)row_len * unit));
    int M = 31 + (wsum > 15 ? wsum - 15 : 0);
    if (M > 40) M = 40;
    out->M = M;
    return ORACLE_OK;
}

/* Phi of Eq. (13): ln2 ~ (0.1011)b, three separate floor shifts of the (negative) operand. */
static int64_t phi_bitexp(int64_t u) { return fshr(u, 1) + fshr(u, 3) + fshr(u, 4); }

int64_t oracle_softmax_exp(int64_t d, const oracle_softmax_consts_t* c)
{
    int64_t x0 = c->x0;
    if (c->variant == ORACLE_SM_POLY || c->variant == ORACLE_SM_LOG2) {
        int64_t z = d / c->qln2;                       /* octave */
        int64_t p = -(d - z * c->qln2);                /* in (-qln2, 0] */
        int64_t poly = (p + c->qb) * (p + c->qb) + c->qc;
        int64_t e = fshr(poly << c->norm_l, c->norm_r);
        return z > 31 ? 0 : fshr(e, (int)z);
    }
    int64_t Qd = -d;                                   /* Q_delta <= 0 */
    int64_t Qp = Qd + fshr(Qd, 1) - fshr(Qd, 4);       /* Eq. (7): * log2(e) ~ 1 + 1/2 - 1/16 */
    int64_t P = -Qp;                                   /* >= 0 */
    int64_t q = P / x0;                                /* Eq. (8): integer octave */
    int64_t r = P - q * x0;                            /* fraction, in [0, x0) */
    int64_t base;
    if (c->variant == ORACLE_SM_BITEXP)
        base = phi_bitexp(-r) + x0;                    /* Eqs. (13)-(14) */
    else
        base = fshr(-r, 1) + x0;                       /* Eq. (10): 1 + x/2 */
    return q > 31 ? 0 : fshr(base << c->nsh, (int)q);  /* Eq. (9) */
}

void oracle_softmax_row(const int64_t* s, const uint8_t* mask, int n, const oracle_softmax_consts_t* c, uint8_t* p)
{
    /* Eq. (6): subtract the row maximum (over unmasked entries). */
    int have = 0;
    int64_t mx = 0;
    for (int j = 0; j < n; j++) {
        if (mask && mask[j]) continue;
        if (!have || s[j] > mx) { mx = s[j]; have = 1; }
    }
    int64_t* e = (int64_t*)malloc(sizeof(int64_t) * (size_t)n);
    int64_t sum = 0;
    for (int j = 0; j < n; j++) {
        if (mask && mask[j]) { e[j] = 0; continue; }
        int64_t d = mx - s[j];
        if (d > c->dcap) d = c->dcap;
        e[j] = oracle_softmax_exp(d, c);
        sum += e[j];
    }
    if (c->variant == ORACLE_SM_LOG2) {
        /* reading (the "logarithm" candidate of Sec. 3.2 is named, not defined): the probability is rounded to a
         * power of two, p = 2^-code, code = round(log2(round(sum / e))) kept in 4 bits; smaller probabilities,
         * and entries whose exponential is 0, are exactly 0 (code ORACLE_LOG2_ZERO).  Integer form of the
         * rounded logarithm: the position of the leading one, plus one when the bit below it is set. */
        for (int j = 0; j < n; j++) {
            if (e[j] == 0) { p[j] = ORACLE_LOG2_ZERO; continue; }
            int64_t r = (2 * sum + e[j]) / (2 * e[j]);             /* round(sum / e), halves up; >= 1 */
            int fl = bitlen_u64((uint64_t)r) - 1;                  /* floor(log2 r) */
            int code = fl + ((fl >= 1 && ((r >> (fl - 1)) & 1)) ? 1 : 0);
            p[j] = code > 15 ? ORACLE_LOG2_ZERO : (uint8_t)code;
        }
        free(e);
        return;
    }
    /* Eq. (15): IntDiv. */
    int64_t f = have ? (((int64_t)1 << c->M) / sum) : 0;
    int sh = c->M - (c->out_bits - 1);
    for (int j = 0; j < n; j++) p[j] = (uint8_t)fshr(f * e[j], sh);
    free(e);
}

int oracle_softmax(const int32_t* scores, uint8_t* probs, int64_t rows, int row_len,
                   const int32_t* bias, int64_t bias_period, const oracle_softmax_consts_t* c)
{
    if (!scores || !probs || !c) return ORACLE_ERR_ARG;
    if (bias && bias_period < 1) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; i++) {
        int64_t* s = (int64_t*)malloc(sizeof(int64_t) * (size_t)row_len);
        const int32_t* brow = bias ? bias + (i % bias_period) * row_len : NULL;
        for (int j = 0; j < row_len; j++) s[j] = (int64_t)scores[i * row_len + j] + (brow ? brow[j] : 0);
        oracle_softmax_row(s, NULL, row_len, c, probs + i * row_len);
        free(s);
    }
    return ORACLE_OK;
}

/* ---------- GELU (Sec. 3.3, Eqs. (1)-(5)) ------------------------------- */

static int gelu_prepare_impl(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                             int variant, double A, double Bf, oracle_gelu_consts_t* out);

int oracle_gelu_prepare(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                        int variant, oracle_gelu_consts_t* out)
{
    /* Eq. (3): a = -0.019913, b = -2.698088 (quartic); the second-order
     * erf polynomial of the cited prior work has a = -0.2888, b = -1.769. */
    const double A = (variant == ORACLE_GELU_POLY4) ? 0.019913 : 0.2888;
    const double Bf = (variant == ORACLE_GELU_POLY4) ? 2.698088 : 1.769;
    return gelu_prepare_impl(in_scale, in_bits, out_scale, out_zp, out_bits, variant, A, Bf, out);
}

/* Quartic polynomial with coefficients refitted to the data range (Eq. (4)): a < 0, b < 0 as in Eq. (3). */
int oracle_gelu_prepare_coeffs(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                               double a, double b, oracle_gelu_consts_t* out)
{
    if (!(a < 0.0) || !(b < 0.0)) return ORACLE_ERR_RANGE;
    return gelu_prepare_impl(in_scale, in_bits, out_scale, out_zp, out_bits, ORACLE_GELU_POLY4, -a, -b, out);
}

static int gelu_prepare_impl(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                             int variant, double A, double Bf, oracle_gelu_consts_t* out)
{
    if (!out) return ORACLE_ERR_ARG;
    if (in_bits < 8 || in_bits > 16 || out_bits < 4 || out_bits > 8) return ORACLE_ERR_ARG;
    if (!(in_scale > 0.0) || !(out_scale > 0.0)) return ORACLE_ERR_RANGE;
    memset(out, 0, sizeof(*out));
    out->variant = variant;
    out->in_bits = in_bits;
    double Sy;
    if (variant == ORACLE_GELU_POLY4 || variant == ORACLE_GELU_POLY2) {
        double Sp = in_scale / sqrt(2.0);              /* scale of x / sqrt(2), Eq. (5) */
        double Bqd = floor(Bf / Sp);
        if (!(Bqd >= 1.0) || !(Bqd < 32768.0)) return ORACLE_ERR_RANGE;
        int64_t Bq = (int64_t)Bqd;
        int nb = bitlen_u64((uint64_t)Bq);
        int sh2 = 2 * nb - 15; if (sh2 < 0) sh2 = 0;
        double Cd;
        if (variant == ORACLE_GELU_POLY4)
            Cd = floor(1.0 / (A * Sp * Sp * Sp * Sp) / ldexp(1.0, 2 * sh2));
        else
            Cd = floor(1.0 / (A * Sp * Sp) / ldexp(1.0, sh2));
        if (!(Cd >= 1.0) || !(Cd < 1073741824.0)) return ORACLE_ERR_RANGE;
        int64_t C = (int64_t)Cd;
        int gs = bitlen_u64((uint64_t)(2 * C)) + in_bits - 31; if (gs < 0) gs = 0;
        out->Bq = (int32_t)Bq; out->sh2 = sh2; out->C = (int32_t)C; out->gs = gs;
        Sy = in_scale * ldexp(1.0, gs) / (2.0 * (double)C);
    } else if (variant == ORACLE_GELU_SHIFT) {
        /* reading: x * sigmoid(1.702 x) with the shift exponential of Eqs. (7)-(10). */
        double inv = floor(1.0 / in_scale);
        if (!(inv >= 8.0) || !(inv < 16777216.0)) return ORACLE_ERR_RANGE;
        int64_t x0 = (int64_t)inv;
        int w = bitlen_u64((uint64_t)x0);
        out->x0 = (int32_t)x0;
        out->nsh = w < 14 ? 14 - w : 0;
        if (w > 14) return ORACLE_ERR_RANGE;           /* keeps D + e below 2^15 */
        out->dcap = (int32_t)(34 * x0);
        Sy = in_scale * ldexp(1.0, -15);
    } else {
        return ORACLE_ERR_ARG;
    }
    int32_t qmin = -(1 << (out_bits - 1)), qmax = (1 << (out_bits - 1)) - 1;
    return oracle_requant_prepare(Sy / out_scale, out_zp, qmin, qmax, &out->out);
}

double oracle_gelu_core_scale(double in_scale, const oracle_gelu_consts_t* c)
{
    if (c->variant == ORACLE_GELU_SHIFT) return in_scale * ldexp(1.0, -15);
    return in_scale * ldexp(1.0, c->gs) / (2.0 * (double)c->C);
}

int64_t oracle_gelu_core(int64_t x, const oracle_gelu_consts_t* c)
{
    int64_t lo = -((int64_t)1 << (c->in_bits - 1)), hi = ((int64_t)1 << (c->in_bits - 1)) - 1;
    x = clamp64(x, lo, hi);
    if (c->variant == ORACLE_GELU_SHIFT) {
        int64_t xp = x + fshr(x, 1) + fshr(x, 3) + fshr(x, 4);       /* ~1.702 x */
        int64_t d = xp < 0 ? -xp : xp;
        if (d > c->dcap) d = c->dcap;
        oracle_softmax_consts_t sc;
        memset(&sc, 0, sizeof(sc));
        sc.variant = ORACLE_SM_SHIFTMAX; sc.x0 = c->x0; sc.nsh = c->nsh;
        int64_t e = oracle_softmax_exp(d, &sc);                      /* exp(-|xp| S) */
        int64_t D = (int64_t)c->x0 << c->nsh;                        /* 1.0 */
        int64_t f = ((int64_t)1 << 31) / (D + e);                    /* IntDiv, M = 31 */
        int64_t num = xp >= 0 ? D : e;                               /* stable sigmoid */
        int64_t sig = fshr(f * num, 16);                             /* Q15 */
        return x * sig;
    }
    int64_t ax = x < 0 ? -x : x;
    int64_t m = ax < c->Bq ? ax : c->Bq;          /* clip(|x|, max = -b) */
    int64_t t = c->Bq - m;                        /* -(clip + b) >= 0 */
    int64_t t2 = fshr(t * t, c->sh2);             /* squared term, reused */
    int64_t pw = (c->variant == ORACLE_GELU_POLY4) ? t2 * t2 : t2;
    int64_t E = c->C - pw;                        /* a (.)^4 + 1 in units of 1/C */
    int64_t sg = x > 0 ? 1 : (x < 0 ? -1 : 0);
    int64_t G = sg * E + c->C;                    /* 1 + L(x / sqrt 2) */
    return x * fshr(G, c->gs);                    /* x/2 * [1 + L], Eq. (5); 1/2 is in the scale */
}

int oracle_gelu(const int32_t* x, int8_t* y, int64_t n, const oracle_gelu_consts_t* c)
{
    if (!x || !y || !c) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; i++) {
        int64_t core = oracle_gelu_core(x[i], c);
        y[i] = (int8_t)oracle_requant((int32_t)core, &c->out);
    }
    return ORACLE_OK;
}

/* ---------- LayerNorm (candidates named in Sec. 3.2; algorithm is a reading) */

int oracle_layernorm_prepare(int dim, const float* gamma, const float* beta, double out_scale, int out_zp,
                             int out_bits, int variant, int32_t* gamma_q, int32_t* beta_q, oracle_ln_consts_t* out)
{
    if (!gamma || !beta || !gamma_q || !beta_q || !out) return ORACLE_ERR_ARG;
    if (dim < 2 || dim > 3072 || out_bits < 4 || out_bits > 8) return ORACLE_ERR_ARG;
    if (variant < 0 || variant > 2) return ORACLE_ERR_ARG;
    if (!(out_scale > 0.0)) return ORACLE_ERR_RANGE;
    double gmax = 0.0;
    for (int c = 0; c < dim; c++) { double a = fabs((double)gamma[c]); if (a > gmax) gmax = a; }
    if (!(gmax > 0.0)) return ORACLE_ERR_RANGE;
    double Sg = gmax / 32767.0;                   /* one per-tensor scale for gamma */
    double Sb = ldexp(Sg, -10);                   /* normalised values are Q10 */
    double gq_max = 0.0, bq_max = 0.0;
    for (int c = 0; c < dim; c++) {
        double g = floor((double)gamma[c] / Sg + 0.5);
        double b = floor((double)beta[c] / Sb + 0.5);
        if (fabs(g) > gq_max) gq_max = fabs(g);
        if (fabs(b) > bq_max) bq_max = fabs(b);
        if (fabs(b) >= 1073741824.0) return ORACLE_ERR_RANGE;
        gamma_q[c] = (int32_t)g;
        beta_q[c] = (int32_t)b;
    }
    /* |n_c| <= 1.125 sqrt(D) 2^10, so n*gamma_q + beta_q must stay inside int32 */
    if (1.125 * sqrt((double)dim) * 1024.0 * gq_max + bq_max >= 2147483648.0) return ORACLE_ERR_RANGE;
    out->variant = variant;
    out->dim = dim;
    int32_t qmin = -(1 << (out_bits - 1)), qmax = (1 << (out_bits - 1)) - 1;
    return oracle_requant_prepare(Sb / out_scale, out_zp, qmin, qmax, &out->out);
}

uint64_t oracle_isqrt(uint64_t V, int variant)
{
    if (V == 0) return 0;
    int w = bitlen_u64(V);
    uint64_t r = (uint64_t)1 << ((w + 1) / 2);    /* 2^ceil(bitlen/2) >= sqrt(V) */
    if (variant == ORACLE_LN_SHIFT) {
        /* "bit-shifting": the same recurrence for a fixed 10 steps, halving by a shift, no convergence test */
        for (int it = 0; it < 10; it++) r = (r + V / r) >> 1;
        return r;
    }
    /* Newton to convergence: exactly floor(sqrt(V)) */
    for (;;) {
        uint64_t r1 = (r + V / r) >> 1;
        if (r1 >= r) return r;
        r = r1;
    }
}

static void layernorm_row(const int8_t* x, int8_t* y, int D, const int32_t* gq, const int32_t* bq,
                          const uint8_t* ptf, const oracle_ln_consts_t* c)
{
    int64_t s1 = 0, s2 = 0;
    for (int j = 0; j < D; j++) {
        int64_t xh = (int64_t)x[j] << (ptf ? ptf[j] : 0);     /* power-of-two factor per channel */
        s1 += xh; s2 += xh * xh;
    }
    int64_t V = (int64_t)D * s2 - s1 * s1;                    /* D^2 * variance, exact */
    uint64_t r = oracle_isqrt((uint64_t)V, c->variant);       /* D * std */
    int64_t F = r ? (int64_t)((((uint64_t)1) << 40) / r) : 0;
    for (int j = 0; j < D; j++) {
        int64_t xh = (int64_t)x[j] << (ptf ? ptf[j] : 0);
        int64_t u = (int64_t)D * xh - s1;                     /* D * (x - mean), exact */
        int64_t n = r ? fshr(u * F, 30) : 0;                  /* (x - mean) / std in Q10 */
        int64_t v = n * gq[j] + bq[j];
        y[j] = (int8_t)oracle_requant((int32_t)v, &c->out);
    }
}

int oracle_layernorm(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gamma_q,
                     const int32_t* beta_q, const uint8_t* ptf_shift, const oracle_ln_consts_t* c)
{
    if (!x || !y || !gamma_q || !beta_q || !c) return ORACLE_ERR_ARG;
    if (dim != c->dim) return ORACLE_ERR_ARG;
    if (c->variant != ORACLE_LN_PTF) ptf_shift = NULL;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; i++)
        layernorm_row(x + i * dim, y + i * dim, dim, gamma_q, beta_q, ptf_shift, c);
    return ORACLE_OK;
}

/* ---------- integer GEMM carriers -------------------------------------- */

/* reading: int4 weights are two's complement nibbles, element k of a row in
 * byte k/2, even k in the low nibble. */
static int64_t weight_at(const void* w, int w_bits, int64_t row, int K, int k)
{
    if (w_bits == 8) return ((const int8_t*)w)[row * K + k];
    uint8_t byte = ((const uint8_t*)w)[row * (K / 2) + k / 2];
    int v = (k & 1) ? (byte >> 4) : (byte & 15);
    return v >= 8 ? v - 16 : v;
}

int oracle_linear(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                  const int8_t* shift, int32_t out_zp, const int8_t* residual, const oracle_requant_t* residual_rq,
                  int8_t* y, int64_t M, int N, int K)
{
    return oracle_linear_bits(x, w, w_bits, bias, mult, shift, out_zp, residual, residual_rq, y, M, N, K, 8);
}

/* The same layer with out_bits-wide activations (W6A6 setting): the output is clamped to
 * [-2^(out_bits-1), 2^(out_bits-1) - 1] instead of the int8 range. */
int oracle_linear_bits(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                       const int8_t* shift, int32_t out_zp, const int8_t* residual,
                       const oracle_requant_t* residual_rq, int8_t* y, int64_t M, int N, int K, int out_bits)
{
    if (!x || !w || !mult || !shift || !y) return ORACLE_ERR_ARG;
    if (out_bits < 4 || out_bits > 8) return ORACLE_ERR_ARG;
    const int64_t qmin = -((int64_t)1 << (out_bits - 1)), qmax = ((int64_t)1 << (out_bits - 1)) - 1;
    if (w_bits != 8 && w_bits != 4) return ORACLE_ERR_ARG;
    if (residual && !residual_rq) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; m++) {
        for (int n = 0; n < N; n++) {
            int64_t acc = bias ? bias[n] : 0;
            for (int k = 0; k < K; k++) acc += (int64_t)x[m * K + k] * weight_at(w, w_bits, n, K, k);
            int64_t v = requant_noclamp(acc, mult[n], shift[n]);
            if (residual) {
                /* the 8-bit residual is widened by 2^16 so that its ratio is < 1/4 */
                int64_t rr = ((int64_t)residual[m * N + n] - residual_rq->zp) << 16;
                v += requant_noclamp(rr, residual_rq->mult, residual_rq->shift);
            }
            y[m * N + n] = (int8_t)clamp64(v + out_zp, qmin, qmax);
        }
    }
    return ORACLE_OK;
}

int oracle_attention_strided(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H, int N,
                             int dh, int64_t tok_stride, int64_t head_stride, int64_t batch_stride,
                             const int32_t* bias, const uint8_t* mask_id, const oracle_softmax_consts_t* sc,
                             const oracle_requant_t* out_rq)
{
    if (!q || !k || !v || !out || !sc || !out_rq) return ORACLE_ERR_ARG;
    int64_t problems = B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t ph = 0; ph < problems; ph++) {
        int64_t b = ph / H; int h = (int)(ph % H);
        const int8_t* qp = q + b * batch_stride + h * head_stride;
        const int8_t* kp = k + b * batch_stride + h * head_stride;
        const int8_t* vp = v + b * batch_stride + h * head_stride;
        int64_t* s = (int64_t*)malloc(sizeof(int64_t) * (size_t)N);
        uint8_t* msk = (uint8_t*)malloc((size_t)N);
        uint8_t* p = (uint8_t*)malloc((size_t)N);
        for (int i = 0; i < N; i++) {
            for (int j = 0; j < N; j++) {
                int64_t acc = 0;
                for (int d = 0; d < dh; d++) acc += (int64_t)qp[i * tok_stride + d] * kp[j * tok_stride + d];
                if (bias) acc += bias[((int64_t)h * N + i) * N + j];
                s[j] = acc;
                msk[j] = mask_id ? (mask_id[b * N + i] != mask_id[b * N + j]) : 0;
            }
            oracle_softmax_row(s, mask_id ? msk : NULL, N, sc, p);
            for (int d = 0; d < dh; d++) {
                int64_t acc = 0;
                if (sc->variant == ORACLE_SM_LOG2) {
                    /* shift-accumulate: p = 2^-code at scale 2^-15, i.e. the value shifted left by 15 - code */
                    for (int j = 0; j < N; j++)
                        if (p[j] != ORACLE_LOG2_ZERO) acc += (int64_t)vp[j * tok_stride + d] << (15 - p[j]);
                } else {
                    for (int j = 0; j < N; j++) acc += (int64_t)p[j] * vp[j * tok_stride + d];
                }
                out[(b * N + i) * (int64_t)(H * dh) + h * dh + d] = (int8_t)oracle_requant((int32_t)acc, out_rq);
            }
        }
        free(s); free(msk); free(p);
    }
    return ORACLE_OK;
}

int oracle_attention_block(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H, int N,
                           int dh, const int32_t* bias, const uint8_t* mask_id, const oracle_softmax_consts_t* sc,
                           const oracle_requant_t* out_rq)
{
    /* q, k, v are [B, H, N, dh] */
    return oracle_attention_strided(q, k, v, out, B, H, N, dh, dh, (int64_t)N * dh, (int64_t)H * N * dh,
                                    bias, mask_id, sc, out_rq);
}

int oracle_mlp_block(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                     const oracle_gelu_consts_t* gc, const void* w2, const int32_t* b2, const int32_t* m2,
                     const int8_t* s2, int32_t out_zp, const int8_t* residual, const oracle_requant_t* residual_rq,
                     int8_t* y, int64_t M, int D, int Dh, int w_bits)
{
    return oracle_mlp_block_bits(x, w1, b1, m1, s1, gc, w2, b2, m2, s2, out_zp, residual, residual_rq, y, M, D, Dh,
                                 w_bits, 8);
}

int oracle_mlp_block_bits(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                          const oracle_gelu_consts_t* gc, const void* w2, const int32_t* b2, const int32_t* m2,
                          const int8_t* s2, int32_t out_zp, const int8_t* residual,
                          const oracle_requant_t* residual_rq, int8_t* y, int64_t M, int D, int Dh, int w_bits,
                          int out_bits)
{
    if (!x || !w1 || !m1 || !s1 || !gc || !y) return ORACLE_ERR_ARG;
    if (w_bits != 8 && w_bits != 4) return ORACLE_ERR_ARG;
    int8_t* h = w2 ? (int8_t*)malloc((size_t)M * (size_t)Dh) : y;
    int64_t lo = -((int64_t)1 << (gc->in_bits - 1)), hi = ((int64_t)1 << (gc->in_bits - 1)) - 1;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; m++) {
        for (int n = 0; n < Dh; n++) {
            int64_t acc = b1 ? b1[n] : 0;
            for (int k = 0; k < D; k++) acc += (int64_t)x[m * D + k] * weight_at(w1, w_bits, n, D, k);
            /* per-channel requant of the accumulator to the common GELU input scale, at in_bits */
            int64_t xin = clamp64(requant_noclamp(acc, m1[n], s1[n]), lo, hi);
            int64_t core = oracle_gelu_core(xin, gc);
            h[m * Dh + n] = (int8_t)oracle_requant((int32_t)core, &gc->out);
        }
    }
    if (!w2) return ORACLE_OK;
    int rc = oracle_linear_bits(h, w2, w_bits, b2, m2, s2, out_zp, residual, residual_rq, y, M, D, Dh, out_bits);
    free(h);
    return rc;
}

int oracle_encoder_block(const int8_t* x, int8_t* y, const oracle_block_params_t* p)
{
    if (!x || !y || !p) return ORACLE_ERR_ARG;
    int64_t T = p->B * p->N;
    int D = p->D;
    int rc;
    const int ab = p->act_bits ? p->act_bits : 8;      /* activation width of the three linear outputs */
    int8_t* h1 = (int8_t*)malloc((size_t)T * D);
    int8_t* qkv = (int8_t*)malloc((size_t)T * 3 * D);
    int8_t* att = (int8_t*)malloc((size_t)T * D);
    int8_t* x1 = (int8_t*)malloc((size_t)T * D);
    int8_t* h2 = (int8_t*)malloc((size_t)T * D);
    rc = oracle_layernorm(x, h1, T, D, p->ln1_gamma, p->ln1_beta, p->ln1_ptf, p->ln1);
    if (!rc) rc = oracle_linear_bits(h1, p->w_qkv, p->w_bits, p->b_qkv, p->m_qkv, p->s_qkv, 0, NULL, NULL, qkv, T, 3 * D, D, ab);
    /* qkv row = [q | k | v], head h at columns h*dh */
    if (!rc) rc = oracle_attention_strided(qkv, qkv + D, qkv + 2 * D, att, p->B, p->H, p->N, p->dh,
                                           3 * (int64_t)D, p->dh, (int64_t)p->N * 3 * D,
                                           p->attn_bias, p->mask_id, p->sm, p->pv_rq);
    if (!rc) rc = oracle_linear_bits(att, p->w_proj, p->w_bits, p->b_proj, p->m_proj, p->s_proj, p->proj_zp,
                                     x, p->res1_rq, x1, T, D, D, ab);
    if (!rc) rc = oracle_layernorm(x1, h2, T, D, p->ln2_gamma, p->ln2_beta, p->ln2_ptf, p->ln2);
    if (!rc) rc = oracle_mlp_block_bits(h2, p->w_fc1, p->b_fc1, p->m_fc1, p->s_fc1, p->gelu, p->w_fc2, p->b_fc2,
                                        p->m_fc2, p->s_fc2, p->fc2_zp, x1, p->res2_rq, y, T, D, p->Dh, p->w_bits, ab);
    free(h1); free(qkv); free(att); free(x1); free(h2);
    return rc;
}
