/*
 * CPU oracle for the integer-only non-linear path of IPTQ-ViT.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a deliberately plain, slow, one-element-
 * at-a-time restatement of what the method computes, written from the paper's
 * formulas with 64-bit intermediates.  It shares no code, header, table or
 * constant generator with the CUDA library: only tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.  All pointers are HOST memory.
 *
 * Notation used throughout (paper, Sec. 3.1 "Background"): a tensor is an
 * integer array Q plus a scale S (and zero point); "x >> k" on a negative
 * value is an arithmetic shift, i.e. floor(x / 2^k); floor() is the floor.
 *
 * Functions whose definition the paper leaves open carry the words
 * "reading:" beside the choice that was made.
 *
 * Parity status: every function below is pinned by CPU tests except
 *   - ORACLE_SM_POLY, ORACLE_SM_LOG2 and ORACLE_GELU_SHIFT: the paper names these candidates
 *     (Sec. 3.2) but defines none of them; pinned only against the float functions
 *     they approximate, with constants from the cited prior work
 *     ("parity unpinned" beyond that);
 *   - the three LayerNorm variants: named in Sec. 3.2, defined nowhere in the
 *     paper; pinned against exact integer square roots and the fp64
 *     LayerNorm ("parity unpinned" against the paper, which prints nothing).
 */
#ifndef IPTQ_ORACLE_H
#define IPTQ_ORACLE_H

#include <stdint.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_OK = 0, ORACLE_ERR_RANGE = 1, ORACLE_ERR_ARG = 2 };

enum { ORACLE_SM_BITEXP = 0, ORACLE_SM_SHIFTMAX = 1, ORACLE_SM_POLY = 2, ORACLE_SM_LOG2 = 3 };
/* ORACLE_SM_LOG2 writes codes instead of probabilities: p = 2^-code for code 0..15, ORACLE_LOG2_ZERO for p = 0;
 * the attention then accumulates shifted values at scale 2^-15. */
#define ORACLE_LOG2_ZERO 255
enum { ORACLE_GELU_POLY4 = 0, ORACLE_GELU_POLY2 = 1, ORACLE_GELU_SHIFT = 2 };
enum { ORACLE_LN_SHIFT = 0, ORACLE_LN_NEWTON = 1, ORACLE_LN_PTF = 2 };

/* Dyadic requantisation: real ratio = mult * 2^-(32+shift). */
typedef struct {
    int32_t mult;   /* in [2^30, 2^31) */
    int32_t shift;  /* in [1, 31] */
    int32_t zp;     /* added after the shift */
    int32_t qmin, qmax;
} oracle_requant_t;

typedef struct {
    int32_t variant;
    int32_t out_bits;  /* b of Eq. (15) */
    int32_t row_len;   /* n, used to size M */
    int32_t x0;        /* floor(1/S), Eq. (14) */
    int32_t nsh;       /* left pre-shift N applied before ">> q" (Eq. (9)) */
    int32_t M;         /* exponent of IntDiv, Eq. (15) */
    int32_t dcap;      /* clamp of (max - s) */
    /* ORACLE_SM_POLY only */
    int32_t qln2, qb, qc, norm_l, norm_r;
} oracle_softmax_consts_t;

typedef struct {
    int32_t variant;
    int32_t in_bits;
    int32_t Bq;        /* floor(|b| / S') */
    int32_t sh2;       /* shift after the first square */
    int32_t C;         /* integer meaning "1.0" of the erf polynomial */
    int32_t gs;        /* shift of G before the final multiply */
    /* ORACLE_GELU_SHIFT only */
    int32_t x0, nsh, dcap;
    oracle_requant_t out;
} oracle_gelu_consts_t;

typedef struct {
    int32_t variant;
    int32_t dim;
    oracle_requant_t out;
} oracle_ln_consts_t;

/* ---- requant ---------------------------------------------------------- */
int     oracle_requant_prepare(double ratio, int32_t zp, int32_t qmin, int32_t qmax, oracle_requant_t* out);
int32_t oracle_requant(int32_t y, const oracle_requant_t* rq);

/* ---- Softmax ---------------------------------------------------------- */
int oracle_softmax_prepare(double in_scale, int row_len, int out_bits, int variant, oracle_softmax_consts_t* out);
/* Integer exponential of one clamped distance d = min(max - s, dcap) >= 0. */
int64_t oracle_softmax_exp(int64_t d, const oracle_softmax_consts_t* c);
/* One row; mask (nullable) marks entries to exclude (non-zero = masked). */
void oracle_softmax_row(const int64_t* s, const uint8_t* mask, int n, const oracle_softmax_consts_t* c, uint8_t* p);
int oracle_softmax(const int32_t* scores, uint8_t* probs, int64_t rows, int row_len,
                   const int32_t* bias, int64_t bias_period, const oracle_softmax_consts_t* c);

/* ---- GELU ------------------------------------------------------------- */
int oracle_gelu_prepare(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                        int variant, oracle_gelu_consts_t* out);
/* The quartic variant with coefficients (a, b) of Eq. (3) refitted to the data range (Eq. (4)); a < 0, b < 0. */
int oracle_gelu_prepare_coeffs(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                               double a, double b, oracle_gelu_consts_t* out);
/* Pre-requant integer y = x * (G >> gs) (or x * sigma_q) of one element. */
int64_t oracle_gelu_core(int64_t x, const oracle_gelu_consts_t* c);
/* Scale of the value oracle_gelu_core returns. */
double  oracle_gelu_core_scale(double in_scale, const oracle_gelu_consts_t* c);
int oracle_gelu(const int32_t* x, int8_t* y, int64_t n, const oracle_gelu_consts_t* c);

/* ---- LayerNorm -------------------------------------------------------- */
int oracle_layernorm_prepare(int dim, const float* gamma, const float* beta, double out_scale, int out_zp,
                             int out_bits, int variant, int32_t* gamma_q, int32_t* beta_q, oracle_ln_consts_t* out);
uint64_t oracle_isqrt(uint64_t V, int variant);
int oracle_layernorm(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gamma_q,
                     const int32_t* beta_q, const uint8_t* ptf_shift, const oracle_ln_consts_t* c);

/* ---- integer GEMM carriers and the fused blocks ----------------------- */
int oracle_linear(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                  const int8_t* shift, int32_t out_zp, const int8_t* residual, const oracle_requant_t* residual_rq,
                  int8_t* y, int64_t M, int N, int K);
int oracle_linear_bits(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                       const int8_t* shift, int32_t out_zp, const int8_t* residual,
                       const oracle_requant_t* residual_rq, int8_t* y, int64_t M, int N, int K, int out_bits);
int oracle_attention_block(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H, int N,
                           int dh, const int32_t* bias, const uint8_t* mask_id, const oracle_softmax_consts_t* sc,
                           const oracle_requant_t* out_rq);
/* Same with explicit element strides for q/k/v (token, head, batch), used by the block composition. */
int oracle_attention_strided(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H, int N,
                             int dh, int64_t tok_stride, int64_t head_stride, int64_t batch_stride,
                             const int32_t* bias, const uint8_t* mask_id, const oracle_softmax_consts_t* sc,
                             const oracle_requant_t* out_rq);
int oracle_mlp_block(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                     const oracle_gelu_consts_t* gc, const void* w2, const int32_t* b2, const int32_t* m2,
                     const int8_t* s2, int32_t out_zp, const int8_t* residual, const oracle_requant_t* residual_rq,
                     int8_t* y, int64_t M, int D, int Dh, int w_bits);

int oracle_mlp_block_bits(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                          const oracle_gelu_consts_t* gc, const void* w2, const int32_t* b2, const int32_t* m2,
                          const int8_t* s2, int32_t out_zp, const int8_t* residual,
                          const oracle_requant_t* residual_rq, int8_t* y, int64_t M, int D, int Dh, int w_bits,
                          int out_bits);

/* Parameters of one encoder block (all host pointers). */
typedef struct {
    int64_t B; int32_t N, D, H, dh, Dh, w_bits;
    int32_t sm_variant, gelu_variant, ln1_variant, ln2_variant;   /* informative: the consts carry them */
    const int32_t *ln1_gamma, *ln1_beta; const uint8_t* ln1_ptf; const oracle_ln_consts_t* ln1;
    const void* w_qkv; const int32_t *b_qkv, *m_qkv; const int8_t* s_qkv;
    const int32_t* attn_bias; const uint8_t* mask_id;
    const oracle_softmax_consts_t* sm; const oracle_requant_t* pv_rq;
    const void* w_proj; const int32_t *b_proj, *m_proj; const int8_t* s_proj; int32_t proj_zp;
    const oracle_requant_t* res1_rq;
    const int32_t *ln2_gamma, *ln2_beta; const uint8_t* ln2_ptf; const oracle_ln_consts_t* ln2;
    const void* w_fc1; const int32_t *b_fc1, *m_fc1; const int8_t* s_fc1; const oracle_gelu_consts_t* gelu;
    const void* w_fc2; const int32_t *b_fc2, *m_fc2; const int8_t* s_fc2; int32_t fc2_zp;
    const oracle_requant_t* res2_rq;
    int32_t act_bits;      /* width of the QKV / proj / FC2 outputs: 0 or 8 = int8, 6 = the W6A6 setting */
} oracle_block_params_t;
/* x [B*N, D] -> y [B*N, D]; scratch is allocated inside (host malloc). */
int oracle_encoder_block(const int8_t* x, int8_t* y, const oracle_block_params_t* p);

int oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
