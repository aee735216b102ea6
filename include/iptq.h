/*
 * iptq.h -- C ABI of the B200 (sm_100a) library for the integer-only non-linear
 * layers of IPTQ-ViT and the INT8 blocks they are fused into.
 *
 * Conventions (all entry points)
 *   - Every function returns an iptq_status (0 = IPTQ_OK).  Argument errors are
 *     detected on the host and reported before anything is launched.
 *   - "dev" pointers are DEVICE memory owned by the caller; they must stay alive
 *     until the work enqueued on `stream` has completed.  "host" pointers are
 *     host memory and are only read/written during the call.
 *   - Work is enqueued on the caller's stream; no call synchronises except
 *     iptq_check().  No call allocates device memory: scratch comes from the
 *     caller's workspace `ws` (device, 256-byte aligned, size from the matching
 *     *_workspace_bytes()).  The first 256 bytes of a workspace hold the status
 *     block that device-side bounded waits write to (see iptq_check()).
 *   - Tensors are dense row-major, base pointers 16-byte aligned.
 *   - ">>" on negative values is an arithmetic shift (floor).  Quantised
 *     tensors follow the uniform quantiser of Sec. 3.1 ("Background"): an
 *     integer array plus (scale, zero point, bit-width) passed as arguments.
 *   - Float scales appear only in the host-side *_prepare() functions, which
 *     turn them into the plain-old-data integer constants the kernels consume.
 */
#ifndef IPTQ_H
#define IPTQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* iptq_stream_t;   /* same type as cudaStream_t */

typedef enum {
    IPTQ_OK = 0,
    IPTQ_ERR_NULL = 1,         /* a required pointer is NULL */
    IPTQ_ERR_SHAPE = 2,        /* a size is zero/negative/unsupported */
    IPTQ_ERR_ALIGN = 3,        /* a pointer or stride breaks the alignment contract */
    IPTQ_ERR_BITS = 4,         /* unsupported bit-width */
    IPTQ_ERR_SCALE_RANGE = 5,  /* a scale/ratio falls outside what the integer constants can hold */
    IPTQ_ERR_VARIANT = 6,      /* unknown approximation variant */
    IPTQ_ERR_WORKSPACE = 7,    /* workspace missing or too small */
    IPTQ_ERR_TIMEOUT = 8,      /* a bounded device-side wait gave up (reported by iptq_check) */
    IPTQ_ERR_CUDA = 9          /* a CUDA runtime/driver call failed */
} iptq_status;

/* Candidate approximation functions per layer type (Sec. 3.2, "Overall Pipeline"). */
typedef enum {
    IPTQ_SM_BITEXP = 0,    /* Efficient Bit-Softmax, Eqs. (13)-(15) (the paper's own; default) */
    IPTQ_SM_SHIFTMAX = 1,  /* bit-shifting candidate, Eqs. (7)-(10) */
    IPTQ_SM_POLY = 2,      /* polynomial candidate (second-order integer exp) */
    IPTQ_SM_LOG2 = 3       /* logarithm candidate: probabilities rounded to powers of two, 4-bit codes */
} iptq_softmax_variant;
typedef enum {
    IPTQ_GELU_POLY4 = 0,   /* Data-aware Poly-GELU, Eqs. (3), (5) (the paper's own; default) */
    IPTQ_GELU_POLY2 = 1,   /* polynomial candidate (second-order erf), Eq. (2) */
    IPTQ_GELU_SHIFT = 2    /* bit-shifting candidate: x * sigmoid(1.702 x) with the shift exponential */
} iptq_gelu_variant;
typedef enum {
    IPTQ_LN_SHIFT = 0,     /* bit-shifting candidate: fixed 10-step shift/add square root (default) */
    IPTQ_LN_NEWTON = 1,    /* polynomial candidate: integer square root iterated to convergence */
    IPTQ_LN_PTF = 2        /* logarithm candidate: per-channel power-of-two factors on the input */
} iptq_ln_variant;

/* The per-layer table of Sec. 3.2: which candidate each activation layer of one block runs. */
typedef struct {
    iptq_softmax_variant sm;
    iptq_gelu_variant gelu;
    iptq_ln_variant ln1, ln2;
} iptq_variant_table;

/*
 * Dyadic requantisation R (the integer-only pipelines of Sec. 2 use a dyadic
 * multiplier; the paper gives no formula, this is the library's definition):
 *   R(y) = clamp(((hi32(y * mult) + 2^(shift-1)) >> shift) + zp, qmin, qmax)
 * hi32(p) = floor(p / 2^32) of the exact 64-bit product; the real ratio is
 * mult * 2^-(32 + shift), mult in [2^30, 2^31), shift in [1, 31].
 */
typedef struct {
    int32_t mult, shift, zp, qmin, qmax;
} iptq_requant;

/* host: ratio must be in [2^-33, 1/4) -> IPTQ_ERR_SCALE_RANGE otherwise. */
int iptq_requant_prepare(double ratio, int32_t zp, int32_t qmin, int32_t qmax, iptq_requant* out /*host*/);
/* host: per-output-channel ratios[n] -> mult[n], shift[n] (all host arrays). */
int iptq_channel_requant_prepare(const double* ratios, int n, int32_t* mult, int8_t* shift);

/* ------------------------------------------------------------------ Softmax
 * Sec. 3.4 ("Efficient Bit-exp for Integer-only Softmax"), Eqs. (6)-(15).
 * Per row of int32 scores s at scale S: mx = max s; d = min(mx - s, dcap);
 * Qp = -d + (-d >> 1) - (-d >> 4) (Eq. (7)); (q, r) = divmod(-Qp, x0), x0 = floor(1/S)
 * (Eq. (8)); e = ((Phi(-r) + x0) << nsh) >> q with Phi(u) = (u>>1)+(u>>3)+(u>>4)
 * (Eqs. (9), (13), (14)); p = (floor(2^M / sum e) * e) >> (M - (out_bits-1)) (Eq. (15)).
 * Output: uint8 probabilities at scale 2^-(out_bits-1), values in [0, 2^(out_bits-1)].
 *
 * IPTQ_SM_LOG2 (the "logarithm" candidate of Sec. 3.2, which the paper names without defining; out_bits must be
 * 4): with the polynomial exponential e and its row sum, r = round(sum / e) and
 * code = round(log2 r) = position of the leading one of r, plus one when the bit below it is set; the output byte
 * is that code (probability 2^-code) for code <= 15 and IPTQ_LOG2_ZERO (probability 0) beyond or where e = 0.
 */
#define IPTQ_LOG2_ZERO 255
typedef struct {
    int32_t variant, out_bits, row_len;
    int32_t x0, nsh, M, dcap;
    int32_t qln2, qb, qc, norm_l, norm_r;    /* IPTQ_SM_POLY only */
    /* derived, for the kernels: floor(v / x0) == umulhi(v, div_mul) >> div_shift for 0 <= v < 2^31 */
    uint32_t div_mul; int32_t div_shift;
    int32_t f_shl, p_shr;                    /* p = umulhi(f << f_shl, e) >> p_shr */
    const uint16_t* table;                   /* optional: dev, from iptq_softmax_table(); NULL = none */
    int32_t table_n;                         /* entries e(0) .. e(table_n - 1) of that table */
} iptq_softmax_consts;

/* host.  in_scale: scale of the scores (1/sqrt(d_head) folded in); needs 8 <= floor(1/in_scale) < 2^24
 * and row_len * (x0 << nsh) < 2^31 (IPTQ_ERR_SCALE_RANGE); out_bits in [4, 8] (IPTQ_SM_LOG2: 4, else
 * IPTQ_ERR_BITS); 1 <= row_len <= 1024. */
int iptq_softmax_prepare(double in_scale, int row_len, int out_bits, iptq_softmax_variant variant,
                         iptq_softmax_consts* out /*host*/);
/* The integer exponential of every variant (Eq. (9) for IPTQ_SM_BITEXP / IPTQ_SM_SHIFTMAX, the second-order
 * polynomial behind IPTQ_SM_POLY / IPTQ_SM_LOG2) is a function of d = max - s alone, is 0 from some d on (a few
 * x0) and, where its largest value is below 2^16, fits 16 bits, so the whole function is a short table.
 * iptq_softmax() and the attention kernels build that table per CTA in shared memory; iptq_softmax_table() writes
 * it once to device memory with the same arithmetic -- e(0) .. e(n - 1), then zeros up to the next multiple of 8
 * entries -- and stores the pointer and n in consts, after which the kernels copy it instead.  Results are
 * identical either way.
 * *consts: host, updated (table = NULL, table_n = 0 and nothing written where this scale has no such
 * table).  table: dev uint16 [capacity], 16-byte aligned, caller-owned, must outlive every use of consts;
 * IPTQ_ERR_SHAPE when capacity is too small (IPTQ_SOFTMAX_TABLE_MAX entries always suffice: larger tables are
 * not used by the kernels and count as "no table").  Work submitted to the stream after this call sees the
 * complete table. */
#define IPTQ_SOFTMAX_TABLE_MAX 51200
int iptq_softmax_table(iptq_softmax_consts* consts, uint16_t* table, int32_t capacity, iptq_stream_t stream);
/* scores: dev int32 [rows, row_len], |score| < 2^30 (with a bias: |score + bias| < 2^30).  probs: dev uint8
 * [rows, row_len].  bias: nullable dev int32 [bias_period, row_len] at the score scale; row i adds bias row
 * (i % bias_period).
 * consts: host.  No workspace. */
int iptq_softmax(const int32_t* scores, uint8_t* probs, int64_t rows, int row_len, const int32_t* bias,
                 int64_t bias_period, const iptq_softmax_consts* consts, iptq_stream_t stream);

/* ------------------------------------------------------------------ GELU
 * Sec. 3.3 ("Data-aware Poly-GELU"), Eqs. (1)-(5): GELU(x) ~ x/2 [1 + L(x/sqrt 2)],
 * L(u) = sign(u) [a (min(|u|, -b) + b)^4 + 1], a = -0.019913, b = -2.698088.
 * Integer form per element (x: in_bits-bit value at scale S, S' = S/sqrt 2, Bq = floor(|b|/S')):
 *   m = min(|x|, Bq); t = Bq - m; t2 = (t*t) >> sh2; E = C - t2*t2; G = sgn(x)*E + C;
 *   y = x * (G >> gs); out = R(y).     (IPTQ_GELU_POLY2: E = C - t2.)
 */
typedef struct {
    int32_t variant, in_bits;
    int32_t Bq, sh2, C, gs;
    int32_t x0, nsh, dcap;                   /* IPTQ_GELU_SHIFT only */
    uint32_t div_mul; int32_t div_shift;     /* IPTQ_GELU_SHIFT only: division by x0 */
    iptq_requant out;
    const int8_t* table;                     /* optional: dev, IPTQ_GELU_TABLE_SIZE bytes from iptq_gelu_table(); NULL = none */
} iptq_gelu_consts;

/* The integer GELU maps an in_bits-bit input (<= 16 bits) to 8 bits, so the whole function fits a 64 KB table:
 * table[x + 32768] = the value iptq_gelu() returns for x (x below/above the in_bits range is clamped first, as
 * in the kernel).  iptq_gelu_table() fills such a table with the same arithmetic; when consts->table points to it,
 * the FC1 epilogue of iptq_mlp_block() / iptq_encoder_block(), and iptq_gelu() on inputs of 2^20 elements and more,
 * keep a copy in shared memory and replace the polynomial by one read per output.  The results are identical with and without the table.
 * table: dev int8 [IPTQ_GELU_TABLE_SIZE], 16-byte aligned, caller-owned; consts: host (its own `table` is ignored).
 * Work submitted to the stream after this call sees the complete table. */
#define IPTQ_GELU_TABLE_SIZE 65536
int iptq_gelu_table(const iptq_gelu_consts* consts, int8_t* table, iptq_stream_t stream);

/* host.  in_bits in [8, 16], out_bits in [4, 8]; floor(|b| / S') must be in [1, 2^15). */
int iptq_gelu_prepare(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                      iptq_gelu_variant variant, iptq_gelu_consts* out /*host*/);
/* Data-aware coefficients (Sec. 3.3, Eq. (4)): the paper re-computes (a, b) of Eq. (3) for the value range of the
 * data, [min(T), max(T)], by least squares against erf.  iptq_gelu_fit does that on a uniform grid of `points`
 * values over [lo, hi] (the paper gives the range, not the sample): *a, *b receive the coefficients (both
 * negative), *rms (nullable) the root-mean-square residual.  Host only; 8 <= points <= 2^22, hi > lo.
 * iptq_gelu_prepare_coeffs is iptq_gelu_prepare(IPTQ_GELU_POLY4) with these coefficients in place of the
 * paper's constants (a, b < 0, else IPTQ_ERR_SCALE_RANGE); the kernels need nothing else. */
int iptq_gelu_fit(double lo, double hi, int points, double* a /*host*/, double* b /*host*/, double* rms /*host*/);
int iptq_gelu_prepare_coeffs(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits, double a,
                             double b, iptq_gelu_consts* out /*host*/);
/* x: dev int32 [n] (clamped to in_bits inside); y: dev int8 [n]; consts: host. */
int iptq_gelu(const int32_t* x, int8_t* y, int64_t n, const iptq_gelu_consts* consts, iptq_stream_t stream);

/* ------------------------------------------------------------------ LayerNorm
 * Sec. 3.2 names the LayerNorm candidates; the paper defines none, so the integer
 * algorithm is the library's: s1 = sum x, s2 = sum x^2, u_c = D x_c - s1, V = D s2 - s1^2,
 * r = isqrt_variant(V), F = floor(2^40 / r), n_c = (u_c F) >> 30 (Q10, 0 when r = 0),
 * y_c = n_c gamma_q[c] + beta_q[c], out = R(y_c).  The input scale cancels.
 */
typedef struct {
    int32_t variant, dim;
    iptq_requant out;
} iptq_ln_consts;

/* host.  gamma/beta: host float [dim]; gamma_q/beta_q: host int32 [dim] outputs
 * (gamma_q = round(gamma / S_g), S_g = max|gamma| / 32767; beta_q = round(beta / (2^-10 S_g))).
 * 2 <= dim <= 3072 (n_c gamma_q + beta_q must stay below 2^31), dim % 4 == 0. */
int iptq_layernorm_prepare(int dim, const float* gamma, const float* beta, double out_scale, int out_zp,
                           int out_bits, iptq_ln_variant variant, int32_t* gamma_q, int32_t* beta_q,
                           iptq_ln_consts* out /*host*/);
/* x, y: dev int8 [rows, dim]; gamma_q, beta_q: dev int32 [dim];
 * ptf_shift: dev uint8 [dim] in 0..3, used (and required) only by IPTQ_LN_PTF; consts: host. */
int iptq_layernorm(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gamma_q,
                   const int32_t* beta_q, const uint8_t* ptf_shift, const iptq_ln_consts* consts,
                   iptq_stream_t stream);

/* ------------------------------------------------------------------ INT8 GEMM carrier
 * Linear ops run in integer arithmetic (Sec. 3.1): acc[m,n] = sum_k x[m,k] w[n,k] + bias[n], which must fit int32
 * (K <= 4096 keeps the sum below 2^26 in magnitude);
 * y = clamp(R_n(acc) + R_res((residual - residual_rq.zp) << 16) + out_zp, -128, 127), where R_n uses
 * (mult[n], shift[n]) without zero point/clamp and the residual term is present only if residual != NULL.
 * x: dev int8 [M, K]; w: dev int8 [N, K] (w_bits = 8) or packed int4 [N, K/2] (w_bits = 4: element k in
 * byte k/2, even k in the low nibble, two's complement); bias: nullable dev int32 [N] (input zero point
 * folded in by the caller); mult: dev int32 [N]; shift: dev int8 [N]; residual: nullable dev int8 [M, N];
 * residual_rq: host; y: dev int8 [M, N].  K % 16 == 0, N % 16 == 0, K <= 4096.
 * ws: required (status block; plus N*K bytes of unpack scratch when w_bits = 4).
 */
/* Packed int4 weights -> int8 [n_elems] (the format w_bits = 8 takes), for deployments that keep the W4 checkpoint
 * packed on disk but unpack each weight once at load time instead of at every call: the same values, so the same
 * results as w_bits = 4.  packed: dev [n_elems / 2] bytes; out: dev int8 [n_elems], both 16-byte aligned;
 * n_elems even (IPTQ_ERR_SHAPE otherwise). */
int iptq_unpack_int4(const void* packed, int8_t* out, int64_t n_elems, iptq_stream_t stream);
size_t iptq_linear_workspace_bytes(int64_t M, int N, int K, int w_bits);
/* How iptq_linear() would tile an [M, K] x [N, K]^T product (no counterpart in the paper; host arithmetic only, for
 * capacity planning and tests): tokens per tile (64, 128, 192 or 256), depth of the operand ring, whether CTA pairs
 * (clusters of two, one 256-channel MMA stream) are used, dynamic shared memory per CTA, grid size, the tile
 * counts, and whether the epilogue stages outputs and residuals in one buffer per warp or in two used by alternate
 * tiles (two where they cost no ring stage).  has_residual / has_gelu_table: the epilogue's staging needs;
 * sm_count: SMs to plan for, 0 = those of the current device (the only case that touches CUDA).  IPTQ_ERR_SHAPE
 * for sizes iptq_linear() rejects. */
typedef struct {
    int32_t tile_tokens, stages, cta_pairs, smem_bytes, grid, channel_tiles, token_tiles, staging_buffers;
} iptq_linear_plan_info;
int iptq_linear_plan(int64_t M, int N, int K, int has_residual, int has_gelu_table, int sm_count,
                     iptq_linear_plan_info* out);
int iptq_linear(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                const int8_t* shift, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                int8_t* y, int64_t M, int N, int K, void* ws, size_t ws_bytes, iptq_stream_t stream);
/* The same layer with activations out_bits wide (4..8; the W6A6 setting of Sec. 4 uses 6): y is clamped to
 * [-2^(out_bits-1), 2^(out_bits-1) - 1] instead of the int8 range, still stored as int8.  iptq_linear() is out_bits = 8. */
int iptq_linear_bits(const int8_t* x, const void* w, int w_bits, const int32_t* bias, const int32_t* mult,
                     const int8_t* shift, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                     int8_t* y, int64_t M, int N, int K, int out_bits, void* ws, size_t ws_bytes,
                     iptq_stream_t stream);

/* ------------------------------------------------------------------ 4-bit-weight GEMM without any allocation
 * (No counterpart in the paper: this is a packaging variant of iptq_linear(w_bits = 4) for callers that
 * cannot provide a workspace.)
 *
 * Who needs it: code that is not allowed to allocate device memory at the point where it runs the layer --
 * an inference loop that must never reach cudaMalloc/cudaFree (both may synchronise the whole device and
 * their latency is unbounded), a plug-in running inside a host application that handed it a fixed set of
 * buffers, or a process whose memory pool is owned by another component.  Such a caller has the layer's
 * inputs and outputs but nowhere to put the N*K bytes of sign-extended weights that the tensor-core kernel
 * reads, so the library keeps that scratch itself: one file-scope device array of
 * 256 + IPTQ_STATIC_SCRATCH_BYTES bytes, present on every GPU that loads the library until the process ends.
 *
 * Same arithmetic, arguments and result as iptq_linear(..., w_bits = 4, ...), minus the workspace:
 *   - N * K must not exceed IPTQ_STATIC_SCRATCH_BYTES (4 MiB; ViT-Base FC1/FC2 need 2.25 MiB);
 *     larger weights return IPTQ_ERR_WORKSPACE before anything is launched.
 *   - status: nullable dev pointer to a caller-owned 256-byte, 256-byte-aligned status block (as at the start
 *     of a workspace; read it with iptq_check).  With NULL the array's own status block is used and cleared
 *     on the stream at the start of the call; a bounded wait that gives up then still ends the kernel but
 *     cannot be queried.
 *   - The call allocates nothing (no cudaMalloc/cudaFree, no allocating library routine); it enqueues the
 *     unpack kernel, the GEMM kernel and, with status == NULL, one 256-byte memset on `stream`.
 *   - The first call on each device looks up the array's device address (a one-time set-up done with that
 *     device current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array, and it keeps the previous call's contents: every byte a call
 *     reads is rewritten by that call first, but two calls whose GPU work overlaps (different streams, or
 *     several host threads) race on it.  Serialise them on one stream or with events.
 */
#define IPTQ_STATIC_SCRATCH_BYTES (4u << 20)
int iptq_linear_w4_static(const int8_t* x, const void* w_packed, const int32_t* bias, const int32_t* mult,
                          const int8_t* shift, int32_t out_zp, const int8_t* residual,
                          const iptq_requant* residual_rq, int8_t* y, int64_t M, int N, int K,
                          void* status /*nullable dev*/, iptq_stream_t stream);

/* ------------------------------------------------------------------ fused attention
 * QK^T (INT8 -> int32, kept on chip) -> (+ bias) -> integer Softmax of Sec. 3.4 -> uint8 P -> P.V
 * (INT8 -> int32) -> R(out_rq) -> int8, heads re-interleaved.  No int32 intermediate reaches HBM.
 * q, k, v: dev int8 [B, H, N, dh] (zero point 0); out: dev int8 [B, N, H*dh];
 * bias: nullable dev int32 [H, N, N] at the score scale; mask_id: nullable dev uint8 [B, N]: the pair
 * (i, j) is masked (probability 0, excluded from max and sum) iff mask_id[b,i] != mask_id[b,j].
 * N <= 256, dh in {32, 64}; sm (host) prepared with row_len = N; out_rq: host.  ws: the status block.
 * The real ratio of out_rq is 2^-(out_bits-1) * S_v / S_out.  With IPTQ_SM_LOG2 the probabilities are the powers
 * of two 2^-code and the product is the shift-accumulate sum_j v_j << (15 - code_ij) (codes above 15: nothing),
 * so out_rq's ratio is 2^-15 * S_v / S_out.
 *
 * The relative-position bias of a window model is a weight.  For N <= 64 the kernel gives one thread a whole score
 * row, and reads the bias fastest from a copy laid out as [H][ceil(N/4)][64 rows] x 4 int32 columns (zeros past
 * column N).  iptq_attention_bias_prepare() writes that copy once, at load time, into caller-owned device memory of
 * iptq_attention_bias_bytes(H, N) bytes (16-byte aligned; 0 bytes and nothing to do for N > 64); pass it as
 * bias_t together with bias.  With bias_t == NULL the row-major bias is read as it is (same results, slower).
 */
size_t iptq_attention_workspace_bytes(int64_t B, int H, int N, int dh);
size_t iptq_attention_bias_bytes(int H, int N);
int iptq_attention_bias_prepare(const int32_t* bias, int32_t* bias_t, int H, int N, iptq_stream_t stream);
int iptq_attention_block(const int8_t* q, const int8_t* k, const int8_t* v, int8_t* out, int64_t B, int H,
                         int N, int dh, const int32_t* bias, const int32_t* bias_t /*nullable*/,
                         const uint8_t* mask_id, const iptq_softmax_consts* sm, const iptq_requant* out_rq,
                         void* ws, size_t ws_bytes, iptq_stream_t stream);

/* ------------------------------------------------------------------ fused MLP
 * FC1 (INT8 GEMM) with the integer GELU of Sec. 3.3 applied in the int32 epilogue:
 *   xin = clamp(R_n(acc1; m1[n], s1[n]), in_bits range); h = R(gelu_core(xin))  -> int8 [M, Dh]
 * then, unless w2 == NULL (stop after GELU, y is [M, Dh]), FC2 as iptq_linear with (b2, m2, s2, out_zp,
 * residual) -> y int8 [M, D].  The hidden tensor lives in the workspace.  w1: [Dh, D], w2: [D, Dh].
 */
size_t iptq_mlp_workspace_bytes(int64_t M, int D, int Dh, int w_bits);
int iptq_mlp_block(const int8_t* x, const void* w1, const int32_t* b1, const int32_t* m1, const int8_t* s1,
                   const iptq_gelu_consts* gelu, const void* w2, const int32_t* b2, const int32_t* m2,
                   const int8_t* s2, int32_t out_zp, const int8_t* residual, const iptq_requant* residual_rq,
                   int8_t* y, int64_t M, int D, int Dh, int w_bits, void* ws, size_t ws_bytes,
                   iptq_stream_t stream);

/* ------------------------------------------------------------------ token re-ordering
 * The Swin models of Sec. 4 run the block on 7x7 windows of a token grid (with a cyclic shift in every other
 * block) and merge 2x2 patches between stages; the paper does not describe either, so the layout is the usual
 * one and is expressed as a row gather: dst row i = concatenation over p < parts of src row index[i*parts + p]
 * (each row_bytes long; index < 0 -> zeros).  src: dev int8 [n_src, row_bytes]; dst: dev int8
 * [n_dst, parts*row_bytes]; index: dev int32 [n_dst, parts], built on the host; row_bytes % 16 == 0. */
int iptq_gather_rows(const int8_t* src, int8_t* dst, const int32_t* index, int64_t n_dst, int parts,
                     int row_bytes, iptq_stream_t stream);

/* Patch embedding front end of the ViT / DeiT models of Sec. 4 (the paper does not describe it; the usual one):
 * the P x P, stride-P convolution is an INT8 linear layer on patch rows, and this call lays the rows out:
 * out[(b, py, px), (c, dy, dx)] = img[b, c, py*P + dy, px*P + dx].
 * img: dev int8 [B, C, H, W]; out: dev int8 [B * (H/P) * (W/P), C*P*P]; P % 16 == 0, H % P == W % P == 0. */
int iptq_patchify(const int8_t* img, int8_t* out, int64_t B, int C, int H, int W, int P, iptq_stream_t stream);

/* ------------------------------------------------------------------ one encoder block
 * LN1 -> QKV GEMM -> fused attention -> proj GEMM (+ residual x) -> LN2 -> fused MLP (+ residual),
 * each layer running the variant its consts name (the per-layer table of Sec. 3.2).
 * All array members are dev pointers, all consts/requant members host pointers.
 * w_qkv: [3D, D], rows ordered [q | k | v], head h in rows h*dh .. h*dh+dh-1 of each third.
 */
typedef struct {
    int64_t B; int32_t N, D, H, dh, Dh, w_bits;
    iptq_variant_table table;      /* informative: must agree with the consts below */
    const int32_t *ln1_gamma, *ln1_beta; const uint8_t* ln1_ptf; const iptq_ln_consts* ln1;
    const void* w_qkv; const int32_t *b_qkv, *m_qkv; const int8_t* s_qkv;
    const int32_t* attn_bias; const uint8_t* mask_id;
    const iptq_softmax_consts* sm; const iptq_requant* pv_rq;
    const void* w_proj; const int32_t *b_proj, *m_proj; const int8_t* s_proj; int32_t proj_zp;
    const iptq_requant* res1_rq;
    const int32_t *ln2_gamma, *ln2_beta; const uint8_t* ln2_ptf; const iptq_ln_consts* ln2;
    const void* w_fc1; const int32_t *b_fc1, *m_fc1; const int8_t* s_fc1; const iptq_gelu_consts* gelu;
    const void* w_fc2; const int32_t *b_fc2, *m_fc2; const int8_t* s_fc2; int32_t fc2_zp;
    const iptq_requant* res2_rq;
    int32_t act_bits;              /* width of the QKV / proj / FC2 outputs: 0 or 8 = int8; 6 with 6-bit LayerNorm, Softmax,
                                      attention and GELU constants is the W6A6 setting of the detection results (Sec. 4) */
    const int32_t* attn_bias_t;    /* nullable: attn_bias as laid out by iptq_attention_bias_prepare() (N <= 64) */
} iptq_block_params;

size_t iptq_encoder_block_workspace_bytes(const iptq_block_params* p /*host*/);
/* x, y: dev int8 [B*N, D]. */
int iptq_encoder_block(const int8_t* x, int8_t* y, const iptq_block_params* p /*host*/, void* ws, size_t ws_bytes,
                       iptq_stream_t stream);

/* The same block with a stage boundary recorded into caller-owned events, for per-kernel timing:
 * events (host array of IPTQ_BLOCK_STAGES + 1 cudaEvent_t handles created with timing enabled) --
 * events[0] is recorded before the first launch and events[i] after stage i, in the order
 * LN1, QKV, attention, proj, LN2, FC1+GELU, FC2 (the int4 unpack launches of w_bits = 4 fall into stage 1).
 * The kernels and their results are those of iptq_encoder_block(). */
#define IPTQ_BLOCK_STAGES 7
int iptq_encoder_block_profiled(const int8_t* x, int8_t* y, const iptq_block_params* p /*host*/, void* ws,
                                size_t ws_bytes, iptq_stream_t stream, void* const* events /*host*/, int n_events);

/* ------------------------------------------------------------------ Unified Metric
 * Sec. 3.5 ("Unified Metric for Approximation Function Assignment"), Eqs. (16)-(20): every non-linear layer is
 * run with each candidate function and scored by
 *     term = 3 / ( 1/N(Q) + N(P) + N(C) ),   N(v) = log(1 + exp(v))                       Eqs. (16), (17)
 *     Q = 10 log10( E[X^2] / E[(X - Qd)^2] )  (dB; the worked example beside Eq. (18) fixes 10 log10)
 *     P = || X - Qd ||_2^2                                                                   Eq. (19)
 *     C = integer operation count of the layer                                             Eq. (20)
 * where X is the float layer and Qd the de-quantised output of the integer candidate; the layer takes the candidate
 * with the largest term (stage 2 of the pipeline).
 *
 * Device part: after the candidate's own kernel (iptq_softmax / iptq_gelu / iptq_layernorm) has produced the
 * integer output, iptq_metric_*() evaluate X in fp64 on the de-quantised integer input and reduce
 *     sums[0] = sum X^2,   sums[1] = sum (X - Qd)^2
 * over the whole tensor with a fixed summation order (the same device and sizes give the same bits).
 *   Softmax:   X = softmax(in_scale * scores) per row;  Qd = probs * 2^-(out_bits-1), or, with out_bits =
 *              IPTQ_PROBS_LOG2, 2^-code of the IPTQ_SM_LOG2 codes in probs (0 for IPTQ_LOG2_ZERO)
 *   GELU:      X = v/2 (1 + erf(v / sqrt 2)), v = in_scale * x;  Qd = (y - out_zp) * out_scale
 *   LayerNorm: X = (v - mean)/std * gamma + beta per row, v = x << ptf_shift[channel] (biased variance, no
 *              epsilon; a constant row gives beta);  Qd = (y - out_zp) * out_scale
 * sums: dev double [2], 16-byte aligned, written by the call.  work: dev scratch of IPTQ_METRIC_WORK_BYTES,
 * 16-byte aligned, caller-owned, free for reuse once the call has completed on the stream.  gamma / beta: dev
 * float [dim] (the float parameters handed to iptq_layernorm_prepare); ptf_shift nullable.  row_len <= 1024,
 * dim % 4 == 0 and dim <= 3072 as for the kernels measured.  Empty tensors give sums of 0. */
#define IPTQ_METRIC_WORK_BYTES 32768
#define IPTQ_PROBS_LOG2 0
int iptq_metric_softmax(const int32_t* scores, const uint8_t* probs, int64_t rows, int row_len, double in_scale,
                        int out_bits, double* sums, void* work, iptq_stream_t stream);
int iptq_metric_gelu(const int32_t* x, const int8_t* y, int64_t n, double in_scale, double out_scale, int out_zp,
                     double* sums, void* work, iptq_stream_t stream);
int iptq_metric_layernorm(const int8_t* x, const int8_t* y, int64_t rows, int dim, const float* gamma,
                          const float* beta, const uint8_t* ptf_shift, double out_scale, int out_zp, double* sums,
                          void* work, iptq_stream_t stream);

/* Host part.  iptq_sqnr_db returns +inf for sum_err2 == 0.  iptq_metric_term: op_count is divided by c_unit before
 * N() (the paper gives no unit; raw counts of 1e7 and more would leave N(C) as the only term that matters).
 * iptq_op_count: integer operations of one layer on [rows, row_len] (GELU: rows * row_len elements) counted from
 * this library's integer definitions, one per binary add / subtract / multiply / divide / shift / mask and per
 * comparison (sign flips, copies and prepared constants are free; a value that is the same for a whole row counts
 * once per row); returns a negative value for an unknown kind or variant.  iptq_metric_select: index of the largest term, the first of
 * equals; -1 for n < 1. */
typedef enum { IPTQ_LAYER_SOFTMAX = 0, IPTQ_LAYER_GELU = 1, IPTQ_LAYER_LAYERNORM = 2 } iptq_layer_kind;
double iptq_softplus(double v);
double iptq_sqnr_db(double sum_x2, double sum_err2);
double iptq_metric_term(double sqnr_db, double perturbation, double op_count, double c_unit);
double iptq_op_count(int layer_kind, int variant, int64_t rows, int row_len);
int iptq_metric_select(const double* terms /*host*/, int n);

/* ------------------------------------------------------------------ status
 * iptq_workspace_init: zero the status block (enqueued on the stream); call once per workspace.
 * iptq_check: synchronise the stream and return IPTQ_ERR_TIMEOUT if any kernel that used `ws`
 * abandoned a bounded wait, IPTQ_ERR_CUDA if the stream reports an error, else IPTQ_OK. */
int iptq_workspace_init(void* ws, size_t ws_bytes, iptq_stream_t stream);
int iptq_check(iptq_stream_t stream, const void* ws);
/* Every wait inside the tensor-core kernels (on a copy, on the tensor core, on another warp) is bounded: after the
 * limit it records itself in the status block -- flag, id of the wait, block index, at int32 offsets 0, 1, 2 -- makes
 * its CTA drain and return, and iptq_check() reports IPTQ_ERR_TIMEOUT.  The limit is 2 s unless the workspace
 * carries its own: iptq_workspace_set_wait_limit() stores one in the status block (microseconds; 0 = default;
 * enqueued on the stream; iptq_workspace_init() clears it again).  The host pointer is read during the call.
 * iptq_selftest_wait_timeout() (no counterpart in the paper: a diagnostic) launches one warp that waits on a
 * barrier nothing arrives at, so that the give-up path can be observed on a healthy device: afterwards iptq_check()
 * returns IPTQ_ERR_TIMEOUT with wait id 99 and block 0, the kernel has returned, and the workspace is usable
 * again after iptq_workspace_init(). */
int iptq_workspace_set_wait_limit(void* ws, size_t ws_bytes, int32_t microseconds, iptq_stream_t stream);
int iptq_selftest_wait_timeout(void* ws, size_t ws_bytes, iptq_stream_t stream);
const char* iptq_strerror(int status);
/* Number of kernels the library has launched so far in this process (for launch accounting). */
int64_t iptq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* IPTQ_H */
