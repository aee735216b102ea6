// Host side of the iptq library: float scales -> integer constants, status helpers.
#include <atomic>
#include <cmath>
#include <vector>
#include <cstring>
#include <mutex>

#include "iptq_common.cuh"

namespace iptq {

static std::atomic<int64_t> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int cuda_status(cudaError_t e) { return e == cudaSuccess ? IPTQ_OK : IPTQ_ERR_CUDA; }
int last_launch_status() { return cuda_status(cudaGetLastError()); }

int sm_count()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

static int top_bit_len(uint64_t v)
{
    int n = 0;
    for (; v; v >>= 1) ++n;
    return n;
}

// Magic multiplier for floor(v / d), 0 <= v < 2^31, 2 <= d < 2^31:
// with l = ceil(log2 d), mul = ceil(2^(31+l) / d) < 2^32 and the quotient is umulhi(v, mul) >> (l - 1).
static void magic_div31(uint32_t d, uint32_t* mul, int32_t* shift)
{
    int l = top_bit_len((uint64_t)d - 1);        // ceil(log2 d) for d >= 2
    unsigned __int128 num = (unsigned __int128)1 << (31 + l);
    uint64_t m = (uint64_t)((num + d - 1) / d);
    if (l == 0) { *mul = 0xFFFFFFFFu; *shift = 0; return; }   // d == 1 (not used: divisors are >= 8)
    *mul = (uint32_t)m;
    *shift = l - 1;
}

int check_requant(const iptq_requant* r)
{
    if (!r) return IPTQ_ERR_NULL;
    if (r->shift < 1 || r->shift > 31 || r->mult < (1 << 30)) return IPTQ_ERR_SCALE_RANGE;
    if (r->qmin > r->qmax) return IPTQ_ERR_BITS;
    return IPTQ_OK;
}

RequantDev to_dev(const iptq_requant& r)
{
    RequantDev d;
    d.mult = r.mult; d.shift = r.shift; d.rnd = 1 << (r.shift - 1);
    d.zp = r.zp; d.qmin = r.qmin; d.qmax = r.qmax;
    return d;
}

ExpDev to_dev_exp(const iptq_softmax_consts& c)
{
    ExpDev e;
    e.x0 = c.x0; e.nsh = c.nsh; e.dcap = c.dcap;
    e.div_mul = c.div_mul; e.div_shift = c.div_shift;
    e.qln2 = c.qln2; e.qb = c.qb; e.qc = c.qc; e.norm_l = c.norm_l; e.norm_r = c.norm_r;
    return e;
}

GeluDev to_dev(const iptq_gelu_consts& c)
{
    GeluDev g;
    g.variant = c.variant;
    g.lo = -(1 << (c.in_bits - 1));
    g.hi = (1 << (c.in_bits - 1)) - 1;
    g.Bq = c.Bq; g.sh2 = c.sh2; g.C = c.C; g.gs = c.gs;
    g.ex.x0 = c.x0; g.ex.nsh = c.nsh; g.ex.dcap = c.dcap;
    g.ex.div_mul = c.div_mul; g.ex.div_shift = c.div_shift;
    g.ex.qln2 = g.ex.qb = g.ex.qc = g.ex.norm_l = g.ex.norm_r = 0;
    g.out = to_dev(c.out);
    return g;
}

}  // namespace iptq

using namespace iptq;

extern "C" {

int iptq_requant_prepare(double ratio, int32_t zp, int32_t qmin, int32_t qmax, iptq_requant* out)
{
    if (!out) return IPTQ_ERR_NULL;
    if (qmin > qmax) return IPTQ_ERR_BITS;
    if (!(ratio > 0.0) || !(ratio < 0.25)) return IPTQ_ERR_SCALE_RANGE;
    // ratio = mult * 2^-(32 + shift) with mult in [2^30, 2^31)
    int e = std::ilogb(ratio);                               // floor(log2 ratio)
    double scaled = std::scalbn(ratio, 30 - e);              // in [2^30, 2^31)
    int64_t mult = (int64_t)std::floor(scaled + 0.5);
    if (mult >= (int64_t)1 << 31) { mult = (int64_t)1 << 30; ++e; }
    int shift = -e - 2;
    if (shift < 1 || shift > 31) return IPTQ_ERR_SCALE_RANGE;
    out->mult = (int32_t)mult; out->shift = shift; out->zp = zp; out->qmin = qmin; out->qmax = qmax;
    return IPTQ_OK;
}

int iptq_channel_requant_prepare(const double* ratios, int n, int32_t* mult, int8_t* shift)
{
    if (!ratios || !mult || !shift) return IPTQ_ERR_NULL;
    if (n < 1) return IPTQ_ERR_SHAPE;
    for (int i = 0; i < n; ++i) {
        iptq_requant r;
        int rc = iptq_requant_prepare(ratios[i], 0, -128, 127, &r);
        if (rc != IPTQ_OK) return rc;
        mult[i] = r.mult;
        shift[i] = (int8_t)r.shift;
    }
    return IPTQ_OK;
}

int iptq_softmax_prepare(double in_scale, int row_len, int out_bits, iptq_softmax_variant variant,
                         iptq_softmax_consts* out)
{
    if (!out) return IPTQ_ERR_NULL;
    if (row_len < 1 || row_len > 1024) return IPTQ_ERR_SHAPE;
    if (out_bits < 4 || out_bits > 8) return IPTQ_ERR_BITS;
    if (variant != IPTQ_SM_BITEXP && variant != IPTQ_SM_SHIFTMAX && variant != IPTQ_SM_POLY &&
        variant != IPTQ_SM_LOG2) return IPTQ_ERR_VARIANT;
    if (variant == IPTQ_SM_LOG2 && out_bits != 4) return IPTQ_ERR_BITS;     // 4-bit codes
    if (!(in_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    std::memset(out, 0, sizeof(*out));
    const double one = std::floor(1.0 / in_scale);           // Eq. (14): the integer 1.0
    if (!(one >= 8.0 && one < 16777216.0)) return IPTQ_ERR_SCALE_RANGE;
    const int64_t x0 = (int64_t)one;
    out->variant = (int32_t)variant; out->out_bits = out_bits; out->row_len = row_len;
    out->x0 = (int32_t)x0;
    out->dcap = (int32_t)(34 * x0);
    int64_t unit;
    if (variant == IPTQ_SM_POLY || variant == IPTQ_SM_LOG2) {
        const double a = 0.3585, b = 1.353, c = 0.344;       // exp(p) ~ a (p + b)^2 + c on (-ln 2, 0]
        const double l2 = std::floor(std::log(2.0) / in_scale);
        const double qb = std::floor(b / in_scale);
        const double qc = std::floor(c / (a * in_scale * in_scale));
        if (l2 < 1.0 || qb >= 32768.0 || qc >= 1073741824.0) return IPTQ_ERR_SCALE_RANGE;
        out->qln2 = (int32_t)l2; out->qb = (int32_t)qb; out->qc = (int32_t)qc;
        const int64_t top = (int64_t)out->qb * out->qb + out->qc;      // value at p = 0
        const int w = top_bit_len((uint64_t)top);
        out->norm_l = w <= 14 ? 14 - w : 0;
        out->norm_r = w > 14 ? w - 14 : 0;
        unit = (top << out->norm_l) >> out->norm_r;
        out->nsh = 0;
        magic_div31((uint32_t)out->qln2, &out->div_mul, &out->div_shift);
    } else {
        const int w = top_bit_len((uint64_t)x0);
        out->nsh = w < 14 ? 14 - w : 0;                       // x0 << nsh in [2^13, 2^14) when x0 < 2^13
        unit = x0 << out->nsh;
        magic_div31((uint32_t)x0, &out->div_mul, &out->div_shift);
    }
    const int64_t worst_sum = (int64_t)row_len * unit;
    if (worst_sum >= (int64_t)1 << 31) return IPTQ_ERR_SCALE_RANGE;
    int M = 31 + std::max(0, top_bit_len((uint64_t)worst_sum) - 15);
    if (M > 40) M = 40;
    out->M = M;
    const int sh = M - (out_bits - 1);                        // Eq. (15): >> (M - (b - 1))
    out->f_shl = sh <= 32 ? 32 - sh : 0;
    out->p_shr = sh > 32 ? sh - 32 : 0;
    return IPTQ_OK;
}

static int gelu_prepare_with(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                             iptq_gelu_variant variant, double A, double Bf, iptq_gelu_consts* out);

int iptq_gelu_prepare(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                      iptq_gelu_variant variant, iptq_gelu_consts* out)
{
    const bool quartic = variant == IPTQ_GELU_POLY4;
    // |a|, |b| of Eq. (3) / of the second-order erf polynomial
    return gelu_prepare_with(in_scale, in_bits, out_scale, out_zp, out_bits, variant, quartic ? 0.019913 : 0.2888,
                             quartic ? 2.698088 : 1.769, out);
}

int iptq_gelu_prepare_coeffs(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits, double a,
                             double b, iptq_gelu_consts* out)
{
    if (!(a < 0.0) || !(b < 0.0)) return IPTQ_ERR_SCALE_RANGE;
    return gelu_prepare_with(in_scale, in_bits, out_scale, out_zp, out_bits, IPTQ_GELU_POLY4, -a, -b, out);
}

// Eq. (4): least squares of Eq. (3) against erf on a uniform grid over [lo, hi].  Both functions are odd, so the
// grid is folded to u = |x|; for a fixed b the optimum a is the ratio of two sums, which leaves a search in b:
// a scan over 400 values, then bisection on the sign of the slope between neighbours of the best cell.
int iptq_gelu_fit(double lo, double hi, int points, double* a_out, double* b_out, double* rms_out)
{
    if (!a_out || !b_out) return IPTQ_ERR_NULL;
    if (!(hi > lo) || points < 8 || points > (1 << 22)) return IPTQ_ERR_SHAPE;
    std::vector<double> u, tgt;
    u.reserve((size_t)points); tgt.reserve((size_t)points);
    for (int i = 0; i < points; ++i) {
        const double x = lo + (hi - lo) * (double)i / (double)(points - 1);
        if (x == 0.0) continue;
        u.push_back(std::fabs(x));
        tgt.push_back(std::erf(std::fabs(x)));
    }
    if (u.size() < 4) return IPTQ_ERR_SHAPE;
    auto a_of = [&](double b) {
        long double num = 0.0L, den = 0.0L;
        for (size_t i = 0; i < u.size(); ++i) {
            const double c = std::min(u[i], -b) + b, t = c * c * c * c;
            num += (long double)t * (tgt[i] - 1.0);
            den += (long double)t * t;
        }
        return den > 0.0L ? (double)(num / den) : 0.0;
    };
    auto loss = [&](double b) {
        const double a = a_of(b);
        long double ss = 0.0L;
        for (size_t i = 0; i < u.size(); ++i) {
            const double c = std::min(u[i], -b) + b, t = c * c * c * c;
            const double r = tgt[i] - (a * t + 1.0);
            ss += (long double)r * r;
        }
        return (double)ss;
    };
    const double b_lo = -8.0, b_hi = -0.25;
    const int cells = 400;
    int best = 0;
    double best_loss = loss(b_lo);
    for (int k = 1; k <= cells; ++k) {
        const double l = loss(b_lo + (b_hi - b_lo) * k / cells);
        if (l < best_loss) { best_loss = l; best = k; }
    }
    double l = b_lo + (b_hi - b_lo) * std::max(best - 1, 0) / cells;
    double r = b_lo + (b_hi - b_lo) * std::min(best + 1, cells) / cells;
    for (int it = 0; it < 100 && r - l > 1e-13; ++it) {      // ternary search: the loss is unimodal inside the cell pair
        const double m1 = l + (r - l) / 3.0, m2 = r - (r - l) / 3.0;
        if (loss(m1) < loss(m2)) r = m2; else l = m1;
    }
    const double b = 0.5 * (l + r);
    *a_out = a_of(b);
    *b_out = b;
    if (rms_out) *rms_out = std::sqrt(loss(b) / (double)u.size());
    return IPTQ_OK;
}

static int gelu_prepare_with(double in_scale, int in_bits, double out_scale, int out_zp, int out_bits,
                             iptq_gelu_variant variant, double A, double Bf, iptq_gelu_consts* out)
{
    if (!out) return IPTQ_ERR_NULL;
    if (in_bits < 8 || in_bits > 16 || out_bits < 4 || out_bits > 8) return IPTQ_ERR_BITS;
    if (!(in_scale > 0.0) || !(out_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    std::memset(out, 0, sizeof(*out));
    out->variant = (int32_t)variant; out->in_bits = in_bits;
    double y_scale;
    if (variant == IPTQ_GELU_POLY4 || variant == IPTQ_GELU_POLY2) {
        const bool quartic = variant == IPTQ_GELU_POLY4;
        const double sp = in_scale / std::sqrt(2.0);          // scale of x / sqrt(2)
        const double bq = std::floor(Bf / sp);
        if (!(bq >= 1.0 && bq < 32768.0)) return IPTQ_ERR_SCALE_RANGE;
        const int nb = top_bit_len((uint64_t)bq);
        const int sh2 = std::max(0, 2 * nb - 15);
        const double cd = quartic ? std::floor(1.0 / (A * sp * sp * sp * sp) / std::ldexp(1.0, 2 * sh2))
                                  : std::floor(1.0 / (A * sp * sp) / std::ldexp(1.0, sh2));
        if (!(cd >= 1.0 && cd < 1073741824.0)) return IPTQ_ERR_SCALE_RANGE;
        const int64_t C = (int64_t)cd;
        const int gs = std::max(0, top_bit_len((uint64_t)(2 * C)) + in_bits - 31);
        out->Bq = (int32_t)bq; out->sh2 = sh2; out->C = (int32_t)C; out->gs = gs;
        y_scale = in_scale * std::ldexp(1.0, gs) / (2.0 * (double)C);
    } else if (variant == IPTQ_GELU_SHIFT) {
        const double one = std::floor(1.0 / in_scale);
        if (!(one >= 8.0 && one < 16777216.0)) return IPTQ_ERR_SCALE_RANGE;
        const int64_t x0 = (int64_t)one;
        const int w = top_bit_len((uint64_t)x0);
        if (w > 14) return IPTQ_ERR_SCALE_RANGE;              // keeps 1.0 + e below 2^15
        out->x0 = (int32_t)x0; out->nsh = w < 14 ? 14 - w : 0; out->dcap = (int32_t)(34 * x0);
        magic_div31((uint32_t)x0, &out->div_mul, &out->div_shift);
        y_scale = in_scale * std::ldexp(1.0, -15);
    } else {
        return IPTQ_ERR_VARIANT;
    }
    return iptq_requant_prepare(y_scale / out_scale, out_zp, -(1 << (out_bits - 1)), (1 << (out_bits - 1)) - 1,
                                &out->out);
}

int iptq_layernorm_prepare(int dim, const float* gamma, const float* beta, double out_scale, int out_zp,
                           int out_bits, iptq_ln_variant variant, int32_t* gamma_q, int32_t* beta_q,
                           iptq_ln_consts* out)
{
    if (!gamma || !beta || !gamma_q || !beta_q || !out) return IPTQ_ERR_NULL;
    if (dim < 2 || dim > 3072 || (dim & 3)) return IPTQ_ERR_SHAPE;
    if (out_bits < 4 || out_bits > 8) return IPTQ_ERR_BITS;
    if (variant != IPTQ_LN_SHIFT && variant != IPTQ_LN_NEWTON && variant != IPTQ_LN_PTF) return IPTQ_ERR_VARIANT;
    if (!(out_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    double gmax = 0.0;
    for (int c = 0; c < dim; ++c) gmax = std::max(gmax, std::fabs((double)gamma[c]));
    if (!(gmax > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    const double sg = gmax / 32767.0;                         // per-tensor gamma scale
    const double sb = std::ldexp(sg, -10);                    // normalised values are Q10
    double gq_max = 0.0, bq_max = 0.0;
    for (int c = 0; c < dim; ++c) {
        const double g = std::floor((double)gamma[c] / sg + 0.5);
        const double b = std::floor((double)beta[c] / sb + 0.5);
        if (std::fabs(b) >= 1073741824.0) return IPTQ_ERR_SCALE_RANGE;
        gq_max = std::max(gq_max, std::fabs(g));
        bq_max = std::max(bq_max, std::fabs(b));
        gamma_q[c] = (int32_t)g;
        beta_q[c] = (int32_t)b;
    }
    // |n_c| <= 1.125 sqrt(dim) 2^10: n * gamma_q + beta_q has to stay inside int32
    if (1.125 * std::sqrt((double)dim) * 1024.0 * gq_max + bq_max >= 2147483648.0) return IPTQ_ERR_SCALE_RANGE;
    out->variant = (int32_t)variant; out->dim = dim;
    return iptq_requant_prepare(sb / out_scale, out_zp, -(1 << (out_bits - 1)), (1 << (out_bits - 1)) - 1, &out->out);
}

int iptq_workspace_init(void* ws, size_t ws_bytes, iptq_stream_t stream)
{
    if (!ws) return IPTQ_ERR_NULL;
    if (ws_bytes < kStatusBytes) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    return cuda_status(cudaMemsetAsync(ws, 0, kStatusBytes, stream));
}

int iptq_check(iptq_stream_t stream, const void* ws)
{
    if (cudaStreamSynchronize(stream) != cudaSuccess) return IPTQ_ERR_CUDA;
    if (!ws) return IPTQ_OK;
    StatusBlock sb;
    if (cudaMemcpy(&sb, ws, sizeof(sb), cudaMemcpyDeviceToHost) != cudaSuccess) return IPTQ_ERR_CUDA;
    return sb.timeout_flag ? IPTQ_ERR_TIMEOUT : IPTQ_OK;
}

const char* iptq_strerror(int status)
{
    switch (status) {
        case IPTQ_OK: return "ok";
        case IPTQ_ERR_NULL: return "a required pointer is NULL";
        case IPTQ_ERR_SHAPE: return "unsupported shape or size";
        case IPTQ_ERR_ALIGN: return "pointer or stride not aligned as required";
        case IPTQ_ERR_BITS: return "unsupported bit-width";
        case IPTQ_ERR_SCALE_RANGE: return "scale or ratio outside the representable range";
        case IPTQ_ERR_VARIANT: return "unknown approximation variant";
        case IPTQ_ERR_WORKSPACE: return "workspace missing or too small";
        case IPTQ_ERR_TIMEOUT: return "a bounded device-side wait timed out";
        case IPTQ_ERR_CUDA: return "a CUDA call failed";
        default: return "unknown iptq status";
    }
}

int64_t iptq_launch_count(void) { return iptq::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
