// Unified Metric (Sec. 3.5, Eqs. (16)-(20)): fp64 reference layers and error reductions on the device, the
// Softplus / harmonic-mean scoring and the operation-count model on the host.
#include <climits>
#include <cmath>

#include "iptq_common.cuh"

namespace iptq {

constexpr unsigned kAll = 0xffffffffu;
constexpr int kMetricThreads = 256;
constexpr int kMetricMaxBlocks = IPTQ_METRIC_WORK_BYTES / 16;      // one (sum X^2, sum err^2) pair per CTA

// Butterfly sum: every lane ends with the same value, and the order of the additions is fixed.
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(kAll, v, o);
    return v;
}

// CTA partial -> work[2 * blockIdx.x ..]; warps are added in index order by thread 0.
__device__ __forceinline__ void block_store_partial(double a, double b, double* work)
{
    __shared__ double sh[2][kMetricThreads / 32];
    a = warp_sum(a);
    b = warp_sum(b);
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { sh[0][w] = a; sh[1][w] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double ta = 0.0, tb = 0.0;
        for (int i = 0; i < kMetricThreads / 32; ++i) { ta += sh[0][i]; tb += sh[1][i]; }
        work[2 * blockIdx.x] = ta;
        work[2 * blockIdx.x + 1] = tb;
    }
}

// One warp adds the CTA partials: lane i takes partials i, i + 32, ... in order, then the butterfly.
__global__ void __launch_bounds__(32)
metric_finish_kernel(const double* __restrict__ work, int nblocks, double* __restrict__ sums)
{
    grid_dep_wait();
    double a = 0.0, b = 0.0;
    for (int i = threadIdx.x; i < nblocks; i += 32) { a += work[2 * i]; b += work[2 * i + 1]; }
    a = warp_sum(a);
    b = warp_sum(b);
    if (threadIdx.x == 0) { sums[0] = a; sums[1] = b; }
}

// Softmax: a warp per row.  X_j = exp(z_j - z_max) / sum_k exp(z_k - z_max) with z = in_scale * score (fp64).
__global__ void __launch_bounds__(kMetricThreads)
metric_softmax_kernel(const int32_t* __restrict__ scores, const uint8_t* __restrict__ probs, int64_t rows, int n,
                      double in_scale, double out_step, double* __restrict__ work)
{
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (kMetricThreads >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (kMetricThreads >> 5);
    double ax2 = 0.0, ae2 = 0.0;
    for (int64_t row = warp; row < rows; row += nwarps) {
        const int32_t* sr = scores + row * n;
        const uint8_t* pr = probs + row * n;
        int mx = INT_MIN;
        for (int j = lane; j < n; j += 32) mx = max(mx, __ldg(sr + j));
        mx = __reduce_max_sync(kAll, mx);
        const double zmax = (double)mx * in_scale;
        double den = 0.0;
        for (int j = lane; j < n; j += 32) den += exp((double)__ldg(sr + j) * in_scale - zmax);
        den = warp_sum(den);
        for (int j = lane; j < n; j += 32) {
            const double X = exp((double)__ldg(sr + j) * in_scale - zmax) / den;
            const unsigned pb = __ldg(pr + j);
            // out_step = 0: the byte is a logarithm-candidate code, 2^-code (255: zero) built from the exponent bits
            const double Qd = out_step != 0.0 ? (double)pb * out_step
                                              : (pb == IPTQ_LOG2_ZERO ? 0.0 : __longlong_as_double((long long)(1023 - (int)min(pb, 15u)) << 52));
            const double d = X - Qd;
            ax2 += X * X;
            ae2 += d * d;
        }
    }
    block_store_partial(ax2, ae2, work);
}

// GELU: element-wise.  X = v/2 (1 + erf(v / sqrt 2)), v = in_scale * x.
__global__ void __launch_bounds__(kMetricThreads)
metric_gelu_kernel(const int32_t* __restrict__ x, const int8_t* __restrict__ y, int64_t n, double in_scale,
                   double out_scale, int out_zp, double* __restrict__ work)
{
    grid_dep_wait();
    const int64_t stride = (int64_t)gridDim.x * kMetricThreads;
    double ax2 = 0.0, ae2 = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * kMetricThreads + threadIdx.x; i < n; i += stride) {
        const double v = (double)__ldg(x + i) * in_scale;
        const double X = 0.5 * v * (1.0 + erf(v / 1.4142135623730951));
        const double d = X - (double)((int)__ldg(y + i) - out_zp) * out_scale;
        ax2 += X * X;
        ae2 += d * d;
    }
    block_store_partial(ax2, ae2, work);
}

// LayerNorm: a warp per row.  Mean from the exact integer sum, biased variance, no epsilon.
__global__ void __launch_bounds__(kMetricThreads)
metric_layernorm_kernel(const int8_t* __restrict__ x, const int8_t* __restrict__ y, int64_t rows, int D,
                        const float* __restrict__ gamma, const float* __restrict__ beta,
                        const uint8_t* __restrict__ ptf, double out_scale, int out_zp, double* __restrict__ work)
{
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (kMetricThreads >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (kMetricThreads >> 5);
    double ax2 = 0.0, ae2 = 0.0;
    for (int64_t row = warp; row < rows; row += nwarps) {
        const int8_t* xr = x + row * D;
        const int8_t* yr = y + row * D;
        long long s1 = 0;
        for (int j = lane; j < D; j += 32) s1 += (long long)((int)xr[j] << (ptf ? (int)ptf[j] : 0));
#pragma unroll
        for (int o = 16; o; o >>= 1) s1 += __shfl_xor_sync(kAll, s1, o);
        const double mu = (double)s1 / (double)D;
        double ss = 0.0;
        for (int j = lane; j < D; j += 32) {
            const double c = (double)((int)xr[j] << (ptf ? (int)ptf[j] : 0)) - mu;
            ss += c * c;
        }
        const double sd = sqrt(warp_sum(ss) / (double)D);
        for (int j = lane; j < D; j += 32) {
            const double b = (double)__ldg(beta + j);
            double X = b;
            if (sd != 0.0) X = ((double)((int)xr[j] << (ptf ? (int)ptf[j] : 0)) - mu) / sd * (double)__ldg(gamma + j) + b;
            const double d = X - (double)((int)yr[j] - out_zp) * out_scale;
            ax2 += X * X;
            ae2 += d * d;
        }
    }
    block_store_partial(ax2, ae2, work);
}

static int metric_grid(int64_t units_per_block_total)
{
    const int64_t cap = std::min<int64_t>((int64_t)sm_count() * 8, kMetricMaxBlocks);
    return (int)std::max<int64_t>(1, std::min<int64_t>(units_per_block_total, cap));
}

static int metric_args_ok(const void* sums, const void* work)
{
    if (!sums || !work) return IPTQ_ERR_NULL;
    if (!aligned16(sums) || !aligned16(work)) return IPTQ_ERR_ALIGN;
    return IPTQ_OK;
}

static int metric_finish(double* work, int grid, double* sums, cudaStream_t st)
{
    launch_kernel(metric_finish_kernel, 1, 32, 0, st, (const double*)work, grid, sums);
    note_launch(2);
    return last_launch_status();
}

}  // namespace iptq

using namespace iptq;

extern "C" {

int iptq_metric_softmax(const int32_t* scores, const uint8_t* probs, int64_t rows, int row_len, double in_scale,
                        int out_bits, double* sums, void* work, iptq_stream_t stream)
{
    int rc = metric_args_ok(sums, work);
    if (rc != IPTQ_OK) return rc;
    if (rows < 0 || row_len < 1 || row_len > 1024) return IPTQ_ERR_SHAPE;
    if (out_bits != IPTQ_PROBS_LOG2 && (out_bits < 4 || out_bits > 8)) return IPTQ_ERR_BITS;
    if (!(in_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    if (rows > 0 && (!scores || !probs)) return IPTQ_ERR_NULL;
    const int grid = metric_grid((rows + 7) / 8);
    const double out_step = out_bits == IPTQ_PROBS_LOG2 ? 0.0 : 1.0 / (double)(1 << (out_bits - 1));
    launch_kernel(metric_softmax_kernel, grid, kMetricThreads, 0, stream, scores, probs, rows, row_len, in_scale,
                  out_step, (double*)work);
    return metric_finish((double*)work, grid, sums, stream);
}

int iptq_metric_gelu(const int32_t* x, const int8_t* y, int64_t n, double in_scale, double out_scale, int out_zp,
                     double* sums, void* work, iptq_stream_t stream)
{
    int rc = metric_args_ok(sums, work);
    if (rc != IPTQ_OK) return rc;
    if (n < 0) return IPTQ_ERR_SHAPE;
    if (!(in_scale > 0.0) || !(out_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    if (n > 0 && (!x || !y)) return IPTQ_ERR_NULL;
    const int grid = metric_grid((n + 4 * kMetricThreads - 1) / (4 * kMetricThreads));
    launch_kernel(metric_gelu_kernel, grid, kMetricThreads, 0, stream, x, y, n, in_scale, out_scale, out_zp,
                  (double*)work);
    return metric_finish((double*)work, grid, sums, stream);
}

int iptq_metric_layernorm(const int8_t* x, const int8_t* y, int64_t rows, int dim, const float* gamma,
                          const float* beta, const uint8_t* ptf_shift, double out_scale, int out_zp, double* sums,
                          void* work, iptq_stream_t stream)
{
    int rc = metric_args_ok(sums, work);
    if (rc != IPTQ_OK) return rc;
    if (rows < 0 || dim < 4 || dim > 3072 || (dim & 3)) return IPTQ_ERR_SHAPE;
    if (!(out_scale > 0.0)) return IPTQ_ERR_SCALE_RANGE;
    if (!gamma || !beta || (rows > 0 && (!x || !y))) return IPTQ_ERR_NULL;
    const int grid = metric_grid((rows + 7) / 8);
    launch_kernel(metric_layernorm_kernel, grid, kMetricThreads, 0, stream, x, y, rows, dim, gamma, beta, ptf_shift,
                  out_scale, out_zp, (double*)work);
    return metric_finish((double*)work, grid, sums, stream);
}

// ---------------------------------------------------------------- host: Eqs. (16)-(18), (20)

double iptq_softplus(double v)
{
    // log(1 + e^v) = max(v, 0) + log1p(e^-|v|): no overflow for large v, no cancellation for small
    return (v > 0.0 ? v : 0.0) + log1p(exp(-fabs(v)));
}

double iptq_sqnr_db(double sum_x2, double sum_err2)
{
    if (sum_err2 == 0.0) return INFINITY;
    return 10.0 * log10(sum_x2 / sum_err2);
}

double iptq_metric_term(double sqnr_db, double perturbation, double op_count, double c_unit)
{
    const double nq = iptq_softplus(sqnr_db);
    const double inv_nq = std::isinf(nq) ? 0.0 : 1.0 / nq;
    return 3.0 / (inv_nq + iptq_softplus(perturbation) + iptq_softplus(op_count / c_unit));
}

// Operations per element / per row of the integer definitions in this library: one per binary add, subtract,
// multiply, divide, shift or mask and per comparison (min, max, |.|, sign and leading-one position count as one);
// sign flips, copies, constants prepared before inference and values that are the same for a whole row are not
// per-element operations.  Softmax: max, distance, clamp (3), Eq. (7) (4), Eq. (8) (3), Phi and + x0 (6; Shiftmax
// 2), Eq. (9) (2), sum (1), Eq. (15) (2), one division per row; the polynomial exponential has 15, the logarithm
// candidate 13 for exponential and sum plus 12 for the rounded ratio and its rounded logarithm.  GELU: clamp (2),
// |x|, min, subtract (3), two squares and a shift (3; second order 2), C - (.), sign, times, + C (4), shift and
// x * G (2), requantisation (7: multiply, high word, round, shift, zero point, two clamps; also the LayerNorm's);
// the shift-based sigmoid form has 34.  LayerNorm: sums (3), D x - sum (2), reciprocal multiply and shift (2),
// gamma and beta (2), requantisation (7), one more shift with power-of-two factors; per row the variance (3), the
// start value of the square root (4), its steps (10 fixed steps of 3 operations; 5 steps of 4 when iterated to
// convergence, the most the rows of the workloads need) and the reciprocal (1).
double iptq_op_count(int layer_kind, int variant, int64_t rows, int row_len)
{
    if (variant < 0 || variant > (layer_kind == IPTQ_LAYER_SOFTMAX ? 3 : 2) || rows < 0 || row_len < 0) return -1.0;
    const double r = (double)rows, n = (double)rows * (double)row_len;
    switch (layer_kind) {
        case IPTQ_LAYER_SOFTMAX: {
            static const double per_elem[4] = {21.0, 17.0, 15.0, 25.0};
            return per_elem[variant] * n + r;
        }
        case IPTQ_LAYER_GELU: {
            static const double per_elem[3] = {21.0, 20.0, 34.0};
            return per_elem[variant] * n;
        }
        case IPTQ_LAYER_LAYERNORM: {
            static const double per_elem[3] = {16.0, 16.0, 17.0};
            static const double per_row[3] = {38.0, 28.0, 28.0};
            return per_elem[variant] * n + per_row[variant] * r;
        }
        default: return -1.0;
    }
}

int iptq_metric_select(const double* terms, int n)
{
    if (!terms || n < 1) return -1;
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (terms[i] > terms[best]) best = i;
    return best;
}

}  // extern "C"
