// Stand-alone integer Softmax / GELU / LayerNorm kernels (row- and element-wise, HBM/ALU bound).
#include <climits>
#include <type_traits>

#include "iptq_common.cuh"

namespace iptq {

constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------------------------------------
// Softmax: one warp per row, the row lives in registers (NITER values per lane), row max / row sum
// by warp reduction, one fp64 division per row for floor(2^M / sum).
// ------------------------------------------------------------------------------------------------
struct SoftmaxDev {
    ExpDev ex;
    int M, f_shl, p_shr;
    int tab_n;                 // entries of the exponential table, 0: evaluate
    const uint16_t* tab_src;   // the table in device memory, or null: each CTA builds it
};

template <int VARIANT, int NITER, bool HAS_BIAS, bool PSHR>
__global__ void __launch_bounds__(256)
softmax_rows_kernel(const int32_t* __restrict__ scores, uint8_t* __restrict__ probs, int64_t rows, int n,
                    const int32_t* __restrict__ bias, int64_t bias_period, const SoftmaxDev c)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    grid_dep_launch();
    grid_dep_wait();
    for (int64_t row = warp; row < rows; row += nwarps) {
        const int32_t* sr = scores + row * n;
        const int32_t* br = HAS_BIAS ? bias + (row % bias_period) * n : nullptr;
        int v[NITER];
        int mx = INT_MIN;
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            const int j = lane + 32 * k;
            int s = kNoScore;                                  // lanes past the row end
            if (j < n) {
                s = __ldcs(sr + j);
                if (HAS_BIAS) s += __ldg(br + j);
            }
            v[k] = s;
            mx = max(mx, s);
        }
        mx = __reduce_max_sync(kFull, mx);                      // Eq. (6)
        unsigned sum = 0;
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            const unsigned e = exp_core_nd<VARIANT>(exp_distance(mx, v[k]), c.ex);
            v[k] = (int)e;
            sum += e;
        }
        sum = __reduce_add_sync(kFull, sum);
        uint8_t* pr = probs + row * n;
        if (VARIANT == IPTQ_SM_LOG2) {
#pragma unroll
            for (int k = 0; k < NITER; ++k) {
                const int j = lane + 32 * k;
                if (j < n) __stcs(pr + j, (uint8_t)log2_code(sum, (unsigned)v[k]));
            }
            continue;
        }
        const unsigned f = intdiv_factor(sum, c.M) << c.f_shl;  // Eq. (15)
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            const int j = lane + 32 * k;
            unsigned pv = __umulhi(f, (unsigned)v[k]);
            if (PSHR) pv >>= c.p_shr;
            if (j < n) __stcs(pr + j, (uint8_t)pv);
        }
    }
}

// Tabulated form: the integer exponential (Eq. (9), or the second-order polynomial of the other two candidates)
// depends on max - s alone, is 0 beyond a few multiples of x0 and below 2^16, so each CTA keeps it as a table in
// shared memory (copied from the one iptq_softmax_table() wrote, or
// built here with the same arithmetic) and a score costs one 16-bit shared-memory load instead of the evaluation.
// Two CTAs of 1024 threads per SM: 32 registers per thread, 64 warps to cover the load latency.
constexpr int kSmTabThreads = 1024;
constexpr int kSmTabMaxBytes = 2 * IPTQ_SOFTMAX_TABLE_MAX;
// Smallest inputs for which the table pays for its set-up (copied from device memory / built by every CTA).
constexpr int64_t kSmTabMinElemsCopy = 1 << 20, kSmTabMinElemsBuild = 16 << 20;

template <int VARIANT, int NITER, bool HAS_BIAS, bool PSHR>
__global__ void __launch_bounds__(kSmTabThreads, 2)
softmax_rows_tab_kernel(const int32_t* __restrict__ scores, uint8_t* __restrict__ probs, int64_t rows, int n,
                        const int32_t* __restrict__ bias, int64_t bias_period, const SoftmaxDev c, int tab_n,
                        const uint16_t* __restrict__ tab_src)
{
    constexpr int TPB = kSmTabThreads;
    extern __shared__ __align__(16) uint16_t exp_tab[];
    if (tab_src) {
        // Written by iptq_softmax_table() and fenced there, so it may be read ahead of the dependency wait.
        const int4* src = reinterpret_cast<const int4*>(tab_src);
        int4* dst = reinterpret_cast<int4*>(exp_tab);
        for (int i = threadIdx.x; i < (tab_n + 8) / 8; i += TPB) dst[i] = __ldg(src + i);
    } else {
        for (int d = threadIdx.x; d <= tab_n; d += TPB)
            exp_tab[d] = d < tab_n ? (uint16_t)exp_core_nd<VARIANT>(-d, c.ex) : (uint16_t)0;
    }
    __syncthreads();
    const uint32_t tab_addr = (uint32_t)__cvta_generic_to_shared(exp_tab);
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (TPB >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (TPB >> 5);
    grid_dep_launch();
    grid_dep_wait();
    // Only the last 32-column step of a row can pass the row end.
    const bool tail_ok = lane + 32 * (NITER - 1) < n;
    auto load_row = [&](int64_t row, int (&v)[NITER]) {
        const int32_t* sr = scores + row * n + lane;
        const int32_t* br = HAS_BIAS ? bias + (row % bias_period) * n + lane : nullptr;
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            int s = kNoScore;                                  // lanes past the row end
            if (k < NITER - 1 || tail_ok) {
                s = __ldcs(sr + 32 * k);
                if (HAS_BIAS) s += __ldg(br + 32 * k);
            }
            v[k] = s;
        }
    };
    auto finish_row = [&](int64_t row, int (&v)[NITER]) {
        int mx = INT_MIN;
#pragma unroll
        for (int k = 0; k < NITER; ++k) mx = max(mx, v[k]);
        mx = __reduce_max_sync(kFull, mx);                      // Eq. (6)
        unsigned sum = 0;
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            const unsigned d = min((unsigned)mx - (unsigned)v[k], (unsigned)tab_n);   // exact for any int32 pair
            unsigned e;
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(e) : "r"(tab_addr + 2u * d));
            v[k] = (int)e;
            sum += e;
        }
        sum = __reduce_add_sync(kFull, sum);
        uint8_t* pr = probs + row * n + lane;
        if constexpr (VARIANT == IPTQ_SM_LOG2) {
#pragma unroll
            for (int k = 0; k < NITER; ++k)
                if (k < NITER - 1 || tail_ok) __stcs(pr + 32 * k, (uint8_t)log2_code(sum, (unsigned)v[k]));
            return;
        }
        const unsigned f = intdiv_factor(sum, c.M) << c.f_shl;  // Eq. (15)
#pragma unroll
        for (int k = 0; k < NITER; ++k) {
            unsigned pv = __umulhi(f, (unsigned)v[k]);
            if (PSHR) pv >>= c.p_shr;
            if (k < NITER - 1 || tail_ok) __stcs(pr + 32 * k, (uint8_t)pv);
        }
    };
    int v[NITER];
    for (int64_t row = warp; row < rows; row += nwarps) {
        load_row(row, v);
        finish_row(row, v);
    }
}

template <int VARIANT, int NITER>
static int launch_softmax2(const int32_t* s, uint8_t* p, int64_t rows, int n, const int32_t* bias, int64_t period,
                           const SoftmaxDev& c, cudaStream_t st)
{
    if constexpr (NITER <= 8)
    if (c.tab_n > 0 && ((c.tab_n + 8) & ~7) <= IPTQ_SOFTMAX_TABLE_MAX &&
        rows * n >= (c.tab_src ? kSmTabMinElemsCopy : kSmTabMinElemsBuild)) {
        // Tabulated exponential: worth the per-CTA table set-up once every warp has several rows.
        const size_t smem = (2 * ((size_t)c.tab_n + 1) + 15) & ~(size_t)15;
        const int wpc = kSmTabThreads / 32;
        const int grid = (int)std::min<int64_t>((rows + wpc - 1) / wpc, (int64_t)sm_count() * 2);
#define IPTQ_SM_TAB(HB, PS)                                                                                         \
        do {                                                                                                        \
            auto kern = softmax_rows_tab_kernel<VARIANT, NITER, HB, PS>;                                            \
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmTabMaxBytes);              \
            launch_kernel(kern, grid, kSmTabThreads, smem, st, s, p, rows, n, bias, period, c, c.tab_n, c.tab_src); \
        } while (0)
        if (bias) { if (c.p_shr) IPTQ_SM_TAB(true, true); else IPTQ_SM_TAB(true, false); }
        else      { if (c.p_shr) IPTQ_SM_TAB(false, true); else IPTQ_SM_TAB(false, false); }
#undef IPTQ_SM_TAB
        note_launch();
        return last_launch_status();
    }
    const int threads = 256;
    const int64_t want = (rows + 7) / 8;
    const int grid = (int)std::min<int64_t>(want, (int64_t)sm_count() * 8);
    if (bias) {
        if (c.p_shr) launch_kernel(softmax_rows_kernel<VARIANT, NITER, true, true>, grid, threads, 0, st, s, p, rows, n, bias, period, c);
        else         launch_kernel(softmax_rows_kernel<VARIANT, NITER, true, false>, grid, threads, 0, st, s, p, rows, n, bias, period, c);
    } else {
        if (c.p_shr) launch_kernel(softmax_rows_kernel<VARIANT, NITER, false, true>, grid, threads, 0, st, s, p, rows, n, bias, period, c);
        else         launch_kernel(softmax_rows_kernel<VARIANT, NITER, false, false>, grid, threads, 0, st, s, p, rows, n, bias, period, c);
    }
    note_launch();
    return last_launch_status();
}

template <int VARIANT>
static int launch_softmax1(const int32_t* s, uint8_t* p, int64_t rows, int n, const int32_t* bias, int64_t period,
                           const SoftmaxDev& c, cudaStream_t st)
{
    const int it = (n + 31) / 32;
    switch (it) {
        case 1: return launch_softmax2<VARIANT, 1>(s, p, rows, n, bias, period, c, st);
        case 2: return launch_softmax2<VARIANT, 2>(s, p, rows, n, bias, period, c, st);
        case 3: return launch_softmax2<VARIANT, 3>(s, p, rows, n, bias, period, c, st);
        case 4: return launch_softmax2<VARIANT, 4>(s, p, rows, n, bias, period, c, st);
        case 5: return launch_softmax2<VARIANT, 5>(s, p, rows, n, bias, period, c, st);
        case 6: return launch_softmax2<VARIANT, 6>(s, p, rows, n, bias, period, c, st);
        case 7: return launch_softmax2<VARIANT, 7>(s, p, rows, n, bias, period, c, st);
        case 8: return launch_softmax2<VARIANT, 8>(s, p, rows, n, bias, period, c, st);
        default:
            if (it <= 16) return launch_softmax2<VARIANT, 16>(s, p, rows, n, bias, period, c, st);
            return launch_softmax2<VARIANT, 32>(s, p, rows, n, bias, period, c, st);
    }
}

// ------------------------------------------------------------------------------------------------
// GELU: element-wise; each warp iteration covers 512 elements with four coalesced 16-byte loads per
// lane and four coalesced 4-byte stores.
// ------------------------------------------------------------------------------------------------
template <int VARIANT, bool SAT8>
__device__ __forceinline__ unsigned gelu4(int4 a, const GeluDev& c)
{
    if (SAT8)
        return pack4_sat_s8(requant_nosat(gelu_core<VARIANT>(a.x, c), c.out), requant_nosat(gelu_core<VARIANT>(a.y, c), c.out),
                            requant_nosat(gelu_core<VARIANT>(a.z, c), c.out), requant_nosat(gelu_core<VARIANT>(a.w, c), c.out));
    return pack4_s8(requant_full(gelu_core<VARIANT>(a.x, c), c.out), requant_full(gelu_core<VARIANT>(a.y, c), c.out),
                    requant_full(gelu_core<VARIANT>(a.z, c), c.out), requant_full(gelu_core<VARIANT>(a.w, c), c.out));
}

template <int VARIANT, bool SAT8>
__global__ void __launch_bounds__(256)
gelu_kernel(const int32_t* __restrict__ x, int8_t* __restrict__ y, int64_t n, const GeluDev c)
{
    grid_dep_launch();
    grid_dep_wait();
    const int64_t nvec = n >> 2;                                 // int4 / 4-byte groups
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int4* xv = reinterpret_cast<const int4*>(x);
    unsigned* yv = reinterpret_cast<unsigned*>(y);
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    // four independent groups per iteration for memory-level parallelism
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        int4 a[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] = __ldcs(xv + i + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) __stcs(yv + i + u * stride, gelu4<VARIANT, SAT8>(a[u], c));
    }
    for (; i < nvec; i += stride) yv[i] = gelu4<VARIANT, SAT8>(__ldcs(xv + i), c);
    // ragged tail (n % 4 elements)
    const int64_t t = (nvec << 2) + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n) y[t] = (int8_t)requant_full(gelu_core<VARIANT>(x[t], c), c.out);
}

// Tabulated form: with consts->table set (iptq_gelu_table) the whole function is a 64 KB table, copied once per CTA
// into shared memory; an element then costs a clamp to 16 bits and one byte load.  Two CTAs of 1024 threads per SM.
constexpr int kGeluTabThreads = 1024;

__global__ void __launch_bounds__(kGeluTabThreads, 2)
gelu_tab_kernel(const int32_t* __restrict__ x, int8_t* __restrict__ y, int64_t n, const int8_t* __restrict__ table)
{
    extern __shared__ __align__(16) int8_t gelu_tab[];
    {
        // written and fenced by iptq_gelu_table(): safe to read ahead of the dependency wait
        const int4* src = reinterpret_cast<const int4*>(table);
        int4* dst = reinterpret_cast<int4*>(gelu_tab);
        for (int i = threadIdx.x; i < IPTQ_GELU_TABLE_SIZE / 16; i += kGeluTabThreads) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    const uint32_t mid = (uint32_t)__cvta_generic_to_shared(gelu_tab) + 32768u;      // address of table[0 + 32768]
    grid_dep_launch();
    grid_dep_wait();
    auto look = [&](int v) -> int {
        v = max(-32768, min(32767, v));
        int r;
        asm volatile("ld.shared.s8 %0, [%1];" : "=r"(r) : "r"(mid + (uint32_t)v));
        return r;
    };
    auto four = [&](int4 a) -> unsigned { return pack4_sat_s8(look(a.x), look(a.y), look(a.z), look(a.w)); };
    const int64_t nvec = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * kGeluTabThreads;
    const int4* xv = reinterpret_cast<const int4*>(x);
    unsigned* yv = reinterpret_cast<unsigned*>(y);
    int64_t i = (int64_t)blockIdx.x * kGeluTabThreads + threadIdx.x;
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        int4 a[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] = __ldcs(xv + i + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) __stcs(yv + i + u * stride, four(a[u]));
    }
    for (; i < nvec; i += stride) yv[i] = four(__ldcs(xv + i));
    const int64_t t = (nvec << 2) + (int64_t)blockIdx.x * kGeluTabThreads + threadIdx.x;
    if (t < n) y[t] = (int8_t)look(x[t]);
}

// table[x + 32768] = integer GELU of x for every 16-bit x (the input clamp to in_bits is part of gelu_core)
template <int VARIANT>
__global__ void __launch_bounds__(256)
gelu_table_kernel(int8_t* __restrict__ table, const GeluDev c)
{
    grid_dep_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    table[i] = (int8_t)requant_full(gelu_core<VARIANT>(i - 32768, c), c.out);
}

// table[d] = integer exponential of -d for d < n, 0 for n <= d < n_pad
template <int VARIANT>
__global__ void __launch_bounds__(256)
softmax_table_kernel(uint16_t* __restrict__ table, int n, int n_pad, const ExpDev ex)
{
    grid_dep_wait();
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d < n_pad) table[d] = d < n ? (uint16_t)exp_core_nd<VARIANT>(-d, ex) : (uint16_t)0;
}

// Launched without programmatic serialisation behind a table kernel: it starts only once the table is complete
// and visible, so a later kernel that reads the table ahead of its own dependency wait cannot overtake the writer.
__global__ void stream_fence_kernel() {}

// ------------------------------------------------------------------------------------------------
// LayerNorm: a warp takes a few rows at a time; the rows live in registers as packed int8 words (NW per lane).
// ------------------------------------------------------------------------------------------------
struct LnDev {
    int variant, dim;
    RequantDev out;
};

__device__ __forceinline__ unsigned long long isqrt_floor(unsigned long long V)
{
    // V >= 1.  Estimate from the hardware reciprocal square root (about 22 good bits), then walk to the exact
    // floor with the remainder e = V - s^2: one or two steps for the 44-bit values of this kernel.
    const double vd = (double)(long long)V;
    double y;
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(vd));
    long long s = (long long)(vd * y);
    long long e = (long long)V - s * s;
    while (e < 0) { --s; e += 2 * s + 1; }
    while (e > 2 * s) { e -= 2 * s + 1; ++s; }
    return (unsigned long long)s;
}

// floor(a / b) for integers 0 <= a < 2^53, 1 <= b with a / b * b <= 2^53: the correctly rounded fp64 quotient of
// a non-integer a / b lies at least 1 / b below the next integer, i.e. 2^-53 relatively away whenever the
// quotient times b stays below 2^53, so truncation gives the exact floor.
__device__ __forceinline__ double floor_div_f64(double a, double b) { return floor(a / b); }

__device__ __forceinline__ unsigned long long isqrt_variant(unsigned long long V, int variant)
{
    if (V == 0) return 0;
    const unsigned long long s = isqrt_floor(V);
    if (variant != IPTQ_LN_SHIFT) return s;
    // Fixed 10 steps of r <- (r + V / r) >> 1 from 2^ceil(bitlen(V) / 2), no convergence test.  From a start
    // within a factor 2 of sqrt(V) the recurrence reaches floor(sqrt V) in at most 7 steps and then stays there,
    // except when V + 1 is a perfect square, where it alternates between s and s + 1: only then is the
    // recurrence actually run (in fp64, every intermediate is an exact integer below 2^53).
    if ((s + 1) * (s + 1) != V + 1) return s;
    const int w = 64 - __clzll((long long)V);
    double r = (double)(1ull << ((w + 1) >> 1));
    const double Vd = (double)V;
#pragma unroll 1
    for (int it = 0; it < 10; ++it) r = floor((r + floor_div_f64(Vd, r)) * 0.5);
    return (unsigned long long)r;
}

// One warp handles RW rows at a time.  The per-row scalar work (variance, integer square root, reciprocal) is the
// long dependent chain of this kernel; lane r of the warp runs it for row r, so its cost is shared by RW rows.
// EXACT: the row is exactly 32 * NW words, so no lane ever needs a bounds predicate.  ZPF: the output zero point is
// folded into the rounding constant (c.out.rnd already holds rnd + (zp << shift), c.out.zp is 0).  PREFETCH: the rows
// of a warp's next group are loaded before the current group is processed (pays off once a warp has several groups).
template <int NW, int RW, bool PTF, bool SAT8, bool EXACT, bool ZPF, bool PREFETCH>
__global__ void __launch_bounds__(256)
layernorm_rows_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int64_t rows,
                      const int32_t* __restrict__ gamma_q, const int32_t* __restrict__ beta_q,
                      const uint8_t* __restrict__ ptf, const LnDev c)
{
    const int lane = threadIdx.x & 31;
    const int D = c.dim;
    grid_dep_launch();
    const int words = D >> 2;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t groups = (rows + RW - 1) / RW;
    // per-lane channel parameters stay in registers across rows when they fit
    constexpr bool KEEP = NW <= 8;
    int4 g[KEEP ? NW : 1], b[KEEP ? NW : 1];
    unsigned sh[NW];
#pragma unroll
    for (int k = 0; k < NW; ++k) {
        const int wi = lane + 32 * k;
        sh[k] = 0;
        if (EXACT || wi < words) {
            if (KEEP) {
                g[k] = __ldg(reinterpret_cast<const int4*>(gamma_q) + wi);
                b[k] = __ldg(reinterpret_cast<const int4*>(beta_q) + wi);
            }
            if (PTF) sh[k] = __ldg(reinterpret_cast<const unsigned*>(ptf) + wi);
        }
    }
    grid_dep_wait();                                // gamma / beta above are static; the rows come from the previous kernel
    // the rows of the next group are fetched while the current group is processed
    auto fetch = [&](int64_t grp, int (&dst)[RW][NW]) {
        const int64_t row0 = grp * RW;
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            const bool live = grp < groups && row0 + r < rows;
            const int* xr = reinterpret_cast<const int*>(x + (live ? row0 + r : 0) * D);
#pragma unroll
            for (int k = 0; k < NW; ++k) {
                const int wi = lane + 32 * k;
                dst[r][k] = (live && (EXACT || wi < words)) ? __ldcs(xr + wi) : 0;
            }
        }
    };
    int wn[PREFETCH ? RW : 1][PREFETCH ? NW : 1];
    if constexpr (PREFETCH) fetch(warp, wn);
    for (int64_t grp = warp; grp < groups; grp += nwarps) {
        const int64_t row0 = grp * RW;
        int w[RW][NW];
        if constexpr (PREFETCH) {
#pragma unroll
            for (int r = 0; r < RW; ++r)
#pragma unroll
                for (int k = 0; k < NW; ++k) w[r][k] = wn[r][k];
            fetch(grp + nwarps, wn);
        } else {
            fetch(grp, w);
        }
        int my_s1 = 0;
        unsigned my_s2 = 0;
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            int s1 = 0;
            unsigned s2 = 0;
#pragma unroll
            for (int k = 0; k < NW; ++k) {
                if (!PTF) {
                    s1 = __dp4a(w[r][k], 0x01010101, s1);
                    s2 = (unsigned)__dp4a(w[r][k], w[r][k], (int)s2);
                } else {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int xv = ((int)(int8_t)(w[r][k] >> (8 * t))) << ((sh[k] >> (8 * t)) & 3);
                        s1 += xv;
                        s2 += (unsigned)(xv * xv);
                    }
                }
            }
            s1 = __reduce_add_sync(kFull, s1);
            s2 = __reduce_add_sync(kFull, s2);
            if (lane == r) { my_s1 = s1; my_s2 = s2; }
        }
        // lane r: statistics of row r (the other lanes run the same instructions on zeros)
        const long long V = (long long)D * (long long)my_s2 - (long long)my_s1 * (long long)my_s1;   // D^2 var, exact
        const unsigned long long rt = isqrt_variant((unsigned long long)V, c.variant);                // D * std
        const long long F = rt ? (long long)floor_div_f64(1099511627776.0, (double)rt) : 0;          // floor(2^40 / rt)
        // (u F) >> 30 = hi32(u * 4F) when 4F fits in 32 bits (rows whose D * std exceeds 2^11: all but near-constant rows)
        const int my_narrow = F < (1ll << 29);
        const int my_F4 = (int)(F << 2);
#pragma unroll
        for (int r = 0; r < RW; ++r) {
            if (row0 + r >= rows) break;                                        // warp-uniform
            const int s1 = __shfl_sync(kFull, my_s1, r);
            const int F4 = __shfl_sync(kFull, my_F4, r);
            const bool narrow = __shfl_sync(kFull, my_narrow, r) != 0;
            const long long Fr = narrow ? 0 : (((long long)__shfl_sync(kFull, (int)(F >> 32), r) << 32) |
                                               (unsigned)__shfl_sync(kFull, (int)(unsigned)F, r));
            int* yr = reinterpret_cast<int*>(y + (row0 + r) * D);
            const int om = c.out.mult, ornd = c.out.rnd, osh = c.out.shift, ozp = c.out.zp;
            auto emit = [&](auto narrow_c) {
                constexpr bool NARROW = decltype(narrow_c)::value;
                auto elem = [&](int xv, unsigned shw, int t, int gg, int bb) -> int {
                    if (PTF) xv <<= ((shw >> (8 * t)) & 3);
                    const int u = D * xv - s1;                                   // D (x - mean)
                    const int nq = NARROW ? __mulhi(u, F4) : (int)(((long long)u * Fr) >> 30);   // (x - mean) / std, Q10
                    int o = mad_hi(nq * gg + bb, om, ornd) >> osh;
                    if (!ZPF) o += ozp;
                    if (!SAT8) o = max(c.out.qmin, min(c.out.qmax, o));
                    return o;
                };
#pragma unroll
                for (int k = 0; k < NW; ++k) {
                    const int wi = lane + 32 * k;
                    if (EXACT || wi < words) {
                        int4 gg, bb;
                        if (KEEP) { gg = g[k]; bb = b[k]; }
                        else {
                            gg = __ldg(reinterpret_cast<const int4*>(gamma_q) + wi);
                            bb = __ldg(reinterpret_cast<const int4*>(beta_q) + wi);
                        }
                        const unsigned wk = (unsigned)w[r][k];
                        const int o0 = elem(sext_byte<0>(wk), sh[k], 0, gg.x, bb.x);
                        const int o1 = elem(sext_byte<1>(wk), sh[k], 1, gg.y, bb.y);
                        const int o2 = elem(sext_byte<2>(wk), sh[k], 2, gg.z, bb.z);
                        const int o3 = elem(sext_byte<3>(wk), sh[k], 3, gg.w, bb.w);
                        __stcs(yr + wi, SAT8 ? (int)pack4_sat_s8(o0, o1, o2, o3) : (int)pack4_s8(o0, o1, o2, o3));
                    }
                }
            };
            if (narrow) emit(std::true_type{});
            else        emit(std::false_type{});
        }
    }
}

// Short rows (dim <= 128, dim % 16 == 0: the first Swin stage): LPR lanes share a row, so a warp step covers 32 / LPR
// rows.  Lane q of a row takes words q, q + LPR, ... (WPL = dim / (4 LPR) words); row sums are xor-shuffles over the
// LPR lanes, and every lane then runs the scalar part (variance, square root, reciprocal) of its own row, so the
// hundred dependent instructions of that part are shared by 32 / LPR rows without any broadcast.  Two lanes per row
// up to 96 channels (16 rows per scalar part: 96 channels 20.8 -> 19.5 us, 64 channels 17.4 -> 15.1 us on 200 k rows),
// four at 128, where twelve more words per lane would spill.
template <int LPR, int WPL, bool PTF, bool SAT8, bool ZPF>
__global__ void __launch_bounds__(256, 4)
layernorm_short_rows_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int64_t rows,
                            const int32_t* __restrict__ gamma_q, const int32_t* __restrict__ beta_q,
                            const uint8_t* __restrict__ ptf, const LnDev c)
{
    const int lane = threadIdx.x & 31;
    constexpr int RPW = 32 / LPR;                             // rows per warp step
    const int q = lane & (LPR - 1);                           // position inside the row's lanes
    const int D = c.dim;                                      // = 16 * WPL
    grid_dep_launch();
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t steps = (rows + RPW - 1) / RPW;
    // The per-channel parameters live in shared memory (the lanes of a row read consecutive addresses, the rows of a
    // warp the same ones: no bank conflict).  In registers they are 48 per thread and halve the resident warps, and
    // resident warps are what hides a row's chain of dependent steps (load, two reductions, square root, divide):
    // 64 registers and four CTAs per SM instead of 98 and two took the 96-channel case from 25.0 to 20.8 us.
    __shared__ int4 g[LPR * WPL], b[LPR * WPL];
    unsigned sh[WPL];
    for (int i = threadIdx.x; i < LPR * WPL; i += blockDim.x) {
        g[i] = __ldg(reinterpret_cast<const int4*>(gamma_q) + i);
        b[i] = __ldg(reinterpret_cast<const int4*>(beta_q) + i);
    }
#pragma unroll
    for (int k = 0; k < WPL; ++k) sh[k] = PTF ? __ldg(reinterpret_cast<const unsigned*>(ptf) + q + LPR * k) : 0u;
    __syncthreads();
    grid_dep_wait();                                          // gamma / beta above are static; the rows come from the previous kernel
    const int om = c.out.mult, ornd = c.out.rnd, osh = c.out.shift, ozp = c.out.zp;
    for (int64_t step = warp; step < steps; step += nwarps) {
        const int64_t row = step * RPW + lane / LPR;
        const bool live = row < rows;
        const int* xr = reinterpret_cast<const int*>(x + (live ? row : 0) * D);
        int w[WPL];
#pragma unroll
        for (int k = 0; k < WPL; ++k) w[k] = live ? __ldcs(xr + q + LPR * k) : 0;
        int s1 = 0;
        unsigned s2 = 0;
#pragma unroll
        for (int k = 0; k < WPL; ++k) {
            if (!PTF) {
                s1 = __dp4a(w[k], 0x01010101, s1);
                s2 = (unsigned)__dp4a(w[k], w[k], (int)s2);
            } else {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int xv = ((int)(int8_t)(w[k] >> (8 * t))) << ((sh[k] >> (8 * t)) & 3);
                    s1 += xv;
                    s2 += (unsigned)(xv * xv);
                }
            }
        }
        s1 += __shfl_xor_sync(kFull, s1, 1); s2 += __shfl_xor_sync(kFull, s2, 1);
        if (LPR == 4) { s1 += __shfl_xor_sync(kFull, s1, 2); s2 += __shfl_xor_sync(kFull, s2, 2); }
        const long long V = (long long)D * (long long)s2 - (long long)s1 * (long long)s1;            // D^2 var, exact
        const unsigned long long rt = isqrt_variant((unsigned long long)V, c.variant);                // D * std
        const long long F = rt ? (long long)floor_div_f64(1099511627776.0, (double)rt) : 0;          // floor(2^40 / rt)
        const bool narrow = F < (1ll << 29);                  // then (u F) >> 30 = hi32(u * 4F)
        const int F4 = (int)(F << 2);
        int out[WPL];
#pragma unroll
        for (int k = 0; k < WPL; ++k) {
            const unsigned wk = (unsigned)w[k];
            auto elem = [&](int xv, int t, int gg, int bb) -> int {
                if (PTF) xv <<= ((sh[k] >> (8 * t)) & 3);
                const int u = D * xv - s1;                                   // D (x - mean)
                const int nq = narrow ? __mulhi(u, F4) : (int)(((long long)u * F) >> 30);   // (x - mean) / std, Q10
                int o = mad_hi(nq * gg + bb, om, ornd) >> osh;
                if (!ZPF) o += ozp;
                if (!SAT8) o = max(c.out.qmin, min(c.out.qmax, o));
                return o;
            };
            const int4 gk = g[q + LPR * k], bk = b[q + LPR * k];
            const int o0 = elem(sext_byte<0>(wk), 0, gk.x, bk.x);
            const int o1 = elem(sext_byte<1>(wk), 1, gk.y, bk.y);
            const int o2 = elem(sext_byte<2>(wk), 2, gk.z, bk.z);
            const int o3 = elem(sext_byte<3>(wk), 3, gk.w, bk.w);
            out[k] = SAT8 ? (int)pack4_sat_s8(o0, o1, o2, o3) : (int)pack4_s8(o0, o1, o2, o3);
        }
        if (live) {
            int* yr = reinterpret_cast<int*>(y + row * D);
#pragma unroll
            for (int k = 0; k < WPL; ++k) __stcs(yr + q + LPR * k, out[k]);
        }
    }
}

// W16 = dim / 16
template <int W16>
static int launch_ln_short(const int8_t* x, int8_t* y, int64_t rows, const int32_t* gq, const int32_t* bq,
                           const uint8_t* ptf_in, const LnDev& c, cudaStream_t st)
{
    const int threads = 256;
    constexpr int LPR = W16 <= 6 ? 2 : 4, WPL = 4 * W16 / LPR;
    const int64_t want = ((rows + 32 / LPR - 1) / (32 / LPR) + 7) / 8;
    const int grid = (int)std::min<int64_t>(want, (int64_t)sm_count() * 8);
    const bool sat8 = c.out.qmin == -128 && c.out.qmax == 127;
    LnDev cc = c;
    const long long rz = (long long)c.out.rnd + ((long long)c.out.zp << c.out.shift);
    const bool zpf = rz > -(1ll << 30) && rz < (1ll << 30);
    if (zpf) { cc.out.rnd = (int)rz; cc.out.zp = 0; }
#define IPTQ_LNS_GO(P, S8, ZF) launch_kernel(layernorm_short_rows_kernel<LPR, WPL, P, S8, ZF>, grid, threads, 0, st, x, y, rows, gq, bq, ptf_in, cc)
    if (c.variant == IPTQ_LN_PTF) { if (sat8) IPTQ_LNS_GO(true, true, false); else IPTQ_LNS_GO(true, false, false); }
    else if (!sat8)               { IPTQ_LNS_GO(false, false, false); }
    else if (zpf)                 { IPTQ_LNS_GO(false, true, true); }
    else                          { IPTQ_LNS_GO(false, true, false); }
#undef IPTQ_LNS_GO
    note_launch();
    return last_launch_status();
}

template <int NW>
static int launch_ln(const int8_t* x, int8_t* y, int64_t rows, const int32_t* gq, const int32_t* bq,
                     const uint8_t* ptf_in, const LnDev& c, cudaStream_t st)
{
    constexpr int RW = NW == 1 ? 8 : NW <= 4 ? 4 : NW <= 8 ? 2 : 1;
    const int threads = 256;
    const int64_t want = ((rows + RW - 1) / RW + 7) / 8;
    // Wide rows (640 channels and more: two CTAs per SM): two waves, and the next rows prefetched from two groups per
    // warp on; with more CTAs a warp has a single group and nothing to prefetch (ViT-Base LayerNorm 16.7 -> 15.3 us).
    // Narrower rows: four waves and prefetch only for long loops; there the prefetch costs more than it hides
    // (192 channels, 50 176 rows: 15.2 us against 16.4 - 17.2 us).
    constexpr int kCtasPerSm = NW >= 5 ? 4 : 8, kPrefetchFrom = NW >= 5 ? 2 : 4;
    const int grid = (int)std::min<int64_t>(want, (int64_t)sm_count() * kCtasPerSm);
    const bool sat8 = c.out.qmin == -128 && c.out.qmax == 127;
    const bool exact = c.dim == 128 * NW;
    // fold the zero point into the rounding constant when the sum stays clear of 32-bit overflow (|hi32| < 2^30)
    LnDev cc = c;
    const long long rz = (long long)c.out.rnd + ((long long)c.out.zp << c.out.shift);
    const bool zpf = rz > -(1ll << 30) && rz < (1ll << 30);
    if (zpf) { cc.out.rnd = (int)rz; cc.out.zp = 0; }
    const bool ptf = c.variant == IPTQ_LN_PTF;
    const bool pf = (rows + RW - 1) / RW >= (int64_t)kPrefetchFrom * grid * (threads / 32);   // groups per warp
#define IPTQ_LN_GO(P, S8, EX, ZF)                                                                                        \
    do {                                                                                                                 \
        if (pf) launch_kernel(layernorm_rows_kernel<NW, RW, P, S8, EX, ZF, true>, grid, threads, 0, st, x, y, rows, gq, bq, ptf_ptr, cc);  \
        else    launch_kernel(layernorm_rows_kernel<NW, RW, P, S8, EX, ZF, false>, grid, threads, 0, st, x, y, rows, gq, bq, ptf_ptr, cc); \
    } while (0)
    const uint8_t* ptf_ptr = ptf_in;
    if (ptf)                      { if (sat8) IPTQ_LN_GO(true, true, false, false); else IPTQ_LN_GO(true, false, false, false); }
    else if (!sat8)               { IPTQ_LN_GO(false, false, false, false); }
    else if (exact && zpf)        { IPTQ_LN_GO(false, true, true, true); }
    else if (exact)               { IPTQ_LN_GO(false, true, true, false); }
    else if (zpf)                 { IPTQ_LN_GO(false, true, false, true); }
    else                          { IPTQ_LN_GO(false, true, false, false); }
#undef IPTQ_LN_GO
    note_launch();
    return last_launch_status();
}

// Used by the encoder block as well.
int layernorm_launch(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gq, const int32_t* bq,
                     const uint8_t* ptf, const iptq_ln_consts* consts, cudaStream_t st)
{
    if (!consts) return IPTQ_ERR_NULL;
    if (rows < 0 || dim != consts->dim || dim < 2 || dim > 3072 || (dim & 3)) return IPTQ_ERR_SHAPE;
    if (rows == 0) return IPTQ_OK;
    if (!x || !y || !gq || !bq) return IPTQ_ERR_NULL;
    if (consts->variant < 0 || consts->variant > 2) return IPTQ_ERR_VARIANT;
    if (consts->variant == IPTQ_LN_PTF && !ptf) return IPTQ_ERR_NULL;
    if (!aligned16(x) || !aligned16(y) || !aligned16(gq) || !aligned16(bq) ||
        (ptf && (reinterpret_cast<uintptr_t>(ptf) & 3u)))
        return IPTQ_ERR_ALIGN;
    int rc = check_requant(&consts->out);
    if (rc != IPTQ_OK) return rc;
    if (rows == 0) return IPTQ_OK;
    LnDev c;
    c.variant = consts->variant; c.dim = dim; c.out = to_dev(consts->out);
    if ((dim & 15) == 0 && dim <= 128 && rows >= 64) {
        switch (dim / 16) {
            case 1: return launch_ln_short<1>(x, y, rows, gq, bq, ptf, c, st);
            case 2: return launch_ln_short<2>(x, y, rows, gq, bq, ptf, c, st);
            case 3: return launch_ln_short<3>(x, y, rows, gq, bq, ptf, c, st);
            case 4: return launch_ln_short<4>(x, y, rows, gq, bq, ptf, c, st);
            case 6: return launch_ln_short<6>(x, y, rows, gq, bq, ptf, c, st);
            case 8: return launch_ln_short<8>(x, y, rows, gq, bq, ptf, c, st);
            default: break;                                   // other widths take the general kernel
        }
    }
    const int nw = (dim / 4 + 31) / 32;
    switch (nw) {
        case 1: return launch_ln<1>(x, y, rows, gq, bq, ptf, c, st);
        case 2: return launch_ln<2>(x, y, rows, gq, bq, ptf, c, st);
        case 3: return launch_ln<3>(x, y, rows, gq, bq, ptf, c, st);
        case 4: return launch_ln<4>(x, y, rows, gq, bq, ptf, c, st);
        case 5: case 6: return launch_ln<6>(x, y, rows, gq, bq, ptf, c, st);
        case 7: case 8: return launch_ln<8>(x, y, rows, gq, bq, ptf, c, st);
        default:
            if (nw <= 12) return launch_ln<12>(x, y, rows, gq, bq, ptf, c, st);
            if (nw <= 16) return launch_ln<16>(x, y, rows, gq, bq, ptf, c, st);
            return launch_ln<32>(x, y, rows, gq, bq, ptf, c, st);
    }
}

}  // namespace iptq

using namespace iptq;

extern "C" {

int iptq_softmax(const int32_t* scores, uint8_t* probs, int64_t rows, int row_len, const int32_t* bias,
                 int64_t bias_period, const iptq_softmax_consts* consts, iptq_stream_t stream)
{
    if (!consts) return IPTQ_ERR_NULL;
    if (rows < 0 || row_len < 1 || row_len > 1024 || row_len != consts->row_len) return IPTQ_ERR_SHAPE;
    if (rows == 0) return IPTQ_OK;                      // empty input: nothing to read or write
    if (!scores || !probs) return IPTQ_ERR_NULL;
    if (bias && bias_period < 1) return IPTQ_ERR_SHAPE;
    if (!aligned16(scores) || !aligned16(probs) || (bias && !aligned16(bias))) return IPTQ_ERR_ALIGN;
    if (consts->out_bits < 4 || consts->out_bits > 8) return IPTQ_ERR_BITS;
    if (consts->x0 < 8 || consts->M < 31 || consts->M > 40) return IPTQ_ERR_SCALE_RANGE;
    if (rows == 0) return IPTQ_OK;
    SoftmaxDev c;
    c.ex = to_dev_exp(*consts);
    c.M = consts->M; c.f_shl = consts->f_shl; c.p_shr = consts->p_shr;
    c.tab_n = exp_table_entries(*consts);
    c.tab_src = (consts->table && consts->table_n == c.tab_n) ? consts->table : nullptr;
    switch (consts->variant) {
        case IPTQ_SM_BITEXP: return launch_softmax1<IPTQ_SM_BITEXP>(scores, probs, rows, row_len, bias, bias_period, c, stream);
        case IPTQ_SM_SHIFTMAX: return launch_softmax1<IPTQ_SM_SHIFTMAX>(scores, probs, rows, row_len, bias, bias_period, c, stream);
        case IPTQ_SM_POLY: return launch_softmax1<IPTQ_SM_POLY>(scores, probs, rows, row_len, bias, bias_period, c, stream);
        case IPTQ_SM_LOG2: return launch_softmax1<IPTQ_SM_LOG2>(scores, probs, rows, row_len, bias, bias_period, c, stream);
        default: return IPTQ_ERR_VARIANT;
    }
}

int iptq_gelu(const int32_t* x, int8_t* y, int64_t n, const iptq_gelu_consts* consts, iptq_stream_t stream)
{
    if (!consts) return IPTQ_ERR_NULL;
    if (n < 0) return IPTQ_ERR_SHAPE;
    if (n == 0) return IPTQ_OK;
    if (!x || !y) return IPTQ_ERR_NULL;
    if (!aligned16(x) || !aligned16(y)) return IPTQ_ERR_ALIGN;
    if (consts->in_bits < 8 || consts->in_bits > 16) return IPTQ_ERR_BITS;
    int rc = check_requant(&consts->out);
    if (rc != IPTQ_OK) return rc;
    if (n == 0) return IPTQ_OK;
    if (consts->table && n >= (1 << 20)) {
        // tabulated: worth the 64 KB copy per CTA once every thread has a few vectors
        if (!aligned16(consts->table)) return IPTQ_ERR_ALIGN;
        const int64_t vecs = (n + 3) / 4;
        const int grid = (int)std::min<int64_t>((vecs + kGeluTabThreads - 1) / kGeluTabThreads, (int64_t)sm_count() * 2);
        cudaFuncSetAttribute(gelu_tab_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, IPTQ_GELU_TABLE_SIZE);
        launch_kernel(gelu_tab_kernel, grid, kGeluTabThreads, IPTQ_GELU_TABLE_SIZE, stream, x, y, n, consts->table);
        note_launch();
        return last_launch_status();
    }
    const GeluDev c = to_dev(*consts);
    const int threads = 256;
    const int64_t groups = (n + 3) / 4;
    const int grid = (int)std::min<int64_t>((groups + threads - 1) / threads, (int64_t)sm_count() * 16);
    const bool sat8 = consts->out.qmin == -128 && consts->out.qmax == 127;
#define IPTQ_GELU_LAUNCH(V)                                                               \
    do {                                                                                  \
        if (sat8) launch_kernel(gelu_kernel<V, true>, grid, threads, 0, stream, x, y, n, c);         \
        else      launch_kernel(gelu_kernel<V, false>, grid, threads, 0, stream, x, y, n, c);        \
    } while (0)
    switch (consts->variant) {
        case IPTQ_GELU_POLY4: IPTQ_GELU_LAUNCH(IPTQ_GELU_POLY4); break;
        case IPTQ_GELU_POLY2: IPTQ_GELU_LAUNCH(IPTQ_GELU_POLY2); break;
        case IPTQ_GELU_SHIFT: IPTQ_GELU_LAUNCH(IPTQ_GELU_SHIFT); break;
        default: return IPTQ_ERR_VARIANT;
    }
#undef IPTQ_GELU_LAUNCH
    note_launch();
    return last_launch_status();
}

int iptq_gelu_table(const iptq_gelu_consts* consts, int8_t* table, iptq_stream_t stream)
{
    if (!consts || !table) return IPTQ_ERR_NULL;
    if (!aligned16(table)) return IPTQ_ERR_ALIGN;
    if (consts->in_bits < 8 || consts->in_bits > 16) return IPTQ_ERR_BITS;
    int rc = check_requant(&consts->out);
    if (rc != IPTQ_OK) return rc;
    const GeluDev c = to_dev(*consts);
    const int threads = 256, grid = IPTQ_GELU_TABLE_SIZE / threads;
    switch (consts->variant) {
        case IPTQ_GELU_POLY4: launch_kernel(gelu_table_kernel<IPTQ_GELU_POLY4>, grid, threads, 0, stream, table, c); break;
        case IPTQ_GELU_POLY2: launch_kernel(gelu_table_kernel<IPTQ_GELU_POLY2>, grid, threads, 0, stream, table, c); break;
        case IPTQ_GELU_SHIFT: launch_kernel(gelu_table_kernel<IPTQ_GELU_SHIFT>, grid, threads, 0, stream, table, c); break;
        default: return IPTQ_ERR_VARIANT;
    }
    stream_fence_kernel<<<1, 32, 0, stream>>>();
    note_launch();
    return last_launch_status();
}

int iptq_softmax_table(iptq_softmax_consts* consts, uint16_t* table, int32_t capacity, iptq_stream_t stream)
{
    if (!consts) return IPTQ_ERR_NULL;
    consts->table = nullptr;
    consts->table_n = 0;
    const int n = exp_table_entries(*consts);
    const int n_pad = (n + 8) & ~7;                     // at least one zero behind the last entry
    if (n == 0 || n_pad > IPTQ_SOFTMAX_TABLE_MAX) return IPTQ_OK;
    if (!table) return IPTQ_ERR_NULL;
    if (!aligned16(table)) return IPTQ_ERR_ALIGN;
    if (capacity < n_pad) return IPTQ_ERR_SHAPE;
    const ExpDev ex = to_dev_exp(*consts);
    const int threads = 256, grid = (n_pad + threads - 1) / threads;
    if (consts->variant == IPTQ_SM_BITEXP)        launch_kernel(softmax_table_kernel<IPTQ_SM_BITEXP>, grid, threads, 0, stream, table, n, n_pad, ex);
    else if (consts->variant == IPTQ_SM_SHIFTMAX) launch_kernel(softmax_table_kernel<IPTQ_SM_SHIFTMAX>, grid, threads, 0, stream, table, n, n_pad, ex);
    else                                          launch_kernel(softmax_table_kernel<IPTQ_SM_POLY>, grid, threads, 0, stream, table, n, n_pad, ex);   // also behind the logarithm candidate
    stream_fence_kernel<<<1, 32, 0, stream>>>();
    note_launch();
    const int rc = last_launch_status();
    if (rc == IPTQ_OK) { consts->table = table; consts->table_n = n; }
    return rc;
}

int iptq_layernorm(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gamma_q,
                   const int32_t* beta_q, const uint8_t* ptf_shift, const iptq_ln_consts* consts,
                   iptq_stream_t stream)
{
    return layernorm_launch(x, y, rows, dim, gamma_q, beta_q, ptf_shift, consts, stream);
}

}  // extern "C"
