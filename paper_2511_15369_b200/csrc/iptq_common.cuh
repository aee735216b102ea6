// Shared host/device helpers of the iptq CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "iptq.h"

namespace iptq {

// ---------------------------------------------------------------- launch accounting / errors
void note_launch(int n = 1);
int cuda_status(cudaError_t e);                 // cudaSuccess -> IPTQ_OK, else IPTQ_ERR_CUDA (and remembers the text)
int last_launch_status();                       // cudaGetLastError() folded into an iptq_status
int sm_count();                                 // SM count of the current device (cached per device)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The first 256 bytes of every workspace: written by device-side bounded waits.
struct StatusBlock {
    int32_t timeout_flag;     // non-zero once any bounded wait has given up
    int32_t where;            // id of the wait that gave up first (kernel-specific)
    int32_t block;            // blockIdx.x of the CTA that gave up
    int32_t work_next;        // next work item of a kernel that hands out items dynamically (0 between launches)
    int32_t work_done;        // CTAs of that kernel that have finished (0 between launches)
    int32_t wait_limit_us;    // limit of a bounded device-side wait in microseconds; 0 = the default (2 s)
    int32_t pad[58];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");
constexpr size_t kStatusBytes = 256;

// ---------------------------------------------------------------- launches
#ifdef __CUDACC__

// Every kernel of the library is launched with programmatic stream serialisation: its CTAs may become resident and
// run their set-up (barrier init, TMEM allocation, constant tables) while the kernel before it on the stream is
// still draining.  In exchange every kernel calls grid_dep_wait() before it reads or writes anything another
// kernel may touch; grid_dep_launch() lets the kernel after it start its own set-up early.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                        Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
// The same for a grid of thread-block clusters of `cluster_x` CTAs along x (gridDim.x is a multiple of it).
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_kernel_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                                cudaStream_t st, unsigned cluster_x, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
// Blocks until the kernels this one depends on have completed and their writes are visible.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allows the next kernel on the stream to be scheduled once every CTA of this grid has passed this point.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

#endif  // __CUDACC__

// ---------------------------------------------------------------- device arithmetic
#ifdef __CUDACC__

// The integer pipes of sm_100a issue one simple 32-bit instruction (add, shift, min/max, logic, byte pack,
// IMAD) per clock per SM sub-partition; IMAD.HI costs about 1.5 issue slots and 64-bit results about 2.5.
// The helpers below pin the instruction selection where the compiler's choice matters.

// hi32(a * b) + c in one instruction (IMAD.HI with addend).
__device__ __forceinline__ int mad_hi(int a, int b, int c)
{
    int d;
    asm("mad.hi.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// hi32(a * b + c) with a 64-bit addend (IMAD.WIDE; the value is the high word of its result).  With
// c = bias * b + (rnd << 32) this is hi32((a + bias) * b) + rnd exactly: the 64-bit sum cannot overflow for 32-bit
// a, bias and a multiplier below 2^31, and adding a multiple of 2^32 before the floor adds it after the floor.
__device__ __forceinline__ int mad_wide_hi(int a, int b, long long c)
{
    long long d;
    asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return (int)(d >> 32);
}
// Logical right shift that yields 0 for shift amounts >= 32 (PTX shr clamps the amount).
__device__ __forceinline__ unsigned shr_clamp(unsigned v, unsigned n)
{
    unsigned d;
    asm("shr.u32 %0, %1, %2;" : "=r"(d) : "r"(v), "r"(n));
    return d;
}
// Two int32 saturated to int8 / uint8 into the low half of a word, `hi16` supplying the upper half:
// pack4 = pack2(c, d, 0) then pack2(a, b, that) -- two instructions for four values, clamp included.
__device__ __forceinline__ unsigned pack4_sat_s8(int a, int b, int c, int d)
{
    unsigned t, r;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(d), "r"(c), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(b), "r"(a), "r"(t));
    return r;
}
__device__ __forceinline__ unsigned pack4_sat_u8(int a, int b, int c, int d)
{
    unsigned t, r;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(d), "r"(c), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(b), "r"(a), "r"(t));
    return r;
}

// Byte `idx` (compile-time 0..3) of a word, sign-extended to 32 bits: one PRMT whose upper three selector
// nibbles replicate the sign of the selected byte.
template <int IDX>
__device__ __forceinline__ int sext_byte(unsigned w)
{
    int d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(0u), "r"(0x8880u | (unsigned)(IDX * 0x1111)));
    return d;
}

// R without zero point / clamp: (hi32(y * mult) + rnd) >> shift, rnd = 2^(shift-1).
__device__ __forceinline__ int requant_core(int y, int mult, int rnd, int shift)
{
    return mad_hi(y, mult, rnd) >> shift;        // >> on int is arithmetic (floor)
}

struct RequantDev {
    int mult, rnd, shift, zp, qmin, qmax;
};

__device__ __forceinline__ int requant_full(int y, const RequantDev& r)
{
    int v = requant_core(y, r.mult, r.rnd, r.shift) + r.zp;
    return max(r.qmin, min(r.qmax, v));
}
// Same without the clamp, for callers that saturate to 8 bits while packing (qmin/qmax = -128/127).
__device__ __forceinline__ int requant_nosat(int y, const RequantDev& r)
{
    return requant_core(y, r.mult, r.rnd, r.shift) + r.zp;
}

// Constants of the integer exponential (Eqs. (7)-(10), (13)-(14)) as the kernels use them.
struct ExpDev {
    int x0, nsh, dcap;
    unsigned div_mul; int div_shift;     // floor(v / divisor) = umulhi(v, div_mul) >> div_shift, 0 <= v < 2^31
    int qln2, qb, qc, norm_l, norm_r;    // polynomial candidate
};

// Integer exponential of nd = s - max <= 0, i.e. Q_delta of Eq. (6).  The clamp of max - s at dcap = 34 x0 needs no
// instruction: for any nd > -2^31 the magnitude -Q_p stays below 2^32, and from the clamp point on the octave count
// q is at least 48 (the multiply-high quotient of an operand >= 2^31 is >= 127), so the shift of Eq. (9) returns 0
// exactly as the clamped value would.
template <int VARIANT>
__device__ __forceinline__ unsigned exp_core_nd(int nd, const ExpDev& c)
{
    if (VARIANT == IPTQ_SM_POLY || VARIANT == IPTQ_SM_LOG2) {
        const unsigned d = (unsigned)(-nd);
        unsigned z = __umulhi(d, c.div_mul) >> c.div_shift;          // octave: floor(d / qln2)
        int t = (int)(z * (unsigned)c.qln2) - (int)d + c.qb;           // p + qb, p in (-qln2, 0]
        unsigned poly = (unsigned)(t * t + c.qc);
        unsigned e = (poly << c.norm_l) >> c.norm_r;
        return shr_clamp(e, z);
    } else {
        const int a = nd >> 1, b = nd >> 4;
        const unsigned P = (unsigned)b - (unsigned)a - (unsigned)nd;   // -Q_p, Eq. (7); < 2^32 for nd > -2^31
        const unsigned q = __umulhi(P, c.div_mul) >> c.div_shift;      // Eq. (8): floor(P / x0)
        const int u = (int)(q * (unsigned)c.x0) - (int)P;              // -r
        int base;
        if (VARIANT == IPTQ_SM_BITEXP) base = (u >> 1) + (u >> 3) + (u >> 4) + c.x0;   // Eqs. (13)-(14)
        else                           base = (u >> 1) + c.x0;                         // Eq. (10)
        return shr_clamp((unsigned)base << c.nsh, q);                  // Eq. (9); 0 once q >= 32
    }
}
template <int VARIANT>
__device__ __forceinline__ unsigned exp_core(unsigned d, const ExpDev& c)
{
    return exp_core_nd<VARIANT>(-(int)d, c);
}

// Scores that take no part in a row (columns past the row end, masked pairs) carry this value.  The distance to the
// row maximum is formed in unsigned arithmetic, mx - kNoScore >= 2^30 for every admissible maximum (|score| < 2^30),
// and clamped (exp_distance below, or at the table length), so that such a column gets the exponential 0 whatever
// the row holds -- also when every real score of the row is close to -2^30.
constexpr int kNoScore = INT_MIN;
// -(max - s) for the evaluated exponential: exact for real scores (the distance is below 2^31), -(2^31 - 1) for
// kNoScore, where every variant of exp_core_nd returns 0.
__host__ __device__ __forceinline__ int exp_distance(int mx, int s)
{
    const unsigned d = (unsigned)mx - (unsigned)s;
    return -(int)(d < 0x7fffffffu ? d : 0x7fffffffu);
}

// Length of the exponential table: e(d) = 0 for every d >= the value returned; 0 where no 16-bit table exists.
// Shift-based variants: e vanishes once the octave count q of Eq. (8) reaches qz, the bit length of the largest
// value x0 << nsh; -Q_p >= 23 (d >> 4) puts that at d >= 16 qz x0 / 23 + 15.  Polynomial exponential (also behind
// the logarithm candidate): the value at p = 0 is normalised to 14 bits and is the largest, so e vanishes from
// octave 14 on, d >= 14 qln2.
inline int exp_table_entries(const iptq_softmax_consts& sm)
{
    if (sm.variant == IPTQ_SM_POLY || sm.variant == IPTQ_SM_LOG2) {
        const int64_t top = (((int64_t)sm.qb * sm.qb + sm.qc) << sm.norm_l) >> sm.norm_r;
        if (top >= (1 << 14) || sm.qln2 < 1) return 0;
        const int64_t n = 14 * (int64_t)sm.qln2 + 8;
        return n > (1 << 20) ? 0 : (int)n;
    }
    int qz = 0;
    for (int64_t u = (int64_t)sm.x0 << sm.nsh; u; u >>= 1) ++qz;
    if (qz > 16) return 0;
    const int64_t n = (16 * (int64_t)qz * sm.x0) / 23 + 32;
    return n > (1 << 20) ? 0 : (int)n;
}

// Logarithm candidate: code = round(log2(round(sum / e))) for 0 < e <= sum < 2^31, IPTQ_LOG2_ZERO beyond 15 or for
// e = 0.  round(sum / e) with halves up is (sum + (e >> 1)) / e: for odd e no multiple of e lies between
// sum + (e - 1)/2 and sum + e/2.  The rounded logarithm is the position of the leading one, plus the bit below it.
__device__ __forceinline__ unsigned log2_code(unsigned sum, unsigned e)
{
    if (e == 0) return IPTQ_LOG2_ZERO;
    const unsigned r = (sum + (e >> 1)) / e;                 // >= 1
    const int fl = 31 - __clz((int)r);
    const unsigned code = (unsigned)fl + (fl >= 1 ? ((r >> (fl - 1)) & 1u) : 0u);
    return code > 15u ? (unsigned)IPTQ_LOG2_ZERO : code;
}

// floor(2^M / sum) for 0 < sum < 2^31, M <= 40: the fp64 quotient cannot round across an integer
// (a non-integer quotient is at least 2^-M away, relatively, from the next integer).
__device__ __forceinline__ unsigned intdiv_factor(unsigned sum, int M)
{
    double q = __longlong_as_double((long long)(1023 + M) << 52) / (double)sum;
    return (unsigned)(unsigned long long)q;     // truncation == floor for positive values
}

struct GeluDev {
    int variant, lo, hi;
    int Bq, sh2, C, gs;
    ExpDev ex;                 // IPTQ_GELU_SHIFT
    RequantDev out;
};

// Pre-requant GELU value: x * (G >> gs)  (Eqs. (3), (5)), or x * sigmoid_q(1.702 x).
// Polynomial variants: with t = max(Bq - |x|, 0) (zero outside the clip range of Eq. (3)) and
// t2 = (t t) >> sh2, G = 2C - t2^2 for x >= 0 and t2^2 for x < 0 (second order: t2 instead of t2^2).
// x = 0 gives 0 whatever G is, so the sign(0) = 0 case of Eq. (3) needs no branch.
template <int VARIANT>
__device__ __forceinline__ int gelu_core(int x, const GeluDev& c)
{
    if (VARIANT == IPTQ_GELU_SHIFT) {
        x = max(c.lo, min(c.hi, x));
        int xp = x + (x >> 1) + (x >> 3) + (x >> 4);
        unsigned d = min((unsigned)abs(xp), (unsigned)c.ex.dcap);
        unsigned e = exp_core<IPTQ_SM_SHIFTMAX>(d, c.ex);
        unsigned D = (unsigned)c.ex.x0 << c.ex.nsh;
        unsigned f = 0x80000000u / (D + e);          // IntDiv with M = 31
        unsigned num = xp >= 0 ? D : e;
        int sig = (int)((f * num) >> 16);            // Q15; f * num <= 2^31
        return x * sig;
    } else {
        x = max(c.lo, min(c.hi, x));                 // one 3-input min/max instruction
        const int t = max(min(c.Bq - x, c.Bq + x), 0);
        const int t2 = (t * t) >> c.sh2;
        const bool pos = x >= 0;
        int G;
        if (VARIANT == IPTQ_GELU_POLY4) G = t2 * (pos ? -t2 : t2) + (pos ? 2 * c.C : 0);
        else                            G = pos ? 2 * c.C - t2 : t2;
        return x * (G >> c.gs);
    }
}

__device__ __forceinline__ unsigned pack4_s8(int a, int b, int c, int d)
{
    return (unsigned)(a & 255) | ((unsigned)(b & 255) << 8) | ((unsigned)(c & 255) << 16) | ((unsigned)(d & 255) << 24);
}

#endif  // __CUDACC__

// ---------------------------------------------------------------- host: consts -> device structs
RequantDev to_dev(const iptq_requant& r);
ExpDev to_dev_exp(const iptq_softmax_consts& c);
GeluDev to_dev(const iptq_gelu_consts& c);
int check_requant(const iptq_requant* r);

}  // namespace iptq
