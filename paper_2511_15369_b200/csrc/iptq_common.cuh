// Shared host/device helpers of the iptq CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
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
    int32_t pad[61];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");
constexpr size_t kStatusBytes = 256;

// ---------------------------------------------------------------- device arithmetic
#ifdef __CUDACC__

// R without zero point / clamp: (hi32(y * mult) + rnd) >> shift, rnd = 2^(shift-1).
__device__ __forceinline__ int requant_core(int y, int mult, int rnd, int shift)
{
    return (__mulhi(y, mult) + rnd) >> shift;    // >> on int is arithmetic (floor)
}

struct RequantDev {
    int mult, rnd, shift, zp, qmin, qmax;
};

__device__ __forceinline__ int requant_full(int y, const RequantDev& r)
{
    int v = requant_core(y, r.mult, r.rnd, r.shift) + r.zp;
    return max(r.qmin, min(r.qmax, v));
}

// Constants of the integer exponential (Eqs. (7)-(10), (13)-(14)) as the kernels use them.
struct ExpDev {
    int x0, nsh, dcap;
    unsigned div_mul; int div_shift;     // floor(v / divisor) = umulhi(v, div_mul) >> div_shift, 0 <= v < 2^31
    int qln2, qb, qc, norm_l, norm_r;    // polynomial candidate
};

// Integer exponential of a clamped distance d = min(max - s, dcap) >= 0.
template <int VARIANT>
__device__ __forceinline__ unsigned exp_core(unsigned d, const ExpDev& c)
{
    if (VARIANT == IPTQ_SM_POLY) {
        unsigned z = __umulhi(d, c.div_mul) >> c.div_shift;          // octave: floor(d / qln2)
        int p = -(int)(d - z * (unsigned)c.qln2);                      // in (-qln2, 0]
        int t = p + c.qb;
        unsigned poly = (unsigned)(t * t + c.qc);
        unsigned e = (poly << c.norm_l) >> c.norm_r;
        return z > 31u ? 0u : (e >> z);
    } else {
        int nd = -(int)d;                                              // Q_delta
        int Qp = nd + (nd >> 1) - (nd >> 4);                           // Eq. (7)
        unsigned P = (unsigned)(-Qp);
        unsigned q = __umulhi(P, c.div_mul) >> c.div_shift;            // Eq. (8): floor(P / x0)
        int u = -(int)(P - q * (unsigned)c.x0);                        // -r
        int base;
        if (VARIANT == IPTQ_SM_BITEXP) base = (u >> 1) + (u >> 3) + (u >> 4) + c.x0;   // Eqs. (13)-(14)
        else                           base = (u >> 1) + c.x0;                         // Eq. (10)
        unsigned b = (unsigned)base << c.nsh;
        return q > 31u ? 0u : (b >> q);                                // Eq. (9)
    }
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
template <int VARIANT>
__device__ __forceinline__ int gelu_core(int x, const GeluDev& c)
{
    x = max(c.lo, min(c.hi, x));
    if (VARIANT == IPTQ_GELU_SHIFT) {
        int xp = x + (x >> 1) + (x >> 3) + (x >> 4);
        unsigned d = min((unsigned)abs(xp), (unsigned)c.ex.dcap);
        unsigned e = exp_core<IPTQ_SM_SHIFTMAX>(d, c.ex);
        unsigned D = (unsigned)c.ex.x0 << c.ex.nsh;
        unsigned f = 0x80000000u / (D + e);          // IntDiv with M = 31
        unsigned num = xp >= 0 ? D : e;
        int sig = (int)((f * num) >> 16);            // Q15; f * num <= 2^31
        return x * sig;
    } else {
        int m = min(abs(x), c.Bq);
        int t = c.Bq - m;
        int t2 = (t * t) >> c.sh2;
        int pw = (VARIANT == IPTQ_GELU_POLY4) ? t2 * t2 : t2;
        int E = c.C - pw;
        int G = x > 0 ? c.C + E : (x < 0 ? c.C - E : c.C);
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
