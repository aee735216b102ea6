// Micro-benchmarks behind the ceilings the benchmark reports against: (1) a bare tcgen05.mma.kind::i8 issue loop per
// UMMA N (operands resident in shared memory, no loads, no epilogue), burst and sustained; (2) issue rates of the
// integer instructions the epilogues and the Softmax are made of; (3) TMEM load rate; (4) byte-store patterns.
// Every wait is bounded.  Built and run by `python -m paper_2511_15369_b200.peaks`.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>
#include <algorithm>
#include "tc_common.cuh"

using namespace iptq;

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e_), __FILE__, __LINE__); exit(1); } } while (0)

// ------------------------------------------------------------------ (1) MMA issue loop
// One CTA per SM, 128 threads.  smem: A 128 rows x 128 B (SW128), B 256 rows x 128 B.  iters x 4 MMAs (k-steps of 32).
struct MmaOut { unsigned long long clocks, ns; int ok; };

__global__ void __launch_bounds__(128, 1) mma_loop_kernel(int N, int iters, MmaOut* out)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + 16384;
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ CtaControl ctl;
    for (int i = threadIdx.x; i < (16384 + 32768) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); ctl.abort = 0; fence_barrier_init(); }
    fence_proxy_async_smem();
    const int warp = threadIdx.x >> 5;
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    unsigned long long c0 = 0, c1 = 0, t0 = 0, t1 = 0;
    int ok = 1;
    if (warp == 1 && elect_one()) {
        const uint32_t idesc = umma_idesc_i8(128, N, true, true, false, false);
        const uint32_t a_addr = smem_u32(sA), b_addr = smem_u32(sB);
        t0 = global_timer_ns();
        c0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t tacc = tmem_base + (uint32_t)((it & 1) * (N <= 256 ? 256 : 0));
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint64_t da = umma_smem_desc(a_addr + k * 32, 16, 1024, 128);
                const uint64_t db = umma_smem_desc(b_addr + k * 32, 16, 1024, 128);
                umma_i8(tacc, da, db, idesc, 1u);
            }
        }
        umma_commit(&bar);
        ok = mbar_wait(&bar, 0, &ctl, nullptr, 1) ? 1 : 0;
        c1 = clock64();
        t1 = global_timer_ns();
        out[blockIdx.x].clocks = c1 - c0;
        out[blockIdx.x].ns = t1 - t0;
        out[blockIdx.x].ok = ok;
    }
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

// ------------------------------------------------------------------ (2) integer issue rates
// 8 independent chains per thread, UNROLL ops each per loop iteration.
template <int OP>
__device__ __forceinline__ int one_op(int a, int b, int c)
{
    int d;
    if (OP == 0) asm volatile("mad.lo.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));        // IMAD
    else if (OP == 1) asm volatile("mad.hi.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // IMAD.HI
    else if (OP == 2) asm volatile("add.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));                  // IADD
    else if (OP == 3) asm volatile("shr.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));                  // SHF
    else if (OP == 4) asm volatile("max.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));                  // VIMNMX
    else if (OP == 5) asm volatile("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c)); // LOP3
    else if (OP == 6) asm volatile("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c)); // I2IP
    else if (OP == 7) asm volatile("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));     // PRMT
    else if (OP == 8) { asm volatile("{ .reg .s32 t; max.s32 t, %1, %2; min.s32 %0, t, %3; }" : "=r"(d) : "r"(a), "r"(b), "r"(c)); }   // 3-input min/max
    else if (OP == 9) asm volatile("mul.hi.u32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));               // IMAD.HI.U32 no addend
    else if (OP == 11) { asm volatile("{ .reg .s32 t; add.s32 t, %1, %2; max.s32 %0, t, %3; }" : "=r"(d) : "r"(a), "r"(b), "r"(c)); }  // add, then max
    else if (OP == 12) asm volatile("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));          // IDP.4A
    else if (OP == 13) asm volatile("dp2a.lo.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));       // IDP.2A
    else if (OP == 14) asm volatile("shfl.sync.bfly.b32 %0, %1, 1, 0x1f, 0xffffffff;" : "=r"(d) : "r"(a));       // SHFL
    // pairs of independent-pipe candidates, two instructions per call: does one hide behind the other?
    else if (OP == 20) { int t; asm volatile("mad.hi.s32 %0, %1, %2, %3;" : "=r"(t) : "r"(a), "r"(b), "r"(c)); asm volatile("shr.s32 %0, %1, %2;" : "=r"(d) : "r"(t), "r"(b & 7)); }
    else if (OP == 21) { int t; asm volatile("mad.lo.s32 %0, %1, %2, %3;" : "=r"(t) : "r"(a), "r"(b), "r"(c)); asm volatile("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(t), "r"(b), "r"(c)); }
    else if (OP == 22) { int t; asm volatile("mad.hi.s32 %0, %1, %2, %3;" : "=r"(t) : "r"(a), "r"(b), "r"(c)); asm volatile("add.s32 %0, %1, %2;" : "=r"(d) : "r"(t), "r"(c)); }
    else if (OP == 23) { int t; asm volatile("shr.s32 %0, %1, %2;" : "=r"(t) : "r"(a), "r"(b & 7)); asm volatile("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(t), "r"(b), "r"(c)); }
    else { long long w; asm volatile("mul.wide.s32 %0, %1, %2;" : "=l"(w) : "r"(a), "r"(b)); d = (int)(w >> 32) ^ (int)w; }
    return d;
}

template <int OP>
__global__ void __launch_bounds__(1024, 1) int_rate_kernel(int iters, int seed, int* sink, unsigned long long* clocks)
{
    int v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = seed + threadIdx.x * 8 + i;
    const int b = seed | 3, c = seed ^ 0x5555;
    __syncthreads();
    const unsigned long long c0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = one_op<OP>(v[i], b, c);
    }
    const unsigned long long c1 = clock64();
    int s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) s ^= v[i];
    if (s == 0x7fffffff) sink[0] = s;
    if (threadIdx.x == 0) clocks[blockIdx.x] = c1 - c0;
}

// ------------------------------------------------------------------ (3) TMEM load rate: 16 warps read 32x32b.x32 in a loop
__global__ void __launch_bounds__(512, 1) tmem_ld_kernel(int iters, int nwarps, int* sink, unsigned long long* clocks)
{
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tl = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 64);
    uint32_t r[32];
    // define the columns first
#pragma unroll
    for (int j = 0; j < 32; ++j) r[j] = threadIdx.x + j;
    {
        uint32_t z[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) z[j] = r[j];
        for (int c = 0; c < 4; ++c) tmem_st16(tl + c * 16, z);
        tmem_wait_st();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    unsigned acc = 0;
    const unsigned long long c0 = clock64();
    if (warp < nwarps) {
        for (int it = 0; it < iters; ++it) {
            tmem_ld32(tl, r);
            tmem_wait_ld();
            acc += r[0] ^ r[31];
            tmem_ld32(tl + 32, r);
            tmem_wait_ld();
            acc += r[1] ^ r[30];
        }
    }
    const unsigned long long c1 = clock64();
    if (acc == 0x12345u) sink[0] = (int)acc;
    if (threadIdx.x == 0) clocks[blockIdx.x] = c1 - c0;
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

__global__ void __launch_bounds__(512, 1) tmem_ld16_kernel(int iters, int nwarps, int* sink, unsigned long long* clocks)
{
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tl = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 64);
    uint32_t a[16], b[16], c[16], d[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) a[j] = threadIdx.x + j;
    for (int q = 0; q < 4; ++q) tmem_st16(tl + q * 16, a);
    tmem_wait_st();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    unsigned acc = 0;
    const unsigned long long c0 = clock64();
    if (warp < nwarps) {
        for (int it = 0; it < iters; ++it) {
            tmem_ld16(tl, a); tmem_ld16(tl + 16, b); tmem_ld16(tl + 32, c); tmem_ld16(tl + 48, d);
            tmem_wait_ld();
            acc += a[0] ^ b[15] ^ c[3] ^ d[7];
        }
    }
    const unsigned long long c1 = clock64();
    if (acc == 0x12345u) sink[0] = (int)acc;
    if (threadIdx.x == 0) clocks[blockIdx.x] = c1 - c0;
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

// ------------------------------------------------------------------ (4) byte stores: each warp writes rows of 32 consecutive bytes
// mode 0: st.global.u8, lane = byte within a 32-byte segment; mode 1: st.global.v4 (16 B per lane) for comparison
__global__ void __launch_bounds__(512, 1) store_kernel(uint8_t* out, long long bytes, int mode)
{
    const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * (blockDim.x >> 5);
    const int lane = threadIdx.x & 31;
    if (mode == 0) {
        // a warp owns a [64 rows][32 bytes] patch of a row-major matrix with 3072-byte rows
        const long long patches = bytes / (64 * 32);
        for (long long p = gw; p < patches; p += nw) {
            const long long prow = p / 96, pcol = p % 96;
            uint8_t* base = out + (prow * 64) * 3072 + pcol * 32 + lane;
#pragma unroll 16
            for (int j = 0; j < 64; ++j) base[(long long)j * 3072] = (uint8_t)(j + lane);
        }
    } else {
        const long long vecs = bytes / 16;
        for (long long i = gw * 32 + lane; i < vecs; i += nw * 32)
            reinterpret_cast<uint4*>(out)[i] = make_uint4(lane, lane, lane, lane);
    }
}

template <int OP>
static void run_int(const char* name, int* sink, unsigned long long* dclk, int sms, int instr_per_op = 1)
{
    const int iters = 4096;
    int_rate_kernel<OP><<<sms, 1024>>>(iters, 12345, sink, dclk);
    CK(cudaDeviceSynchronize());
    cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
    cudaEventRecord(a);
    int_rate_kernel<OP><<<sms, 1024>>>(iters, 12345, sink, dclk);
    cudaEventRecord(b);
    CK(cudaDeviceSynchronize());
    float ms; cudaEventElapsedTime(&ms, a, b);
    std::vector<unsigned long long> h(sms);
    CK(cudaMemcpy(h.data(), dclk, sms * 8, cudaMemcpyDeviceToHost));
    std::sort(h.begin(), h.end());
    const double warp_instr = (double)iters * 32 * 32 * instr_per_op;       // per SM: 32 warps x iters x 32 ops
    printf("int %-10s median clocks %llu  warp-instr/clk/SM %.3f  (per sub-partition %.3f)  kernel %.3f ms\n", name,
           h[sms / 2], warp_instr / (double)h[sms / 2], warp_instr / (double)h[sms / 2] / 4, ms);
}

int main(int argc, char** argv)
{
    int dev = 0; CK(cudaSetDevice(dev));
    cudaDeviceProp prop; CK(cudaGetDeviceProperties(&prop, dev));
    const int sms = prop.multiProcessorCount;
    printf("device %s, %d SMs\n", prop.name, sms);
    MmaOut* dout; CK(cudaMalloc(&dout, sizeof(MmaOut) * sms));
    int* sink; CK(cudaMalloc(&sink, 64));
    unsigned long long* dclk; CK(cudaMalloc(&dclk, 8 * sms));
    const int smem = 16384 + 32768 + 1024;
    CK(cudaFuncSetAttribute(mma_loop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const bool sustained = argc > 1 && !strcmp(argv[1], "sustained");

    // (1) MMA issue loop
    const int Ns[] = {64, 96, 128, 192, 256};
    for (int N : Ns) {
        for (int grid : {1, sms}) {
            const int iters = 4000;
            mma_loop_kernel<<<grid, 128, smem>>>(N, iters, dout);
            CK(cudaDeviceSynchronize());
            mma_loop_kernel<<<grid, 128, smem>>>(N, iters, dout);
            CK(cudaDeviceSynchronize());
            std::vector<MmaOut> h(grid);
            CK(cudaMemcpy(h.data(), dout, sizeof(MmaOut) * grid, cudaMemcpyDeviceToHost));
            std::vector<unsigned long long> c, t; int ok = 1;
            for (auto& o : h) { c.push_back(o.clocks); t.push_back(o.ns); ok &= o.ok; }
            std::sort(c.begin(), c.end()); std::sort(t.begin(), t.end());
            const double mmas = iters * 4.0;
            const double clk_per = c[grid / 2] / mmas, ns = (double)t[grid / 2];
            const double tops = 2.0 * 128 * N * 32 * mmas * grid / (ns * 1e-9) / 1e12;
            printf("mma N=%3d grid=%3d ok=%d  clocks/MMA %.1f  SM clock %.0f MHz  %.0f TOP/s (whole grid)\n", N, grid, ok,
                   clk_per, c[grid / 2] / ns * 1e3, tops);
        }
    }
    if (sustained) {
        // back-to-back launches for about 3 s at N=256 and N=128: throughput under the power cap
        for (int N : {128, 256}) {
            const int iters = 40000;
            cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
            int reps = 0; float ms = 0;
            cudaEventRecord(a);
            for (; reps < 4000; ++reps) {
                mma_loop_kernel<<<sms, 128, smem>>>(N, iters, dout);
                if ((reps & 15) == 15) { cudaEventRecord(b); cudaEventSynchronize(b); cudaEventElapsedTime(&ms, a, b); if (ms > 3000) { ++reps; break; } }
            }
            cudaEventRecord(b); CK(cudaDeviceSynchronize()); cudaEventElapsedTime(&ms, a, b);
            std::vector<MmaOut> h(sms);
            CK(cudaMemcpy(h.data(), dout, sizeof(MmaOut) * sms, cudaMemcpyDeviceToHost));
            const double tops = 2.0 * 128 * N * 32 * 4.0 * iters * sms * reps / (ms * 1e-3) / 1e12;
            printf("mma sustained N=%d: %d launches in %.0f ms: %.0f TOP/s; last launch SM clock %.0f MHz, clocks/MMA %.1f\n", N, reps, ms,
                   tops, h[0].clocks / (double)h[0].ns * 1e3, h[0].clocks / (4.0 * iters));
        }
    }

    // (2) integer issue rates
    run_int<0>("IMAD", sink, dclk, sms);
    run_int<1>("IMAD.HI", sink, dclk, sms);
    run_int<9>("MUL.HI.U32", sink, dclk, sms);
    run_int<2>("IADD", sink, dclk, sms);
    run_int<3>("SHF", sink, dclk, sms);
    run_int<4>("VIMNMX", sink, dclk, sms);
    run_int<8>("VIMNMX3", sink, dclk, sms);
    run_int<5>("LOP3", sink, dclk, sms);
    run_int<6>("I2IP", sink, dclk, sms);
    run_int<7>("PRMT", sink, dclk, sms);
    run_int<10>("IMAD.WIDE", sink, dclk, sms);
    run_int<11>("ADD+MAX", sink, dclk, sms);
    run_int<12>("DP4A", sink, dclk, sms);
    run_int<13>("DP2A", sink, dclk, sms);
    run_int<14>("SHFL", sink, dclk, sms);
    run_int<20>("IMAD.HI,SHF", sink, dclk, sms, 2);
    run_int<21>("IMAD,PRMT", sink, dclk, sms, 2);
    run_int<22>("IMAD.HI,IADD", sink, dclk, sms, 2);
    run_int<23>("SHF,PRMT", sink, dclk, sms, 2);

    // (3) TMEM loads
    for (int nw : {1, 4, 8, 16}) {
        const int iters = 2000;
        tmem_ld_kernel<<<sms, 512>>>(iters, nw, sink, dclk);
        CK(cudaDeviceSynchronize());
        std::vector<unsigned long long> h(sms);
        CK(cudaMemcpy(h.data(), dclk, sms * 8, cudaMemcpyDeviceToHost));
        std::sort(h.begin(), h.end());
        const double bytes = (double)iters * 2 * 32 * 32 * 4 * nw;
        printf("tmem ld: %2d warps, 2 x (32x32b.x32 + wait) per iteration: %.1f clocks/iteration, %.0f B/clk/SM\n", nw,
               h[sms / 2] / (double)iters, bytes / h[sms / 2]);
    }

    for (int nw : {1, 4, 8, 16}) {
        const int iters = 2000;
        tmem_ld16_kernel<<<sms, 512>>>(iters, nw, sink, dclk);
        CK(cudaDeviceSynchronize());
        std::vector<unsigned long long> h(sms);
        CK(cudaMemcpy(h.data(), dclk, sms * 8, cudaMemcpyDeviceToHost));
        std::sort(h.begin(), h.end());
        const double bytes = (double)iters * 4 * 16 * 32 * 4 * nw;
        printf("tmem ld: %2d warps, 4 x (32x32b.x16) + wait per iteration: %.1f clocks/iteration, %.0f B/clk/SM\n", nw,
               h[sms / 2] / (double)iters, bytes / h[sms / 2]);
    }

    // (4) stores
    {
        const long long bytes = 25216LL * 3072;      // ViT-Base hidden activation
        uint8_t* buf; CK(cudaMalloc(&buf, bytes));
        for (int mode : {0, 1}) {
            cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
            store_kernel<<<sms, 512>>>(buf, bytes, mode);
            CK(cudaDeviceSynchronize());
            cudaEventRecord(a);
            store_kernel<<<sms, 512>>>(buf, bytes, mode);
            cudaEventRecord(b);
            CK(cudaDeviceSynchronize());
            float ms; cudaEventElapsedTime(&ms, a, b);
            printf("store mode %d (%s): %.1f us for %.1f MB: %.0f GB/s\n", mode, mode == 0 ? "st.u8, 32 lanes = 32 consecutive bytes, rows 3072 B apart" : "st.v4 linear",
                   ms * 1e3, bytes / 1e6, bytes / (ms * 1e-3) / 1e9);
        }
    }
    printf("done\n");
    return 0;
}
