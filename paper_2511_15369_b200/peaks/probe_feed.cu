// What feeds and drains the tensor core, measured beside a running tcgen05.mma.kind::i8 issue loop:
// (1) bulk copies from L2 into shared memory while the MMAs read their operands from shared memory, for 1 to all
//     SMs copying at once (the per-SM rate an operand ring can be refilled at);
// (2) TMEM loads by 8 / 16 warps from columns the MMAs do not write (the rate an epilogue can drain at);
// (3) the issue loop of a CTA pair (cta_group::2, 256 x N x 32 over two SMs).
// Every wait is bounded.  Built and run by `python -m paper_2511_15369_b200.peaks`.
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <algorithm>
#include "tc_common.cuh"

using namespace iptq;

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e_), __FILE__, __LINE__); exit(1); } } while (0)

struct MixOut { unsigned long long mma_clocks, copy_clocks; int ok, ld_iters; };

constexpr int STAGE = 49152;                 // one copy: a 128-row weight tile + a 256-row activation tile of 128 B rows
constexpr int SRC_PER_CTA = 512 * 1024;      // every CTA cycles through its own 512 KB of the source (L2-resident)

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// warp 0: TMEM; warp 1: MMA loop (operands at the start of shared memory); warp 2: copies into a `depth`-deep ring behind
// them; warps 4..: TMEM loads from columns 256.. until the MMA loop has ended
__global__ void __launch_bounds__(640, 1) mix_kernel(int N, int iters, int copy_bytes, int depth, int ld_warps,
                                                     const uint8_t* src, MixOut* out, int* sink)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* ring = smem + STAGE;
    __shared__ uint64_t bar, rbar[4];
    __shared__ uint32_t tmem_slot;
    __shared__ CtaControl ctl;
    __shared__ volatile int mma_done;
    for (int i = threadIdx.x; i < STAGE / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        for (int i = 0; i < 4; ++i) mbar_init(&rbar[i], 1);
        ctl.abort = 0; mma_done = 0;
        fence_barrier_init();
    }
    fence_proxy_async_smem();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 1) {
        if (elect_one()) {
            const uint32_t idesc = umma_idesc_i8(128, N, true, true, false, false);
            const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + 16384;
            const unsigned long long c0 = clock64();
            for (int it = 0; it < iters; ++it) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_i8(tmem_base, umma_smem_desc(a_addr + k * 32, 16, 1024, 128),
                            umma_smem_desc(b_addr + k * 32, 16, 1024, 128), idesc, 1u);
            }
            umma_commit(&bar);
            const int ok = mbar_wait(&bar, 0, &ctl, nullptr, 1) ? 1 : 0;
            out[blockIdx.x].mma_clocks = clock64() - c0;
            out[blockIdx.x].ok = ok;
            mma_done = 1;
        }
    } else if (warp == 2) {
        if (lane == 0 && copy_bytes > 0) {
            const uint8_t* base = src + (size_t)blockIdx.x * SRC_PER_CTA;
            const unsigned long long c0 = clock64();
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % depth;
                if (it >= depth) ok = mbar_wait(&rbar[s], (uint32_t)((it / depth) - 1) & 1u, &ctl, nullptr, 2);
                mbar_expect_tx(&rbar[s], (uint32_t)copy_bytes);
                bulk_load(ring + s * copy_bytes, base + (size_t)(it % 10) * STAGE, (uint32_t)copy_bytes, &rbar[s]);
            }
            for (int it = max(iters - depth, 0); it < iters && ok; ++it)
                ok = mbar_wait(&rbar[it % depth], (uint32_t)(it / depth) & 1u, &ctl, nullptr, 3);
            out[blockIdx.x].copy_clocks = clock64() - c0;
            if (!ok) out[blockIdx.x].ok = 0;
        }
    } else if (warp >= 4 && warp < 4 + ld_warps) {
        const int w = warp - 4;
        const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + 256u + (uint32_t)((w >> 2) * 32);
        uint32_t r[16];
        int acc = 0, n = 0;
        while (!mma_done && n < (1 << 22)) {
            tmem_ld16(taddr, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) acc += (int)r[i];
            ++n;
        }
        if (lane == 0 && w == 0) out[blockIdx.x].ld_iters = n;
        if (acc == 0x7fffffff) sink[0] = acc;
    }
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

// issue loop of a CTA pair: each CTA holds 128 rows of A and N / 2 rows of B
__global__ void __launch_bounds__(128, 1) pair_loop_kernel(int N, int iters, MixOut* out)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ CtaControl ctl;
    for (int i = threadIdx.x; i < 32768 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); ctl.abort = 0; fence_barrier_init(); }
    fence_proxy_async_smem();
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = cluster_ctarank();
    if (warp == 0) { tmem_alloc_pair(&tmem_slot, 512); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 1 && rank == 0 && elect_one()) {
        const uint32_t idesc = umma_idesc_i8(256, N, true, true, false, false);
        const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + 16384;
        const unsigned long long c0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t tacc = tmem_base + (uint32_t)((it & 1) * 256);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_i8_pair(tacc, umma_smem_desc(a_addr + k * 32, 16, 1024, 128),
                             umma_smem_desc(b_addr + k * 32, 16, 1024, 128), idesc, 1u);
        }
        umma_commit_pair(&bar, 1);
        const int ok = mbar_wait(&bar, 0, &ctl, nullptr, 1) ? 1 : 0;
        out[blockIdx.x >> 1].mma_clocks = clock64() - c0;
        out[blockIdx.x >> 1].ok = ok;
    }
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc_pair(tmem_base, 512); }
}

int main()
{
    CK(cudaSetDevice(0));
    cudaDeviceProp prop; CK(cudaGetDeviceProperties(&prop, 0));
    const int sms = prop.multiProcessorCount;
    const int smem = 4 * STAGE + 1024;
    CK(cudaFuncSetAttribute(mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    uint8_t* src; CK(cudaMalloc(&src, (size_t)sms * SRC_PER_CTA)); CK(cudaMemset(src, 1, (size_t)sms * SRC_PER_CTA));
    MixOut* out; CK(cudaMalloc(&out, sizeof(MixOut) * sms));
    int* sink; CK(cudaMalloc(&sink, 64));
    std::vector<MixOut> h(sms);
    const int iters = 4000;
    auto run = [&](int N, int copy_bytes, int ld_warps, int grid, int depth = 3) {
        CK(cudaMemset(out, 0, sizeof(MixOut) * sms));
        for (int rep = 0; rep < 2; ++rep) {
            mix_kernel<<<grid, 640, smem>>>(N, iters, copy_bytes, depth, ld_warps, src, out, sink);
            CK(cudaDeviceSynchronize());
        }
        CK(cudaMemcpy(h.data(), out, sizeof(MixOut) * sms, cudaMemcpyDeviceToHost));
        std::vector<double> m, t; int ok = 1; double ldi = 0;
        for (int i = 0; i < grid; ++i) {
            m.push_back((double)h[i].mma_clocks / (iters * 4.0)); t.push_back((double)h[i].copy_clocks / iters);
            ok &= h[i].ok; ldi += h[i].ld_iters;
        }
        std::sort(m.begin(), m.end()); std::sort(t.begin(), t.end());
        const double mm = m[grid / 2], tt = t[grid / 2];
        printf("feed: MMA N=%3d on %3d SMs", N, grid);
        if (copy_bytes) printf(", %d copies of %d B in flight: %.0f clocks each = %.1f B/clk/SM (%.1f KB/clk in all)", depth, copy_bytes, tt,
                               copy_bytes / tt, copy_bytes / tt * grid / 1024.0);
        if (ld_warps) printf(", %2d warps of TMEM loads: one 32x32b.x16 per %.0f clocks per warp = %.0f B/clk/SM", ld_warps,
                             mm * iters * 4.0 / (ldi / grid), 2048.0 * ld_warps * (ldi / grid) / (mm * iters * 4.0));
        printf(": ok=%d clocks/MMA %.1f\n", ok, mm);
    };
    for (int N : {128, 256}) {
        run(N, 0, 0, sms);
        for (int grid : {1, 37, 74, 111, sms}) run(N, 16384 + 128 * N, 0, grid);
        run(N, 0, 8, sms);
        run(N, 0, 16, sms);
        run(N, 16384 + 128 * N, 16, sms);
    }
    // is the rate with all SMs copying a limit of bandwidth or of bytes in flight?  2, 3 and 4 copies of 36 KB
    for (int depth : {2, 3, 4}) run(256, 36864, 0, sms, depth);
    // CTA pairs
    const int psmem = 32768 + 1024;
    CK(cudaFuncSetAttribute(pair_loop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, psmem));
    for (int N : {64, 128, 192, 256}) for (int grid : {2, sms & ~1}) {
        CK(cudaMemset(out, 0, sizeof(MixOut) * sms));
        for (int rep = 0; rep < 2; ++rep) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = grid; cfg.blockDim = 128; cfg.dynamicSmemBytes = psmem; cfg.stream = 0;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            CK(cudaLaunchKernelEx(&cfg, pair_loop_kernel, N, iters, out));
            CK(cudaDeviceSynchronize());
        }
        CK(cudaMemcpy(h.data(), out, sizeof(MixOut) * sms, cudaMemcpyDeviceToHost));
        std::vector<double> m; int ok = 1;
        for (int i = 0; i < grid / 2; ++i) { m.push_back((double)h[i].mma_clocks / (iters * 4.0)); ok &= h[i].ok; }
        std::sort(m.begin(), m.end());
        printf("pair MMA 256 x %3d x 32 on %3d SMs: ok=%d clocks/MMA %.1f = %.0f op/clk per SM\n", N, grid, ok,
               m[m.size() / 2], 2.0 * 256 * N * 32 / m[m.size() / 2] / 2);
    }
    printf("done\n");
    return 0;
}
