// Cost of a wait on an mbarrier whose phase is already complete: try_wait vs test_wait, 1 / 32 / 512 threads.
#include <cstdio>
#include <cstdlib>
#include "tc_common.cuh"
using namespace iptq;
#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
template <int MODE>
__global__ void __launch_bounds__(512, 1) wait_cost_kernel(int nthreads, int reps, long long* out)
{
    __shared__ uint64_t bar;
    __shared__ CtaControl ctl;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); ctl.abort = 0; fence_barrier_init(); }
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive(&bar);      // phase 0 complete
    __syncthreads();
    long long t0 = 0, t1 = 0;
    int okc = 0;
    const bool act = MODE == 3 ? ((threadIdx.x & 31) == 0 && (int)threadIdx.x < nthreads * 32) : (int)threadIdx.x < nthreads;
    __syncthreads();
    t0 = clock64();
    if (act) {
        for (int r = 0; r < reps; ++r) {
            if (MODE == 0) okc += mbar_try_wait(&bar, 0) ? 1 : 0;
            else if (MODE == 1) okc += mbar_test_wait(&bar, 0) ? 1 : 0;
            else okc += mbar_wait(&bar, 0, &ctl, nullptr, 1) ? 1 : 0;
        }
    }
    __syncthreads();
    t1 = clock64();
    if (threadIdx.x == 0) { out[0] = t1 - t0; out[1] = okc; }
}
int main()
{
    long long* d; CK(cudaMalloc(&d, 16));
    long long h[2];
    const int reps = 64;
    for (int mode = 0; mode < 4; ++mode)
        for (int n : {1, 32, 128, 512}) {
            if (mode == 3 && n > 16) continue;
            if (mode == 0) wait_cost_kernel<0><<<1, 512>>>(n, reps, d);
            else if (mode == 1) wait_cost_kernel<1><<<1, 512>>>(n, reps, d);
            else if (mode == 2) wait_cost_kernel<2><<<1, 512>>>(n, reps, d);
            else wait_cost_kernel<3><<<1, 512>>>(n, reps, d);
            CK(cudaDeviceSynchronize());
            CK(cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost));
            printf("%s, %3d %s: %.1f clocks per wait (ok %lld of %d)\n", mode == 0 ? "try_wait" : mode == 1 ? "test_wait" : mode == 2 ? "mbar_wait" : "mbar_wait lane0 of",
                   n, mode == 3 ? "warps" : "threads", (double)h[0] / reps, h[1], reps);
        }
    return 0;
}
