// Micro-benchmark, not part of the library: clocks per tcgen05.mma (cta_group::1, kind::f16 with bf16 operands,
// M = 128, K = 16) for N = 64, 128, 256 and for a K-major and an MN-major B operand.  One CTA per SM; one thread
// issues NMMA MMAs back to back into one TMEM accumulator from fixed shared-memory operands, commits, and waits
// (bounded) for the mbarrier; clock64() before the first issue, after the last issue and after the wait.
// Every access stays inside the 100 KB of dynamic shared memory and the 512 TMEM columns the block allocates.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 --expt-relaxed-constexpr \
//        -I paper_2407_08454_b200/csrc -I include paper_2407_08454_b200/csrc/microbench/mma_rate.cu -o mma_rate -lcuda
#include <cstdio>
#include <cuda.h>
#include <cuda_runtime.h>
#include "tc_common.cuh"
using namespace kvm::tc;
constexpr int NMMA = 64;
template <int N, bool BMN>
__global__ void __launch_bounds__(128, 1) rate_kernel(long long* out) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    const uint32_t base = (smem_u32(smem) + 1023u) & ~1023u;
    for (int i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x < 32) tmem_alloc(&tmem_base_s, 512);
    tc_fence_before(); __syncthreads(); tc_fence_after();
    const uint32_t tm = tmem_base_s;
    if (threadIdx.x == 0) {
        const uint64_t da = smem_desc(base);
        const uint32_t baddr = base + 16384;
        const uint32_t idesc = idesc_bf16(N, BMN);
        long long t0 = clock64();
        for (int i = 0; i < NMMA; ++i) {
            const int ks = i & 3;
            const uint64_t db = BMN ? smem_desc_mn(baddr + ks * 16 * 128, 16384) : smem_desc(baddr + ks * 32);
            umma_bf16(tm, da + ((ks * 32) >> 4), db, idesc, i ? 1u : 0u);
        }
        long long t1 = clock64();
        umma_commit(&bar);
        mbar_wait(&bar, 0, &abort_flag);
        long long t2 = clock64();
        if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
    }
    __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after(); tmem_dealloc(tm, 512); }
}
template <int N, bool BMN> void run(const char* name, long long* d) {
    cudaFuncSetAttribute(rate_kernel<N, BMN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    for (int r = 0; r < 3; ++r) rate_kernel<N, BMN><<<148, 128, 100 * 1024>>>(d);
    cudaError_t e = cudaDeviceSynchronize();
    long long h[2];
    cudaMemcpy(h, d, sizeof(h), cudaMemcpyDeviceToHost);
    printf("%-22s err=%d issue %.1f clk/MMA, complete %.1f clk/MMA\n", name, (int)e, (double)h[0] / NMMA, (double)h[1] / NMMA);
}
int main() {
    long long* d; cudaMalloc(&d, 64);
    run<64, false>("N=64  B K-major", d);
    run<128, false>("N=128 B K-major", d);
    run<256, false>("N=256 B K-major", d);
    run<128, true>("N=128 B MN-major", d);
    return 0;
}
