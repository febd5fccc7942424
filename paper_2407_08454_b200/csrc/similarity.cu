// Cosine similarity of neighbouring key states (Eq. 2, evaluated only on the
// |i-j| = 1 pairs Algorithm 1 consumes):  sim_j = <k_{j-1},k_j> / (|k_{j-1}| |k_j|).
// Bandwidth-bound: every key row is read once with 16-byte loads.  A group of
// LPR lanes owns one row at a time and walks a run of consecutive tokens four
// rows per round (similarity_core.cuh), so each row's norm is computed once and
// reused for both of its pairs.
#include "similarity_core.cuh"

namespace kvm {
namespace {

#ifndef KVM_SIM_CHUNK
#define KVM_SIM_CHUNK 8
#endif
constexpr int CHUNK = KVM_SIM_CHUNK;  // consecutive tokens per lane group

template <typename T, int D>
__global__ void __launch_bounds__(256) similarity_kernel(const T* __restrict__ K, float* __restrict__ sim,
                                                         int S, long long n_groups, int chunks_per_unit) {
    constexpr int LPR = D / Vec<T>::N;    // lanes per row (8, 16 or 32)
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_groups) return;          // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const int gbase = (threadIdx.x % 32) / LPR * LPR;     // first warp lane of this group
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << gbase);
    const long long u = gid / chunks_per_unit;
    const int j0 = (int)(gid % chunks_per_unit) * CHUNK;
    simcore::run<T, D, CHUNK>(K + (size_t)u * S * D, sim + (size_t)u * S, j0, min(j0 + CHUNK, S), lane, gbase, gmask);
}

template <typename T, int D>
cudaError_t launch_t(const Dims& d, const void* K, float* sim, cudaStream_t st) {
    constexpr int LPR = D / Vec<T>::N;
    const int chunks = (d.S + CHUNK - 1) / CHUNK;
    const long long groups = (long long)d.U * chunks;
    const long long threads = groups * LPR;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    similarity_kernel<T, D><<<blocks, 256, 0, st>>>((const T*)K, sim, d.S, groups, chunks);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_similarity(const Dims& d, const void* K, float* sim, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128 ? launch_t<__nv_bfloat16, 128>(d, K, sim, st) : launch_t<__nv_bfloat16, 64>(d, K, sim, st);
    }
    return d.D == 128 ? launch_t<float, 128>(d, K, sim, st) : launch_t<float, 64>(d, K, sim, st);
}

}  // namespace kvm
