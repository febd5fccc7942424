// Run lengths for the "anchor" reading of the set identification (Section 3.2): for every token i, the
// number of consecutive predecessors j = i-1, i-2, ... whose cosine similarity to k_i exceeds epsilon
// (Eq. 2, the pair (i, j) instead of neighbours).  The segment kernel turns them into merging sets.
//
// One lane group (LPR lanes, 16 bytes of the row each) per token walks backwards, four rows per round
// trip; the rows are neighbours of rows other groups read, so after the first touch they are cache hits.
#include "common.cuh"

namespace kvm {
namespace {

constexpr int RPI = 4;      // predecessors fetched per round trip (evaluated in order)

template <typename T, int D>
__global__ void __launch_bounds__(256) anchor_run_kernel(const T* __restrict__ K, float* __restrict__ run_out,
                                                         int S, long long n_rows, float eps) {
    constexpr int N = Vec<T>::N, LPR = D / N;
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_rows) return;                             // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    const long long u = gid / S;
    const int i = (int)(gid % S);
    const T* Ku = K + (size_t)u * S * D;

    float ki[N];
    Vec<T>::unpack(ldg16(Ku + (size_t)i * D + lane * N), ki);
    float ni = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) ni = fmaf(ki[e], ki[e], ni);
#pragma unroll
    for (int off = 1; off < LPR; off <<= 1) ni += __shfl_xor_sync(gmask, ni, off);

    int r = 0;
    bool go = true;                                        // uniform across the lane group
    for (int j = i - 1; go && j >= 0; j -= RPI) {
        uint4 raw[RPI];
#pragma unroll
        for (int t = 0; t < RPI; ++t) raw[t] = ldg16(Ku + (size_t)max(j - t, 0) * D + lane * N);
        float dot[RPI], nj[RPI];
#pragma unroll
        for (int t = 0; t < RPI; ++t) {
            float kj[N];
            Vec<T>::unpack(raw[t], kj);
            dot[t] = 0.f; nj[t] = 0.f;
#pragma unroll
            for (int e = 0; e < N; ++e) { dot[t] = fmaf(ki[e], kj[e], dot[t]); nj[t] = fmaf(kj[e], kj[e], nj[t]); }
        }
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) {
#pragma unroll
            for (int t = 0; t < RPI; ++t) {
                dot[t] += __shfl_xor_sync(gmask, dot[t], off);
                nj[t] += __shfl_xor_sync(gmask, nj[t], off);
            }
        }
#pragma unroll
        for (int t = 0; t < RPI; ++t) {
            if (!go || j - t < 0) { go = false; continue; }
            float c = 0.f;
            if (ni > 0.f && nj[t] > 0.f) {
                c = dot[t] / (sqrtf(ni) * sqrtf(nj[t]));
                c = fminf(1.f, fmaxf(-1.f, c));
            }
            if (c > eps) ++r; else go = false;
        }
    }
    if (lane == 0) run_out[gid] = (float)r;               // at most 65535: exact in fp32
}

template <typename T, int D>
cudaError_t launch_t(const Dims& d, const void* K, float* run_out, cudaStream_t st) {
    constexpr int LPR = D / Vec<T>::N;
    const long long rows = (long long)d.U * d.S;
    const unsigned blocks = (unsigned)((rows * LPR + 255) / 256);
    anchor_run_kernel<T, D><<<blocks, 256, 0, st>>>((const T*)K, run_out, d.S, rows, d.eps);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_anchor_runs(const Dims& d, const void* K, float* run_out, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128 ? launch_t<__nv_bfloat16, 128>(d, K, run_out, st) : launch_t<__nv_bfloat16, 64>(d, K, run_out, st);
    }
    return d.D == 128 ? launch_t<float, 128>(d, K, run_out, st) : launch_t<float, 64>(d, K, run_out, st);
}

}  // namespace kvm
