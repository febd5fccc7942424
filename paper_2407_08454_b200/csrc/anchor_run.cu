// Run lengths for the "anchor" reading of the set identification (Section 3.2): for every token i, the
// number of consecutive predecessors j = i-1, i-2, ... whose cosine similarity to k_i exceeds epsilon
// (Eq. 2, the pair (i, j) instead of neighbours).  The segment kernel turns them into merging sets.
//
// A first kernel stores 1 / |k_j| per token.  Then one lane group (LPR lanes, 16 bytes of the row each) per token
// walks backwards, four rows per round trip and one dot product per pair; the rows are neighbours of rows other
// groups read, so after the first touch they are cache hits.
#include "common.cuh"

namespace kvm {
namespace {

constexpr int RPI = 4;      // predecessors fetched per round trip (evaluated in order)

// 1 / |k_j| per token (0 for a zero row), so that the walk below needs one dot product per pair.
template <typename T, int D>
__global__ void __launch_bounds__(256) key_inv_norm_kernel(const T* __restrict__ K, float* __restrict__ inv_norm,
                                                           long long n_rows) {
    constexpr int N = Vec<T>::N, LPR = D / N;
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_rows) return;
    const int lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    float k[N];
    Vec<T>::unpack(ldg16(K + (size_t)gid * D + lane * N), k);
    float n2 = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) n2 = fmaf(k[e], k[e], n2);
#pragma unroll
    for (int off = 1; off < LPR; off <<= 1) n2 += __shfl_xor_sync(gmask, n2, off);
    if (lane == 0) inv_norm[gid] = n2 > 0.f ? rsqrtf(n2) : 0.f;
}

template <typename T, int D>
__global__ void __launch_bounds__(256) anchor_run_kernel(const T* __restrict__ K, const float* __restrict__ inv_norm,
                                                         float* __restrict__ run_out, int S, long long n_rows,
                                                         float eps) {
    constexpr int N = Vec<T>::N, LPR = D / N;
    static_assert(LPR >= 8, "the transposing reduction needs at least 8 lanes per row");
    grid_dependency_wait();                                // the inverse norms come from the kernel before this one
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_rows) return;                             // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const int gbase = (threadIdx.x % 32) / LPR * LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << gbase);
    const long long u = gid / S;
    const int i = (int)(gid % S);
    const T* Ku = K + (size_t)u * S * D;
    const float* inv_u = inv_norm + (size_t)u * S;

    float ki[N];
    Vec<T>::unpack(ldg16(Ku + (size_t)i * D + lane * N), ki);
    const float inv_i = __ldcg(inv_u + i);
    const int hiA = (lane / (LPR / 2)) & 1, hiB = (lane / (LPR / 4)) & 1;

    int r = 0;
    bool go = true;                                        // uniform across the lane group
    for (int j = i - 1; go && j >= 0; j -= RPI) {
        uint4 raw[RPI];
#pragma unroll
        for (int t = 0; t < RPI; ++t) raw[t] = ldg16(Ku + (size_t)max(j - t, 0) * D + lane * N);
        const float inv_j = __ldcg(inv_u + max(j - (lane & 3), 0));      // lanes 0..3 (mod 4) hold the four rows' values
        float dot[RPI];
#pragma unroll
        for (int t = 0; t < RPI; ++t) {
            float kj[N];
            Vec<T>::unpack(raw[t], kj);
            dot[t] = 0.f;
#pragma unroll
            for (int e = 0; e < N; ++e) dot[t] = fmaf(ki[e], kj[e], dot[t]);
        }
        // four sums over the lane group with a transposing butterfly: 2 + 1 exchanges, then a plain reduction of
        // the one value left per lane; value t ends up in the lanes with (hiA, hiB) = (t >> 1, t & 1)
        const float a0 = (hiA ? dot[2] : dot[0]) + __shfl_xor_sync(gmask, hiA ? dot[0] : dot[2], LPR / 2);
        const float a1 = (hiA ? dot[3] : dot[1]) + __shfl_xor_sync(gmask, hiA ? dot[1] : dot[3], LPR / 2);
        float b = (hiB ? a1 : a0) + __shfl_xor_sync(gmask, hiB ? a0 : a1, LPR / 4);
#pragma unroll
        for (int off = LPR / 8; off >= 1; off >>= 1) b += __shfl_xor_sync(gmask, b, off);
#pragma unroll
        for (int t = 0; t < RPI; ++t) {
            const float d = __shfl_sync(gmask, b, gbase + (t >> 1) * (LPR / 2) + (t & 1) * (LPR / 4));
            const float ij = __shfl_sync(gmask, inv_j, gbase + t);
            if (!go || j - t < 0) { go = false; continue; }
            const float c = fminf(1.f, fmaxf(-1.f, d * inv_i * ij));     // 0 when either row is zero
            if (c > eps) ++r; else go = false;
        }
    }
    if (lane == 0) run_out[gid] = (float)r;               // at most 65535: exact in fp32
}

template <typename T, int D>
cudaError_t launch_t(const Dims& d, const void* K, float* run_out, float* inv_norm, cudaStream_t st) {
    constexpr int LPR = D / Vec<T>::N;
    const long long rows = (long long)d.U * d.S;
    const unsigned blocks = (unsigned)((rows * LPR + 255) / 256);
    key_inv_norm_kernel<T, D><<<blocks, 256, 0, st>>>((const T*)K, inv_norm, rows);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_dependent(anchor_run_kernel<T, D>, dim3(blocks), dim3(256), 0, st, (const T*)K,
                            (const float*)inv_norm, run_out, d.S, rows, d.eps);
}

}  // namespace

// inv_norm: [U,S] fp32 of scratch.
cudaError_t launch_anchor_runs(const Dims& d, const void* K, float* run_out, float* inv_norm, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128 ? launch_t<__nv_bfloat16, 128>(d, K, run_out, inv_norm, st)
                          : launch_t<__nv_bfloat16, 64>(d, K, run_out, inv_norm, st);
    }
    return d.D == 128 ? launch_t<float, 128>(d, K, run_out, inv_norm, st)
                      : launch_t<float, 64>(d, K, run_out, inv_norm, st);
}

}  // namespace kvm
