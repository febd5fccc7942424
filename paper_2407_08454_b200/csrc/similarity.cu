// Cosine similarity of neighbouring key states (Eq. 2, evaluated only on the
// |i-j| = 1 pairs Algorithm 1 consumes):  sim_j = <k_{j-1},k_j> / (|k_{j-1}| |k_j|).
// Bandwidth-bound: every key row is read once with 16-byte loads; a group of
// LPR lanes owns one row at a time and walks a short run of consecutive tokens,
// so each row's norm is computed once and reused for both of its pairs.
#include "common.cuh"

namespace kvm {
namespace {

constexpr int CHUNK = 16;  // consecutive tokens per lane group

template <typename T, int D>
__global__ void __launch_bounds__(256) similarity_kernel(const T* __restrict__ K, float* __restrict__ sim,
                                                         int S, long long n_groups, int chunks_per_unit) {
    constexpr int N = Vec<T>::N;          // elements per 16-byte load
    constexpr int LPR = D / N;            // lanes per row
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_groups) return;          // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    const long long u = gid / chunks_per_unit;
    const int j0 = (int)(gid % chunks_per_unit) * CHUNK;
    const int j1 = min(j0 + CHUNK, S);
    const T* Ku = K + (size_t)u * S * D;
    float* su = sim + (size_t)u * S;

    float prev[N], pn2 = 0.f;
    if (j0 > 0) {
        Vec<T>::unpack(ldg16(Ku + (size_t)(j0 - 1) * D + lane * N), prev);
#pragma unroll
        for (int e = 0; e < N; ++e) pn2 = fmaf(prev[e], prev[e], pn2);
    } else {
#pragma unroll
        for (int e = 0; e < N; ++e) prev[e] = 0.f;
    }
#pragma unroll
    for (int off = 1; off < LPR; off <<= 1) pn2 += __shfl_xor_sync(gmask, pn2, off);

    for (int jb = j0; jb < j1; jb += 4) {
        uint4 raw[4];
#pragma unroll
        for (int t = 0; t < 4; ++t)
            raw[t] = (jb + t < j1) ? ldg16(Ku + (size_t)(jb + t) * D + lane * N) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (jb + t < j1) {   // uniform within the group
                float cur[N], n2 = 0.f, dot = 0.f;
                Vec<T>::unpack(raw[t], cur);
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    n2 = fmaf(cur[e], cur[e], n2);
                    dot = fmaf(cur[e], prev[e], dot);
                }
#pragma unroll
                for (int off = 1; off < LPR; off <<= 1) {
                    n2 += __shfl_xor_sync(gmask, n2, off);
                    dot += __shfl_xor_sync(gmask, dot, off);
                }
                const int j = jb + t;
                if (lane == 0) {
                    float c = 0.f;
                    if (j > 0 && pn2 > 0.f && n2 > 0.f) {
                        c = dot / (sqrtf(pn2) * sqrtf(n2));
                        c = fminf(1.f, fmaxf(-1.f, c)) + 0.f;   // |cos| <= 1; no negative zero
                    }
                    su[j] = c;
                }
                pn2 = n2;
#pragma unroll
                for (int e = 0; e < N; ++e) prev[e] = cur[e];
            }
        }
    }
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
