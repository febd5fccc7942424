// One decode step of attention over a cache whose units may have different
// lengths (Eq. 1: O_t = softmax(q_t K^T / sqrt(d)) V), and the output
// perturbation |O_t - O_t*| of Definition 2.1 between the full and the
// compressed cache.
//
// Bandwidth-bound: every K and V row of the cache is read once per query head
// (the G query heads of a KV head read the same rows within a short time, so
// the repeats are L2 hits).  The rows of one (batch, query head) are split into
// chunks sized so that the blocks fill the GPU in one wave, one block per chunk; inside a block a group of LPR
// lanes owns a row at a time and keeps an online-softmax state (max, sum,
// weighted V sum) in registers; groups, then chunks, are combined in a fixed
// order, so results are reproducible.
#include "common.cuh"

namespace kvm {
namespace {

constexpr int ATT_NT = 256;
constexpr int ATT_MIN_CHUNK = 64;           // fewest cache rows a block is given (bounds the number of chunks)
constexpr int ATT_BLOCKS_PER_SM = 4;        // resident blocks per SM (register-limited): the chunk count aims at one wave
constexpr float LOG2E = 1.4426950408889634f;

// Weight of a partial state with maximum m when the overall maximum is M (an empty state has m = -inf).
__device__ __forceinline__ float rescale(float m, float M) { return m == -INFINITY ? 0.f : exp2f(m - M); }

// part layout per (bh, split): D weighted sums, then the maximum and the sum (log2 domain).
template <typename T, int D>
__global__ void __launch_bounds__(ATT_NT) attend_partial_kernel(const T* __restrict__ q, const T* __restrict__ K,
                                                                const T* __restrict__ V,
                                                                const int32_t* __restrict__ len,
                                                                float* __restrict__ part, int rows, int chunk, int G,
                                                                int Hq, int Hkv, float scale_log2e) {
    constexpr int N = Vec<T>::N, LPR = D / N, NGRP = ATT_NT / LPR;
    __shared__ float sm_m[NGRP], sm_l[NGRP];
    __shared__ __align__(16) float sm_acc[NGRP][D];
    const int split = blockIdx.x, nsplit = gridDim.x;
    const int bh = blockIdx.y;
    const int b = bh / Hq, h = bh % Hq;
    const long long u = (long long)b * Hkv + h / G;
    const int n = len ? max(0, min(len[u], rows)) : rows;
    const int r0 = split * chunk, r1 = min(r0 + chunk, n);
    const int grp = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    const T* Ku = K + (size_t)u * rows * D;
    const T* Vu = V + (size_t)u * rows * D;

    float qf[N];
    Vec<T>::unpack(ldg16(q + (size_t)bh * D + lane * N), qf);
    float m = -INFINITY, l = 0.f, acc[N];
#pragma unroll
    for (int e = 0; e < N; ++e) acc[e] = 0.f;
    // RPI rows per iteration: their loads are independent and in flight together; one rescale per iteration
#ifndef KVM_ATT_RPI
#define KVM_ATT_RPI 4
#endif
    constexpr int RPI = KVM_ATT_RPI;
    for (int r = r0 + grp * RPI; r < r1; r += NGRP * RPI) {
        uint4 kraw[RPI], vraw[RPI];
#pragma unroll
        for (int i = 0; i < RPI; ++i) {
            const int ri = min(r + i, r1 - 1);                   // clamped rows are loaded but given no weight
            kraw[i] = ldg16(Ku + (size_t)ri * D + lane * N);
            vraw[i] = ldg16(Vu + (size_t)ri * D + lane * N);
        }
        float s[RPI];
#pragma unroll
        for (int i = 0; i < RPI; ++i) {
            float kf[N];
            Vec<T>::unpack(kraw[i], kf);
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < N; ++e) dot = fmaf(qf[e], kf[e], dot);
            s[i] = dot;
        }
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) {
#pragma unroll
            for (int i = 0; i < RPI; ++i) s[i] += __shfl_xor_sync(gmask, s[i], off);
        }
        float mn = m;
#pragma unroll
        for (int i = 0; i < RPI; ++i) {
            s[i] = (r + i < r1) ? s[i] * scale_log2e : -INFINITY;
            mn = fmaxf(mn, s[i]);
        }
        const float corr = exp2f(m - mn);                        // first iteration: exp2(-inf) = 0
        l *= corr;
#pragma unroll
        for (int e = 0; e < N; ++e) acc[e] *= corr;
#pragma unroll
        for (int i = 0; i < RPI; ++i) {
            const float pj = exp2f(s[i] - mn);                   // 0 for a clamped row
            float vf[N];
            Vec<T>::unpack(vraw[i], vf);
            l += pj;
#pragma unroll
            for (int e = 0; e < N; ++e) acc[e] = fmaf(pj, vf[e], acc[e]);
        }
        m = mn;
    }
    if (lane == 0) { sm_m[grp] = m; sm_l[grp] = l; }
#pragma unroll
    for (int e = 0; e < N; ++e) sm_acc[grp][lane * N + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < D) {
        float M = -INFINITY;
#pragma unroll
        for (int g = 0; g < NGRP; ++g) M = fmaxf(M, sm_m[g]);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int g = 0; g < NGRP; ++g) {
            const float w = rescale(sm_m[g], M);
            L = fmaf(sm_l[g], w, L);
            o = fmaf(sm_acc[g][threadIdx.x], w, o);
        }
        float* dst = part + ((size_t)bh * nsplit + split) * (D + 2);
        dst[threadIdx.x] = o;
        if (threadIdx.x == 0) { dst[D] = M; dst[D + 1] = L; }
    }
}

template <int D>
__global__ void __launch_bounds__(D) attend_combine_kernel(const float* __restrict__ part, float* __restrict__ out,
                                                           int nsplit) {
    grid_dependency_wait();     // the partial states come from the kernel before this one
    const int bh = blockIdx.x;
    const float* p = part + (size_t)bh * nsplit * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p[(size_t)s * (D + 2) + D]);
    float L = 0.f, o = 0.f;
    for (int s = 0; s < nsplit; ++s) {
        const float* ps = p + (size_t)s * (D + 2);
        const float w = rescale(ps[D], M);
        L = fmaf(ps[D + 1], w, L);
        o = fmaf(ps[threadIdx.x], w, o);
    }
    out[(size_t)bh * D + threadIdx.x] = L > 0.f ? o / L : 0.f;     // an empty cache attends to nothing
}

// err = |O - O*|_2 and ref = |O|_2 per (batch, query head).
template <int D>
__global__ void __launch_bounds__(D) perturbation_kernel(const float* __restrict__ O, const float* __restrict__ Os,
                                                         float* __restrict__ err, float* __restrict__ ref) {
    __shared__ float se[D / 32], sr[D / 32];
    grid_dependency_wait();     // both attention outputs come from the kernels before this one
    const int bh = blockIdx.x;
    const float a = O[(size_t)bh * D + threadIdx.x], c = Os[(size_t)bh * D + threadIdx.x];
    float e = (a - c) * (a - c), r = a * a;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        e += __shfl_xor_sync(0xffffffffu, e, off);
        r += __shfl_xor_sync(0xffffffffu, r, off);
    }
    if ((threadIdx.x & 31) == 0) { se[threadIdx.x >> 5] = e; sr[threadIdx.x >> 5] = r; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float te = 0.f, tr = 0.f;
#pragma unroll
        for (int w = 0; w < D / 32; ++w) { te += se[w]; tr += sr[w]; }
        err[bh] = sqrtf(te);
        ref[bh] = sqrtf(tr);
    }
}

template <typename T, int D>
cudaError_t launch_t(const Dims& d, const void* q, const void* K, const void* V, int rows, const int32_t* len,
                     float* out, float* part, cudaStream_t st) {
    // as many chunks per head as keep every SM's resident blocks busy in a single wave, within the scratch bound
    int dev = 0, sms = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 == cudaSuccess) e0 = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e0 != cudaSuccess) return e0;
    int want = (ATT_BLOCKS_PER_SM * sms) / (d.B * d.Hq);
    want = want < 1 ? 1 : (want > attend_splits(rows) ? attend_splits(rows) : want);
    const int chunk = (rows + want - 1) / want;
    const int nsplit = (rows + chunk - 1) / chunk;
    attend_partial_kernel<T, D><<<dim3(nsplit, d.B * d.Hq), ATT_NT, 0, st>>>(
        (const T*)q, (const T*)K, (const T*)V, len, part, rows, chunk, d.G, d.Hq, d.Hkv, d.scale * LOG2E);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_dependent(attend_combine_kernel<D>, dim3(d.B * d.Hq), dim3(D), 0, st, (const float*)part, out, nsplit);
}

}  // namespace

// Upper bound on the chunks per head (what the scratch is sized for).
int attend_splits(int rows) { return (rows + ATT_MIN_CHUNK - 1) / ATT_MIN_CHUNK; }

size_t attend_scratch_floats(const Dims& d) { return (size_t)d.B * d.Hq * attend_splits(d.S) * (d.D + 2); }

cudaError_t launch_attend(const Dims& d, const void* q, const void* K, const void* V, int rows, const int32_t* len,
                          float* out, float* part, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128 ? launch_t<__nv_bfloat16, 128>(d, q, K, V, rows, len, out, part, st)
                          : launch_t<__nv_bfloat16, 64>(d, q, K, V, rows, len, out, part, st);
    }
    return d.D == 128 ? launch_t<float, 128>(d, q, K, V, rows, len, out, part, st)
                      : launch_t<float, 64>(d, q, K, V, rows, len, out, part, st);
}

cudaError_t launch_perturbation(const Dims& d, const float* O, const float* Os, float* err, float* ref,
                                cudaStream_t st) {
    if (d.D == 128) return launch_dependent(perturbation_kernel<128>, dim3(d.B * d.Hq), dim3(128), 0, st, O, Os, err, ref);
    return launch_dependent(perturbation_kernel<64>, dim3(d.B * d.Hq), dim3(64), 0, st, O, Os, err, ref);
}

}  // namespace kvm
