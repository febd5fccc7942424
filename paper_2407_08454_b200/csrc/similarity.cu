// Cosine similarity of neighbouring key states (Eq. 2, evaluated only on the
// |i-j| = 1 pairs Algorithm 1 consumes):  sim_j = <k_{j-1},k_j> / (|k_{j-1}| |k_j|).
// Bandwidth-bound: every key row is read once with 16-byte loads.  A group of
// LPR lanes owns one row at a time and walks a run of consecutive tokens four
// rows per round, so each row's norm is computed once and reused for both of
// its pairs.  The eight partial sums of a round (4 norms, 4 dot products) are
// reduced across the lane group with one transposing butterfly (8 shuffles
// instead of 32), in a fixed order.
#include "common.cuh"

namespace kvm {
namespace {

#ifndef KVM_SIM_CHUNK
#define KVM_SIM_CHUNK 8
#endif
constexpr int CHUNK = KVM_SIM_CHUNK;  // consecutive tokens per lane group
constexpr int RPR = 4;     // rows per round

__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ float hsum(uint64_t p) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
    return lo + hi;
}

template <typename T, int D>
__global__ void __launch_bounds__(256) similarity_kernel(const T* __restrict__ K, float* __restrict__ sim,
                                                         int S, long long n_groups, int chunks_per_unit) {
    constexpr int N = Vec<T>::N;          // elements per 16-byte load
    constexpr int NP = N / 2;             // packed pairs per load
    constexpr int LPR = D / N;            // lanes per row (8, 16 or 32)
    static_assert(LPR >= 8, "the butterfly needs at least 8 lanes per row");
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_groups) return;          // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const int gbase = (threadIdx.x % 32) / LPR * LPR;     // first warp lane of this group
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << gbase);
    const long long u = gid / chunks_per_unit;
    const int j0 = (int)(gid % chunks_per_unit) * CHUNK;
    const int j1 = min(j0 + CHUNK, S);
    const T* Ku = K + (size_t)u * S * D;
    float* su = sim + (size_t)u * S;

    // previous row (token j0 - 1) as packed pairs, and its squared norm
    uint64_t prev[NP];
    float pn2 = 0.f;
    {
        float f[N];
        if (j0 > 0) Vec<T>::unpack(ldg16(Ku + (size_t)(j0 - 1) * D + lane * N), f);
        else {
#pragma unroll
            for (int e = 0; e < N; ++e) f[e] = 0.f;
        }
        uint64_t a = 0ull;
#pragma unroll
        for (int e = 0; e < NP; ++e) { prev[e] = pk2(f[2 * e], f[2 * e + 1]); a = fma2(prev[e], prev[e], a); }
        pn2 = hsum(a);
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) pn2 += __shfl_xor_sync(gmask, pn2, off);
    }
    // Butterfly over three lane bits at distances SH, SH/2, SH/4 (SH = 8, or 4 for 8-lane groups).  Afterwards a
    // lane holds value (bA*4 + bB*2 + bC) of {n2[0..3], dot[0..3]}; any remaining low bit only replicates.
    constexpr int SH = (LPR >= 16) ? 8 : 4;
    const int b3 = (lane / SH) & 1, b2 = (lane / (SH / 2)) & 1, b1 = (lane / (SH / 4)) & 1;
    const int k = b2 * 2 + b1;                            // row of the round this lane finishes

    for (int jb = j0; jb < j1; jb += RPR) {
        uint4 raw[RPR];
#pragma unroll
        for (int r = 0; r < RPR; ++r)
            raw[r] = (jb + r < j1) ? ldg16(Ku + (size_t)(jb + r) * D + lane * N) : make_uint4(0, 0, 0, 0);
        float val[2 * RPR];                               // n2[0..3], dot[0..3] partial sums of this lane
#pragma unroll
        for (int r = 0; r < RPR; ++r) {
            float f[N];
            Vec<T>::unpack(raw[r], f);
            uint64_t an = 0ull, ad = 0ull;
#pragma unroll
            for (int e = 0; e < NP; ++e) {
                const uint64_t c = pk2(f[2 * e], f[2 * e + 1]);
                an = fma2(c, c, an);
                ad = fma2(c, prev[e], ad);
                prev[e] = c;
            }
            val[r] = hsum(an);
            val[RPR + r] = hsum(ad);
        }
        // lanes beyond 16 per row (LPR = 32) first fold onto the lower 16
        if (LPR == 32) {
#pragma unroll
            for (int i = 0; i < 2 * RPR; ++i) val[i] += __shfl_xor_sync(gmask, val[i], 16);
        }
        float s4[4], s2[2], s1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float mine = b3 ? val[4 + i] : val[i], other = b3 ? val[i] : val[4 + i];
            s4[i] = mine + __shfl_xor_sync(gmask, other, SH);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float mine = b2 ? s4[2 + i] : s4[i], other = b2 ? s4[i] : s4[2 + i];
            s2[i] = mine + __shfl_xor_sync(gmask, other, SH / 2);
        }
        {
            const float mine = b1 ? s2[1] : s2[0], other = b1 ? s2[0] : s2[1];
            s1 = mine + __shfl_xor_sync(gmask, other, SH / 4);
        }
        if (SH / 4 == 2) s1 += __shfl_xor_sync(gmask, s1, 1);
        // gather the two norms next to each dot product: lane k * SH/4 (bA = 0) holds n2[k]
        const float n2k = __shfl_sync(gmask, s1, gbase + k * (SH / 4));
        const float n2km1 = __shfl_sync(gmask, s1, gbase + ((k + 3) & 3) * (SH / 4));
        const float n2last = __shfl_sync(gmask, s1, gbase + 3 * (SH / 4));
        const float nprev = (k == 0) ? pn2 : n2km1;
        const int j = jb + k;
        if (b3 == 1 && lane % (SH / 4) == 0 && lane < 2 * SH && j < j1) {
            float c = 0.f;
            if (j > 0 && nprev > 0.f && n2k > 0.f) {
                c = s1 / (sqrtf(nprev) * sqrtf(n2k));
                c = fminf(1.f, fmaxf(-1.f, c)) + 0.f;     // |cos| <= 1; no negative zero
            }
            su[j] = c;
        }
        pn2 = n2last;
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
