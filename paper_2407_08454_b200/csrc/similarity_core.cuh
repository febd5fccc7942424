// Cosine similarity of neighbouring key states (Eq. 2 on the |i-j| = 1 pairs Algorithm 1 consumes):
// the work of one lane group on one run of consecutive tokens.  Shared by the stand-alone similarity
// kernel and by the score kernel's row pass, whose spare warps compute the similarities on the side.
#pragma once
#include "common.cuh"

namespace kvm {
namespace simcore {

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

// Tokens [j0, j1) of one unit (Ku = its first key row, su = its similarity row), handled by the LPR = D / N
// lanes of one group: `lane` in [0, LPR), `gbase` = the group's first lane within the warp, `gmask` = its
// lane mask.  Each row's norm is computed once and reused for both of its pairs; four rows per round, whose
// eight partial sums (4 norms, 4 dot products) are reduced with one transposing butterfly, in a fixed order.
// All rows of the run (at most CH, a multiple of 4) and the row before it are requested up front, so a run
// costs one memory round trip.
template <typename T, int D, int CH>
__device__ __forceinline__ void run(const T* __restrict__ Ku, float* __restrict__ su, int j0, int j1, int lane,
                                    int gbase, unsigned gmask) {
    static_assert(CH % RPR == 0, "runs are whole rounds");
    constexpr int N = Vec<T>::N;          // elements per 16-byte load
    constexpr int NP = N / 2;             // packed pairs per load
    constexpr int LPR = D / N;            // lanes per row (8, 16 or 32)
    static_assert(LPR >= 8, "the butterfly needs at least 8 lanes per row");
    // previous row (token j0 - 1) as packed pairs, and its squared norm
    uint4 rows[CH];
    const uint4 rowp = (j0 > 0) ? ldg16(Ku + (size_t)(j0 - 1) * D + lane * N) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int r = 0; r < CH; ++r)
        rows[r] = (j0 + r < j1) ? ldg16(Ku + (size_t)(j0 + r) * D + lane * N) : make_uint4(0, 0, 0, 0);
    uint64_t prev[NP];
    float pn2 = 0.f;
    {
        float f[N];
        Vec<T>::unpack(rowp, f);          // all-zero bits are 0.0 in both storage types
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

#pragma unroll
    for (int rd = 0; rd < CH / RPR; ++rd) {
        const int jb = j0 + rd * RPR;
        if (jb >= j1) break;
        float val[2 * RPR];                               // n2[0..3], dot[0..3] partial sums of this lane
#pragma unroll
        for (int r = 0; r < RPR; ++r) {
            float f[N];
            Vec<T>::unpack(rows[rd * RPR + r], f);
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

}  // namespace simcore
}  // namespace kvm
