// Aggregated attention scores in plain fp32 FMA arithmetic (Eq. 1; Algorithm 2 / Eq. 6).
// This is the path for fp32 tensors, where tensor-core input rounding would
// not meet the score tolerance.  Two passes over 64x64 logit tiles:
//   pass 1  lse_i = ln sum_{j<=i} exp(scale * q_i.k_j)                (one block per query tile)
//   pass 2  a_j   = (1/G) sum_g sum_{i>=j} exp(scale*q_i.k_j - lse_i)  (one block per key tile)
// Reductions run in a fixed order, so results are reproducible.
#include "common.cuh"

namespace kvm {
namespace {

constexpr int TM = 64;   // tile rows (queries)
constexpr int TN = 64;   // tile cols (keys)
constexpr int TK = 32;   // depth chunk
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Stage a [64 x 32] chunk of rows [r0, r0+64) and depth [d0, d0+32) transposed into sm[32][64+4].
template <typename T>
__device__ __forceinline__ void stage_chunk(const T* __restrict__ base, int r0, int d0, int S, int D,
                                            float (*sm)[TM + 4]) {
    for (int e = threadIdx.x; e < TM * TK; e += blockDim.x) {
        const int r = e / TK, k = e % TK;
        const int row = r0 + r;
        sm[k][r] = (row < S) ? to_f32<T>(base[(size_t)row * D + d0 + k]) : 0.f;
    }
}

// acc[r][c] += sum_k Qs[k][ty*4+r] * Ks[k][tx*4+c]
__device__ __forceinline__ void mma_chunk(const float (*Qs)[TM + 4], const float (*Ks)[TN + 4], int ty, int tx,
                                          float acc[4][4]) {
#pragma unroll 8
    for (int k = 0; k < TK; ++k) {
        const float4 a = *reinterpret_cast<const float4*>(&Qs[k][ty * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&Ks[k][tx * 4]);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
    }
}

template <typename T>
__global__ void __launch_bounds__(256) lse_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                       float* __restrict__ lse, int Hq, int G, int S, int D,
                                                       float scale2) {
    __shared__ __align__(16) float Qs[TK][TM + 4];
    __shared__ __align__(16) float Ks[TK][TN + 4];
    const int it = blockIdx.x, qh = blockIdx.y;  // qh = b*Hq + h
    const int b = qh / Hq, h = qh % Hq;
    const int Hkv = Hq / G;
    const T* Qh = Q + (size_t)qh * S * D;
    const T* Kh = K + ((size_t)b * Hkv + h / G) * S * D;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;

    float m[4], l[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) { m[r] = -INFINITY; l[r] = 0.f; }

    for (int jt = 0; jt <= it; ++jt) {
        float acc[4][4] = {};
        for (int d0 = 0; d0 < D; d0 += TK) {
            __syncthreads();
            stage_chunk<T>(Qh, it * TM, d0, S, D, Qs);
            stage_chunk<T>(Kh, jt * TN, d0, S, D, Ks);
            __syncthreads();
            mma_chunk(Qs, Ks, ty, tx, acc);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int i = it * TM + ty * 4 + r;
            float s[4], mx = m[r];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int j = jt * TN + tx * 4 + c;
                s[c] = (j <= i && i < S) ? acc[r][c] * scale2 : -INFINITY;
                mx = fmaxf(mx, s[c]);
            }
            if (mx > -INFINITY) {
                float sum = l[r] * exp2f(m[r] - mx);  // m = -inf gives 0
#pragma unroll
                for (int c = 0; c < 4; ++c) sum += exp2f(s[c] - mx);
                l[r] = sum;
                m[r] = mx;
            }
        }
    }
    // combine the 16 column-threads of each row (lanes of one half-warp)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        float mm = m[r], ll = l[r];
#pragma unroll
        for (int off = 1; off < 16; off <<= 1) {
            const float mo = __shfl_xor_sync(0xffffffffu, mm, off);
            const float lo = __shfl_xor_sync(0xffffffffu, ll, off);
            const float mn = fmaxf(mm, mo);
            if (mn > -INFINITY) ll = ll * exp2f(mm - mn) + lo * exp2f(mo - mn);
            mm = mn;
        }
        const int i = it * TM + ty * 4 + r;
        if (tx == 0 && i < S) lse[(size_t)qh * S + i] = (mm + log2f(ll)) * LN2;
    }
}

template <typename T>
__global__ void __launch_bounds__(256) colsum_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                          const float* __restrict__ lse,
                                                          float* __restrict__ scores, int Hq, int G, int S, int D,
                                                          float scale2) {
    __shared__ __align__(16) float Qs[TK][TM + 4];
    __shared__ __align__(16) float Ks[TK][TN + 4];
    __shared__ float red[16][TN];
    const int jt = blockIdx.x, u = blockIdx.y;  // u = b*Hkv + hkv
    const int Hkv = Hq / G;
    const int b = u / Hkv, hk = u % Hkv;
    const T* Kh = K + (size_t)u * S * D;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    const int nT = (S + TM - 1) / TM;

    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int g = 0; g < G; ++g) {
        const size_t qh = (size_t)b * Hq + hk * G + g;
        const T* Qh = Q + qh * S * D;
        const float* lse_h = lse + qh * S;
        for (int it = jt; it < nT; ++it) {
            float acc[4][4] = {};
            for (int d0 = 0; d0 < D; d0 += TK) {
                __syncthreads();
                stage_chunk<T>(Qh, it * TM, d0, S, D, Qs);
                stage_chunk<T>(Kh, jt * TN, d0, S, D, Ks);
                __syncthreads();
                mma_chunk(Qs, Ks, ty, tx, acc);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int i = it * TM + ty * 4 + r;
                const float li = (i < S) ? lse_h[i] * LOG2E : 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int j = jt * TN + tx * 4 + c;
                    if (j <= i && i < S) col[c] += exp2f(acc[r][c] * scale2 - li);
                }
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 4; ++c) red[ty][tx * 4 + c] = col[c];
    __syncthreads();
    if (threadIdx.x < TN) {
        float s = 0.f;
#pragma unroll
        for (int y = 0; y < 16; ++y) s += red[y][threadIdx.x];
        const int j = jt * TN + threadIdx.x;
        if (j < S) scores[(size_t)u * S + j] = s / (float)G;
    }
}

}  // namespace

cudaError_t launch_score_simt(const Dims& d, const void* Q, const void* K, const float* lse_in, float* lse_ws,
                              float* scores, cudaStream_t st) {
    const int nT = (d.S + TM - 1) / TM;
    const float scale2 = d.scale * LOG2E;
    const float* lse = lse_in;
    if (d.dtype == KVM_F32) {
        if (!lse_in) {
            lse_simt_kernel<float><<<dim3(nT, d.B * d.Hq), 256, 0, st>>>((const float*)Q, (const float*)K, lse_ws,
                                                                         d.Hq, d.G, d.S, d.D, scale2);
            lse = lse_ws;
        }
        if (scores)
            colsum_simt_kernel<float><<<dim3(nT, d.U), 256, 0, st>>>((const float*)Q, (const float*)K, lse, scores,
                                                                     d.Hq, d.G, d.S, d.D, scale2);
    } else {
        if (!lse_in) {
            lse_simt_kernel<__nv_bfloat16><<<dim3(nT, d.B * d.Hq), 256, 0, st>>>(
                (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, lse_ws, d.Hq, d.G, d.S, d.D, scale2);
            lse = lse_ws;
        }
        if (scores)
            colsum_simt_kernel<__nv_bfloat16><<<dim3(nT, d.U), 256, 0, st>>>(
                (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, lse, scores, d.Hq, d.G, d.S, d.D, scale2);
    }
    return cudaGetLastError();
}

}  // namespace kvm
