// Gaussian-kernel weighted merge of every merging set into one state, written
// densely in token order (Eq. 4 with fixed sigma, Eq. 5, Definition 4.2,
// Algorithm 2):
//   g_j = exp(-|k_p - k_j|^2 / (2 sigma^2)),  K* = sum g_j k_j / sum g_j,
//   V* = n * sum g_j v_j / sum g_j.
// Bandwidth-bound: K and V are each read once with 16-byte loads (the pivot
// row is read a second time, from cache).  A group of LPR lanes owns one output
// row and walks its set; fp32 accumulation; one round-to-nearest-even
// conversion at the store.  Sets of one token are copied bit for bit.
#include "common.cuh"

namespace kvm {
namespace {

constexpr float LOG2E = 1.4426950408889634f;

template <typename T, int D>
__global__ void __launch_bounds__(256) merge_compact_kernel(const T* __restrict__ K, const T* __restrict__ V,
                                                            const int32_t* __restrict__ set_start,
                                                            const int32_t* __restrict__ pivot,
                                                            const int32_t* __restrict__ out_len,
                                                            T* __restrict__ K_out, T* __restrict__ V_out,
                                                            int32_t* __restrict__ out_size, int S, int cap,
                                                            long long n_rows, float neg_inv_2s2_log2e, int scale_v) {
    constexpr int N = Vec<T>::N;
    constexpr int LPR = D / N;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;   // u*cap + s
    if (row >= n_rows) return;
    const int lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    const long long u = row / cap;
    const int s = (int)(row % cap);
    if (s >= out_len[u]) return;
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const int lo = st[s], hi = st[s + 1];
    const int n = hi - lo;
    const T* Ku = K + (size_t)u * S * D + lane * N;
    const T* Vu = V + (size_t)u * S * D + lane * N;
    T* ko = K_out + (size_t)row * D + lane * N;
    T* vo = V_out + (size_t)row * D + lane * N;
    if (lane == 0 && out_size) out_size[row] = n;

    if (n == 1) {
        *reinterpret_cast<uint4*>(ko) = ldg16(Ku + (size_t)lo * D);
        *reinterpret_cast<uint4*>(vo) = ldg16(Vu + (size_t)lo * D);
        return;
    }
    const int p = pivot[row];
    float kp[N];
    Vec<T>::unpack(ldg16(Ku + (size_t)p * D), kp);
    float accK[N], accV[N], gsum = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) { accK[e] = 0.f; accV[e] = 0.f; }

    for (int jb = lo; jb < hi; jb += 2) {
        const bool two = (jb + 1 < hi);
        const uint4 rk0 = ldg16(Ku + (size_t)jb * D);
        const uint4 rv0 = ldg16(Vu + (size_t)jb * D);
        const uint4 rk1 = two ? ldg16(Ku + (size_t)(jb + 1) * D) : make_uint4(0, 0, 0, 0);
        const uint4 rv1 = two ? ldg16(Vu + (size_t)(jb + 1) * D) : make_uint4(0, 0, 0, 0);
        float k0[N], v0[N], k1[N], v1[N];
        Vec<T>::unpack(rk0, k0); Vec<T>::unpack(rv0, v0);
        Vec<T>::unpack(rk1, k1); Vec<T>::unpack(rv1, v1);
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int e = 0; e < N; ++e) {
            const float a = kp[e] - k0[e], b = kp[e] - k1[e];
            d0 = fmaf(a, a, d0);
            d1 = fmaf(b, b, d1);
        }
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) {
            d0 += __shfl_xor_sync(gmask, d0, off);
            d1 += __shfl_xor_sync(gmask, d1, off);
        }
        const float g0 = exp2f(d0 * neg_inv_2s2_log2e);
        const float g1 = two ? exp2f(d1 * neg_inv_2s2_log2e) : 0.f;
        gsum += g0 + g1;
#pragma unroll
        for (int e = 0; e < N; ++e) {
            accK[e] = fmaf(g0, k0[e], accK[e]);
            accV[e] = fmaf(g0, v0[e], accV[e]);
            accK[e] = fmaf(g1, k1[e], accK[e]);
            accV[e] = fmaf(g1, v1[e], accV[e]);
        }
    }
    const float inv = 1.f / gsum;                       // gsum >= 1: the pivot's own weight is exp(0)
    const float vmul = scale_v ? (float)n * inv : inv;
#pragma unroll
    for (int e = 0; e < N; ++e) { accK[e] *= inv; accV[e] *= vmul; }
    *reinterpret_cast<uint4*>(ko) = Vec<T>::pack(accK);
    *reinterpret_cast<uint4*>(vo) = Vec<T>::pack(accV);
}

template <typename T, int D>
cudaError_t launch_t(const Dims& d, const void* K, const void* V, const int32_t* set_start, const int32_t* pivot,
                     const int32_t* out_len, void* K_out, void* V_out, int32_t* out_size, cudaStream_t st) {
    constexpr int LPR = D / Vec<T>::N;
    const long long rows = (long long)d.U * d.cap;
    const long long threads = rows * LPR;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    const float c = -LOG2E / (2.f * d.sigma * d.sigma);
    merge_compact_kernel<T, D><<<blocks, 256, 0, st>>>((const T*)K, (const T*)V, set_start, pivot, out_len,
                                                       (T*)K_out, (T*)V_out, out_size, d.S, d.cap, rows, c,
                                                       d.scale_v);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_merge(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                         const int32_t* pivot, const int32_t* out_len, void* K_out, void* V_out,
                         int32_t* out_size, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128
                   ? launch_t<__nv_bfloat16, 128>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st)
                   : launch_t<__nv_bfloat16, 64>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st);
    }
    return d.D == 128 ? launch_t<float, 128>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st)
                      : launch_t<float, 64>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st);
}

}  // namespace kvm
