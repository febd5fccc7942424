// Gaussian-kernel weighted merge of every merging set into one state, written
// densely in token order (Eq. 4 with fixed sigma, Eq. 5, Definition 4.2,
// Algorithm 2):
//   g_j = exp(-|k_p - k_j|^2 / (2 sigma^2)),  K* = sum g_j k_j / sum g_j,
//   V* = n * sum g_j v_j / sum g_j.
//
// Bandwidth-bound, and sets can be arbitrarily long, so the work is split by
// TOKENS, not by sets: a block owns TOK consecutive tokens of one unit, pulls
// their K and V rows into shared memory with two bulk copies (issued before the
// kernel even waits for the set data, which comes from the kernel before it), and
//   weights   one lane group per token computes g_j (the pivot row is taken from
//             shared memory when it lies in the tile, else from L2);
//   segments  the tile is cut where the set changes; at most TOK pieces;
//   walk      a lane group as wide as a K row and a V row together takes every fourth
//             piece: a piece that is a whole set of one token is copied, a piece that
//             is a whole set is summed (a loop of 16-byte shared-memory reads and
//             multiply-adds with no branch in it), scaled and stored; a piece of a set that reaches
//             beyond the tile leaves its fp32 sums in a scratch slot per (unit, tile):
//             "head" = the tile's tokens before its first boundary, "tail" = after its
//             last.  A small second kernel adds a crossing set's slots in tile order and
//             stores the row.
// Nothing uses atomics: every sum has a fixed order, results are reproducible.
// Sets of one token are copied bit for bit.
// Variants: average-weighted merging (Section 4.2) is the same kernel with every
// g_j = 1; pivot-only weights and eviction write single input rows (gather_rows_kernel).
#include "common.cuh"

namespace kvm {
namespace {

constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <typename T> __device__ __forceinline__ T f32_to_elem(float v);
template <> __device__ __forceinline__ float f32_to_elem<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 f32_to_elem<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// set_id[u][j] = index of the set holding token j, from the sets' start positions: one thread per set writes
// its index over the set's tokens (sets are a few tokens long on average; a long one costs its thread a loop).
__global__ void __launch_bounds__(256) token_set_kernel(const int32_t* __restrict__ set_start,
                                                        const int32_t* __restrict__ out_len,
                                                        int32_t* __restrict__ set_id, int S, int cap) {
    const int u = blockIdx.y;
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= min(out_len[u], cap)) return;
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const int beg = __ldg(st + s), end = min(__ldg(st + s + 1), S);
    int32_t* dst = set_id + (size_t)u * S;
    for (int j = beg; j < end; ++j) dst[j] = s;
}

// Scratch layout per (unit, tile): [head | tail] x (2*D sums: K channels then V channels), and 2 weight sums.
template <int D> struct Slots {
    float* sums;      // [U][T][2][2*D]
    float* gsum;      // [U][T][2]
    __device__ __forceinline__ float* s(long long u, int T, int tile, int which) const {
        return sums + (((size_t)u * T + tile) * 2 + which) * (2 * D);
    }
    __device__ __forceinline__ float* g(long long u, int T, int tile, int which) const {
        return gsum + ((size_t)u * T + tile) * 2 + which;
    }
};

// Piece kinds of the walk.
enum : int { PIECE_COPY = 0, PIECE_WHOLE = 1, PIECE_HEAD = 2, PIECE_TAIL = 3 };

template <typename T, int D, int TOK>
__global__ void __launch_bounds__(2 * D) merge_tile_kernel(const T* __restrict__ K, const T* __restrict__ V,
                                                           const int32_t* __restrict__ set_start,
                                                           const int32_t* __restrict__ pivot,
                                                           const int32_t* __restrict__ set_id,
                                                           T* __restrict__ K_out, T* __restrict__ V_out,
                                                           int32_t* __restrict__ out_size, Slots<D> slots, int S,
                                                           int cap, float neg_inv_2s2_log2e, int scale_v, int average,
                                                           const float* __restrict__ set_coef, kvm_stats* stats) {
    constexpr int NT = 2 * D;
    constexpr int N = Vec<T>::N, LPR = D / N, NG = NT / LPR;
    static_assert(TOK <= 64 && TOK <= NT, "one thread per token for the set data, two ballots for the pieces");
    extern __shared__ __align__(128) uint8_t smem_raw[];
    T* sK = reinterpret_cast<T*>(smem_raw);
    T* sV = sK + TOK * D;
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_sid[TOK], s_piv[TOK], s_len[TOK];
    __shared__ float s_g[TOK];
    __shared__ float s_coef[TOK];       // squared distance -> exponent of 2, per token (fixed sigma or the set's own)
    __shared__ int s_pbeg[TOK + 1], s_pkind[TOK], s_prow[TOK], s_pn[TOK];   // pieces: first token, kind, output row, set size
    __shared__ int s_npiece, s_warpcnt[2];

    const int tile = blockIdx.x, Tn = gridDim.x;
    const long long u = blockIdx.y;
    const int tok0 = tile * TOK;
    const int ntok = min(TOK, S - tok0);
    const int tile_end = tok0 + ntok;
    const T* Ku = K + (size_t)u * S * D;
    const T* Vu = V + (size_t)u * S * D;
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const uint32_t bytes = (uint32_t)ntok * D * sizeof(T);

    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&bar)), "r"(2 * bytes)
                     : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(sK)), "l"(Ku + (size_t)tok0 * D), "r"(bytes), "r"(smem_u32(&bar)) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(sV)), "l"(Vu + (size_t)tok0 * D), "r"(bytes), "r"(smem_u32(&bar)) : "memory");
    }
    // The K and V rows are inputs; everything read from here on comes from the kernel before this one.
    grid_dependency_wait();
    // The fix-up kernel may move in beside this grid's last blocks and look up its sets (written before this
    // kernel began, as the wait above has just established); it waits for this grid before it reads a slot.
    grid_launch_dependents();
    {
        // ---- set data per token and the pieces of the tile, while the rows are in flight
        {
            const int j = threadIdx.x;
            int sid = -1, beg = 0, end = 0;
            if (j < ntok) {
                // written by the previous kernel while this block may already have been resident: read through L2
                sid = __ldcg(set_id + (size_t)u * S + tok0 + j);
                beg = __ldcg(st + sid);
                end = __ldcg(st + sid + 1);
                s_sid[j] = sid;
                s_len[j] = end - beg;
                s_piv[j] = __ldcg(pivot + (size_t)u * cap + sid);
                s_coef[j] = set_coef ? __ldcg(set_coef + (size_t)u * cap + sid) : neg_inv_2s2_log2e;
            }
            if (j < 64) {                                     // warps 0 and 1: a piece starts where the set changes
                const int prev = __shfl_up_sync(0xffffffffu, sid, 1);
                const bool lane0 = (j & 31) == 0;
                // (lane 0 of warp 1 compares with token 31, fetched again: the shuffle does not cross warps)
                const int before = lane0 ? ((j == 0 || j >= ntok) ? -2 : __ldcg(set_id + (size_t)u * S + tok0 + j - 1)) : prev;
                const bool start = j < ntok && sid != before;
                const unsigned m = __ballot_sync(0xffffffffu, start);
                if (lane0) s_warpcnt[j >> 5] = __popc(m);
                const int below = __popc(m & ((1u << (j & 31)) - 1u));
                asm volatile("bar.sync 1, 64;" ::: "memory");   // the two warps exchange their counts
                const int idx = below + ((j >> 5) ? s_warpcnt[0] : 0);
                if (start) {
                    int kind;
                    if (end - beg == 1) kind = PIECE_COPY;
                    else if (beg >= tok0 && end <= tile_end) kind = PIECE_WHOLE;
                    else kind = (beg < tok0) ? PIECE_HEAD : PIECE_TAIL;
                    s_pbeg[idx] = j; s_pkind[idx] = kind; s_prow[idx] = sid; s_pn[idx] = end - beg;
                }
                if (j == 0) {
                    const int np = s_warpcnt[0] + s_warpcnt[1];
                    s_npiece = np;
                    s_pbeg[np] = ntok;
                }
            }
        }
        {
            // The copies were issued by this block and always complete; the wait is still bounded.  If it ever ran
            // out, the tile's staged rows are replaced by NaN patterns (so every row this block writes is NaN rather
            // than whatever shared memory held) and the condition is reported.
            uint32_t done = 1;
            if (threadIdx.x == 0) {                      // one thread polls, sparsely; the others wait at the block barrier
                done = 0;
                for (uint32_t k = 0; k < (1u << 24) && !done; ++k) {
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
                                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(smem_u32(&bar)) : "memory");
                    if (!done) __nanosleep(100);
                }
            }
            if (!__syncthreads_and((int)done)) {         // (also: set data and pieces visible)
                for (int i = threadIdx.x; i < (int)(2 * TOK * D * sizeof(T) / sizeof(uint32_t)); i += NT)
                    reinterpret_cast<uint32_t*>(sK)[i] = 0xFFFFFFFFu;
                if (threadIdx.x == 0 && stats) stats->status = KVM_E_DEVICE_TIMEOUT;
                __syncthreads();
            }
        }

        // ---- weights, one lane group per token
        if (!average) {
            const int w = threadIdx.x / LPR, lane = threadIdx.x % LPR;
            const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
#pragma unroll 2
            for (int j = w; j < ntok; j += NG) {
                if (s_len[j] == 1) continue;             // a set of one token is copied, its weight is never used
                const int p = s_piv[j];
                float kj[N], kp[N];
                const uint4* sK4 = reinterpret_cast<const uint4*>(sK) + lane;      // rows of LPR 16-byte pieces
                Vec<T>::unpack(sK4[j * LPR], kj);
                if (p >= tok0 && p < tile_end)
                    Vec<T>::unpack(sK4[(p - tok0) * LPR], kp);
                else
                    Vec<T>::unpack(ldg16(Ku + (size_t)p * D + lane * N), kp);
                float d2 = 0.f;
#pragma unroll
                for (int e = 0; e < N; ++e) { const float a = kp[e] - kj[e]; d2 = fmaf(a, a, d2); }
#pragma unroll
                for (int off = 1; off < LPR; off <<= 1) d2 += __shfl_xor_sync(gmask, d2, off);
                if (lane == 0) s_g[j] = exp2f(d2 * s_coef[j]);
            }
        } else {
            for (int j = threadIdx.x; j < ntok; j += NT) s_g[j] = 1.f;
        }
        __syncthreads();

        // ---- walk: a lane group as wide as a K row and a V row together (a warp at most; then K first, V second)
        // takes every NWK-th piece; a lane owns 16 bytes of a row
        constexpr int GL = (2 * LPR <= 32) ? 2 * LPR : 32;   // lanes per walking group
        constexpr int TPASS = 2 * LPR / GL;                  // tensors handled one after the other (1: side by side)
        constexpr int NWK = NT / GL;
        const int wk = threadIdx.x / GL, gl = threadIdx.x % GL;
        const int np = s_npiece;
#pragma unroll
        for (int tp = 0; tp < TPASS; ++tp) {
            const int which = (TPASS == 2) ? tp : gl / LPR;
            const int ch = (gl % LPR) * N;
            const uint4* sX4 = reinterpret_cast<const uint4*>(which ? sV : sK) + (gl % LPR);   // rows of LPR 16-byte pieces
            uint4* out4 = reinterpret_cast<uint4*>((which ? V_out : K_out) + (size_t)u * cap * D) + (gl % LPR);
            for (int k = wk; k < np; k += NWK) {
                const int a = s_pbeg[k], b = s_pbeg[k + 1], kind = s_pkind[k], row = s_prow[k];
                if (kind == PIECE_COPY) {
                    out4[row * LPR] = sX4[a * LPR];
                    if (out_size && gl == 0 && tp == 0) out_size[(size_t)u * cap + row] = 1;
                    continue;
                }
                float acc[N], gs = 0.f;
#pragma unroll
                for (int e = 0; e < N; ++e) acc[e] = 0.f;
                const uint4* px = sX4 + a * LPR;
                const float* pg = s_g + a;
#pragma unroll 4
                for (int n_left = b - a; n_left > 0; --n_left, px += LPR, ++pg) {
                    const float g = *pg;
                    float x[N];
                    Vec<T>::unpack(*px, x);
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[e] = fmaf(g, x[e], acc[e]);
                    gs += g;
                }
                if (kind == PIECE_WHOLE) {
                    const int n = s_pn[k];
                    const float mul = (which && scale_v) ? (float)n / gs : 1.f / gs;
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[e] *= mul;
                    out4[row * LPR] = Vec<T>::pack(acc);
                    if (out_size && gl == 0 && tp == 0) out_size[(size_t)u * cap + row] = n;
                } else {
                    const int slot = (kind == PIECE_TAIL) ? 1 : 0;
                    float* dst = slots.s(u, Tn, tile, slot) + which * D + ch;
#pragma unroll
                    for (int e = 0; e < N; e += 4)
                        *reinterpret_cast<float4*>(dst + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
                    if (gl == 0 && tp == 0) *slots.g(u, Tn, tile, slot) = gs;
                }
            }
        }
    }
}

// Sets that cross a tile boundary: the block of the LAST boundary a set crosses adds its slots in tile order.
template <typename T, int D, int TOK>
__global__ void __launch_bounds__(2 * D) merge_fixup_kernel(const int32_t* __restrict__ set_start,
                                                            const int32_t* __restrict__ set_id,
                                                            T* __restrict__ K_out, T* __restrict__ V_out,
                                                            int32_t* __restrict__ out_size, Slots<D> slots, int S,
                                                            int cap, int Tn, int scale_v) {
    // The sets were written before the tile kernel began (it triggers this launch only after it has waited for
    // them), so they can be looked up while that kernel's last blocks still run; they are read through L2.
    const int c = blockIdx.x + 1;                 // boundary between tiles c-1 and c
    const long long u = blockIdx.y;
    const int b = c * TOK;
    if (b >= S) return;
    const int32_t* sid_u = set_id + (size_t)u * S;
    const int sid = __ldcg(sid_u + b);
    if (__ldcg(sid_u + b - 1) != sid) return;     // no set crosses here
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const int beg = __ldcg(st + sid), end = __ldcg(st + sid + 1);
    if (end > b + TOK) return;                    // crosses a later boundary too: finished there
    const int c_first = beg / TOK;                // tile holding the set's first token (its tail slot)
    grid_dependency_wait();                       // the tile kernel's slots
    // (written while this block may already have been resident: read through L2)
    float acc = __ldcg(slots.s(u, Tn, c_first, 1) + threadIdx.x);
    float gs = __ldcg(slots.g(u, Tn, c_first, 1));
    for (int t = c_first + 1; t <= c; ++t) {
        acc += __ldcg(slots.s(u, Tn, t, 0) + threadIdx.x);
        gs += __ldcg(slots.g(u, Tn, t, 0));
    }
    const int which = threadIdx.x / D, ch = threadIdx.x % D;
    const int n = end - beg;
    T* out = which ? V_out : K_out;
    out[((size_t)u * cap + sid) * D + ch] = f32_to_elem<T>(which && scale_v ? acc * ((float)n / gs) : acc / gs);
    if (out_size && threadIdx.x == 0) out_size[(size_t)u * cap + sid] = n;
}

// Bandwidth per merging set (one non-circular reading of Eq. 4): 2 sigma_s^2 = mean over the set of
// |k_p - k_j|^2.  Sets can be hundreds of tokens long, so the work is split by tokens first:
// token_dist_kernel writes every token's squared distance to its set's pivot (one lane group per token), then
// set_coef_kernel sums them per set (one warp per set, lanes strided, fixed reduction order) and writes the factor
// that turns a squared distance into the exponent of 2: coef = -log2(e) / mean, or 0 (every weight 1) when the
// mean is 0.
template <typename T, int D>
__global__ void __launch_bounds__(256) token_dist_kernel(const T* __restrict__ K, const int32_t* __restrict__ set_id,
                                                         const int32_t* __restrict__ pivot, float* __restrict__ d2_out,
                                                         int S, int cap, long long n_rows) {
    constexpr int N = Vec<T>::N, LPR = D / N;
    grid_dependency_wait();
    const long long gid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    if (gid >= n_rows) return;                            // whole groups leave together
    const int lane = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << ((threadIdx.x % 32) / LPR * LPR));
    const long long u = gid / S;
    const int sid = __ldcg(set_id + gid);
    const int p = __ldcg(pivot + (size_t)u * cap + sid);
    float kj[N], kp[N];
    Vec<T>::unpack(ldg16(K + (size_t)gid * D + lane * N), kj);
    Vec<T>::unpack(ldg16(K + ((size_t)u * S + p) * D + lane * N), kp);
    float d2 = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) { const float a = kp[e] - kj[e]; d2 = fmaf(a, a, d2); }
#pragma unroll
    for (int off = 1; off < LPR; off <<= 1) d2 += __shfl_xor_sync(gmask, d2, off);
    if (lane == 0) d2_out[gid] = d2;
}

__global__ void __launch_bounds__(256) set_coef_kernel(const float* __restrict__ d2, const int32_t* __restrict__ set_start,
                                                       const int32_t* __restrict__ out_len, float* __restrict__ coef,
                                                       int S, int cap) {
    grid_dependency_wait();
    const long long u = blockIdx.y;
    const int s = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (s >= min(__ldcg(out_len + u), cap)) return;       // whole warps leave together
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const int lo = __ldcg(st + s), hi = __ldcg(st + s + 1);
    const float* du = d2 + (size_t)u * S;
    float tot = 0.f;
    for (int j = lo + lane; j < hi; j += 32) tot += __ldcg(du + j);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, off);
    if (lane == 0) coef[(size_t)u * cap + s] = tot > 0.f ? -LOG2E * (float)(hi - lo) / tot : 0.f;
}

// Output rows that are a single input state: row s = K[pivot[s]], V[pivot[s]] (V times the set size when
// asked and the sets are real ones).  One lane group per (row, tensor), 16-byte copies.
template <typename T, int D>
__global__ void __launch_bounds__(256) gather_rows_kernel(const T* __restrict__ K, const T* __restrict__ V,
                                                          const int32_t* __restrict__ set_start,
                                                          const int32_t* __restrict__ pivot,
                                                          const int32_t* __restrict__ out_len, T* __restrict__ K_out,
                                                          T* __restrict__ V_out, int32_t* __restrict__ out_size,
                                                          int S, int cap, int scale_v, int singletons) {
    constexpr int N = Vec<T>::N, LPR = D / N, ROWS = 256 / LPR / 2;
    grid_dependency_wait();     // sets and pivots come from the kernel before this one
    const long long u = blockIdx.y;
    const int g = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    const int s = blockIdx.x * ROWS + (g >> 1), which = g & 1;
    if (s >= min(__ldcg(out_len + u), cap)) return;
    const int p = __ldcg(pivot + (size_t)u * cap + s);
    const int32_t* st = set_start + (size_t)u * (cap + 1);
    const int n = singletons ? 1 : __ldcg(st + s + 1) - __ldcg(st + s);
    const T* src = (which ? V : K) + ((size_t)u * S + p) * D + lane * N;
    T* dst = (which ? V_out : K_out) + ((size_t)u * cap + s) * D + lane * N;
    uint4 r = ldg16(src);
    if (which && scale_v && n > 1) {
        float x[N];
        Vec<T>::unpack(r, x);
#pragma unroll
        for (int e = 0; e < N; ++e) x[e] *= (float)n;
        r = Vec<T>::pack(x);
    }
    *reinterpret_cast<uint4*>(dst) = r;
    if (out_size && which == 0 && lane == 0) out_size[(size_t)u * cap + s] = n;
}

template <typename T, int D>
cudaError_t launch_gather_t(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                            const int32_t* pivot, const int32_t* out_len, void* K_out, void* V_out,
                            int32_t* out_size, cudaStream_t st) {
    constexpr int ROWS = 256 / (D / Vec<T>::N) / 2;
    return launch_dependent(gather_rows_kernel<T, D>, dim3((d.cap + ROWS - 1) / ROWS, d.U), dim3(256), 0, st,
                            (const T*)K, (const T*)V, set_start, pivot, out_len, (T*)K_out, (T*)V_out, out_size, d.S,
                            d.cap, d.scale_v, d.set_rule == KVM_SETS_CONSERVED_ONLY ? 1 : 0);
}

template <typename T, int D, int TOK>
cudaError_t launch_t(const Dims& d, const void* K, const void* V, const int32_t* set_start, const int32_t* pivot,
                     const int32_t* set_id, const int32_t* out_len, void* K_out, void* V_out, int32_t* out_size,
                     float* scratch, float* set_coef, float* token_d2, kvm_stats* stats, cudaStream_t st) {
    const int Tn = (d.S + TOK - 1) / TOK;
    Slots<D> slots;
    slots.sums = scratch;
    slots.gsum = scratch + (size_t)d.U * Tn * 2 * (2 * D);
    const size_t smem = (size_t)2 * TOK * D * sizeof(T);       // 32 KB: below the default limit, no opt-in needed
    cudaError_t e = cudaSuccess;
    const float c = -LOG2E / (2.f * d.sigma * d.sigma);
    const bool per_set = d.weight_rule == KVM_WEIGHT_SET_SIGMA;
    if (per_set) {
        const long long rows = (long long)d.U * d.S;
        const unsigned blocks = (unsigned)((rows * (D / Vec<T>::N) + 255) / 256);
        e = launch_dependent(token_dist_kernel<T, D>, dim3(blocks), dim3(256), 0, st, (const T*)K, set_id, pivot,
                             token_d2, d.S, d.cap, rows);
        if (e != cudaSuccess) return e;
        e = launch_dependent(set_coef_kernel, dim3((d.cap + 7) / 8, d.U), dim3(256), 0, st, (const float*)token_d2,
                             set_start, out_len, set_coef, d.S, d.cap);
        if (e != cudaSuccess) return e;
    }
    e = launch_dependent(merge_tile_kernel<T, D, TOK>, dim3(Tn, d.U), dim3(2 * D), smem, st, (const T*)K,
                         (const T*)V, set_start, pivot, set_id, (T*)K_out, (T*)V_out, out_size, slots, d.S, d.cap, c,
                         d.scale_v, d.weight_rule == KVM_WEIGHT_AVERAGE ? 1 : 0,
                         per_set ? (const float*)set_coef : (const float*)nullptr, stats);
    if (e != cudaSuccess) return e;
    if (Tn > 1)
        e = launch_dependent(merge_fixup_kernel<T, D, TOK>, dim3(Tn - 1, d.U), dim3(2 * D), 0, st, set_start, set_id,
                             (T*)K_out, (T*)V_out, out_size, slots, d.S, d.cap, Tn, d.scale_v);
    return e;
}

}  // namespace

// Tokens per tile.
#ifndef KVM_MERGE_TOK_BF16
#define KVM_MERGE_TOK_BF16 64
#endif
static int merge_tile_tokens(const Dims& d) { return d.dtype == KVM_BF16 ? KVM_MERGE_TOK_BF16 : 32; }

size_t merge_scratch_floats(const Dims& d) {
    const int TOK = merge_tile_tokens(d);
    const size_t Tn = (d.S + TOK - 1) / TOK;
    return (size_t)d.U * Tn * 2 * (2 * d.D) + (size_t)d.U * Tn * 2;
}

cudaError_t launch_token_sets(const Dims& d, const int32_t* set_start, const int32_t* out_len, int32_t* set_id,
                              cudaStream_t st) {
    token_set_kernel<<<dim3((d.cap + 255) / 256, d.U), 256, 0, st>>>(set_start, out_len, set_id, d.S, d.cap);
    return cudaGetLastError();
}

cudaError_t launch_gather(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                          const int32_t* pivot, const int32_t* out_len, void* K_out, void* V_out, int32_t* out_size,
                          cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128
                   ? launch_gather_t<__nv_bfloat16, 128>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st)
                   : launch_gather_t<__nv_bfloat16, 64>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st);
    }
    return d.D == 128 ? launch_gather_t<float, 128>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st)
                      : launch_gather_t<float, 64>(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st);
}

// set_coef [U, cap] and token_d2 [U, S]: fp32 scratch, used only by the per-set bandwidth rule; out_len: device [U].
cudaError_t launch_merge(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                         const int32_t* pivot, const int32_t* set_id, const int32_t* out_len, void* K_out,
                         void* V_out, int32_t* out_size, float* scratch, float* set_coef, float* token_d2,
                         kvm_stats* stats, cudaStream_t st) {
    if (d.dtype == KVM_BF16) {
        return d.D == 128 ? launch_t<__nv_bfloat16, 128, KVM_MERGE_TOK_BF16>(d, K, V, set_start, pivot, set_id, out_len,
                                                                          K_out, V_out, out_size, scratch, set_coef, token_d2, stats, st)
                          : launch_t<__nv_bfloat16, 64, KVM_MERGE_TOK_BF16>(d, K, V, set_start, pivot, set_id, out_len,
                                                                         K_out, V_out, out_size, scratch, set_coef, token_d2, stats, st);
    }
    return d.D == 128 ? launch_t<float, 128, 32>(d, K, V, set_start, pivot, set_id, out_len, K_out, V_out, out_size,
                                                 scratch, set_coef, token_d2, stats, st)
                      : launch_t<float, 64, 32>(d, K, V, set_start, pivot, set_id, out_len, K_out, V_out, out_size,
                                                scratch, set_coef, token_d2, stats, st);
}

}  // namespace kvm
