// Merging-set identification and pivot choice for one unit per thread block
// (Algorithm 1 / Definition 4.1 with the conserved-token rule of Sections 4.1,
// 4.2 and 5.1; pivot of Eq. 6).  Inputs are the unit's aggregated scores and
// neighbour similarities (a few KB), so the whole step lives in one block:
//   1. radix-select the n_h largest scores outside the recent window;
//   2. boundary flags: hard (first token, conserved token or its right
//      neighbour) and soft (similarity not above epsilon);
//   3. budget rule: radix-select the soft cuts with the smallest similarity when
//      the sets would exceed the capacity;
//   4. inclusive scan of the flags -> set ids, set starts, set count;
//   5. segmented arg-max of the scores -> one pivot per set (or of the token
//      index / a caller-supplied key, for the variants of Sections 4.2 and 5.3).
// In eviction mode (Section 2.2) steps 2-5 are replaced by a compaction of the
// conserved tokens.  Under the anchor reading of the set identification (Section
// 3.2) steps 2-3 are replaced by a walk over per-token run lengths, done as
// pointer jumping in shared memory.
// Every tie is broken toward the lower token index, and every reduction has a
// fixed order, so the integer outputs are reproducible bit for bit.
#include <limits.h>

#include "common.cuh"

namespace kvm {
namespace {

constexpr int NT = 1024;
constexpr int NW = NT / 32;

enum : uint8_t { F_KEEP = 1, F_HARD = 2, F_SOFT = 4, F_CUT = 8, F_ANCHOR = 16 };

// Order-preserving map float -> uint32 (ascending).
__device__ __forceinline__ uint32_t order_key(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Shared {
    int hist[256];
    int warp_i[NW];
    float warp_a[NW];
    int warp_p[NW];
    int warp_f[NW];
    int bcast[4];
};

// Exclusive prefix sum of one int per thread; returns the block total through `total`.
__device__ __forceinline__ int block_exscan(int v, int& total, Shared& sh) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    __syncthreads();  // protect warp_i from a previous use
    if (lane == 31) sh.warp_i[w] = inc;
    __syncthreads();
    if (w == 0) {
        int x = sh.warp_i[lane], xi = x;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, xi, off);
            if (lane >= off) xi += t;
        }
        sh.warp_i[lane] = xi - x;  // exclusive warp offsets
        if (lane == 31) sh.bcast[0] = xi;
    }
    __syncthreads();
    total = sh.bcast[0];
    return sh.warp_i[w] + inc - v;
}

// Exclusive prefix maximum of one int per thread (identity -1).
__device__ __forceinline__ int block_exscan_max(int v, Shared& sh) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc = max(inc, t);
    }
    __syncthreads();  // protect warp_i from a previous use
    if (lane == 31) sh.warp_i[w] = inc;
    __syncthreads();
    if (w == 0) {
        int x = sh.warp_i[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x = max(x, t);
        }
        const int ex = __shfl_up_sync(0xffffffffu, x, 1);
        sh.warp_i[lane] = lane ? ex : -1;    // exclusive over warps
    }
    __syncthreads();
    const int prev = __shfl_up_sync(0xffffffffu, inc, 1);
    return max(sh.warp_i[w], lane ? prev : -1);
}

// Among the tokens j in [0, n) for which valid(j), find the k smallest keys (k >= 1,
// k <= number of valid tokens).  On return every valid token with key < cut is
// selected, and of those with key == cut the first `need` in index order are.
template <typename KeyFn, typename ValidFn>
__device__ __forceinline__ void radix_select(int n, int k, KeyFn key, ValidFn valid, uint32_t& cut, int& need,
                                             Shared& sh) {
    uint32_t prefix = 0, mask = 0;
    int k_rem = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        __syncthreads();
        if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += NT) {
            if (valid(j)) {
                const uint32_t kk = key(j);
                if ((kk & mask) == prefix) atomicAdd(&sh.hist[(kk >> shift) & 255u], 1);
            }
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns bins [8l, 8l+8): find the bin where the running count reaches k_rem
            int c[8], s = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) { c[t] = sh.hist[threadIdx.x * 8 + t]; s += c[t]; }
            int inc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, off);
                if ((int)threadIdx.x >= off) inc += t;
            }
            int below = inc - s;
            if (below < k_rem && k_rem <= inc) {
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (below < k_rem && k_rem <= below + c[t]) {
                        sh.bcast[1] = threadIdx.x * 8 + t;
                        sh.bcast[2] = below;
                    }
                    below += c[t];
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)sh.bcast[1] << shift;
        mask |= 255u << shift;
        k_rem -= sh.bcast[2];
    }
    cut = prefix;
    need = k_rem;
}

struct Best {
    float a;
    int i;
};
// Left operand covers lower indices; ties keep the left (lower index).
__device__ __forceinline__ Best better(Best l, Best r) { return (r.a > l.a) ? r : l; }

__global__ void __launch_bounds__(NT) segment_unit_kernel(const float* __restrict__ scores,
                                                          const float* __restrict__ sim, int32_t* __restrict__ set_id,
                                                          int32_t* __restrict__ set_start, int32_t* __restrict__ pivot,
                                                          int32_t* __restrict__ out_len, kvm_stats* stats, int S,
                                                          int cap, int n_r, int n_h, float eps, int enforce,
                                                          int pivot_rule, const float* __restrict__ pivot_key,
                                                          int set_rule) {
    extern __shared__ __align__(16) uint8_t flags[];  // [S] (+ jump arrays for the anchor reading)
    __shared__ Shared sh;
    // One block per unit leaves most SMs idle: let the merge kernel's blocks move in now and stage their K and V
    // tiles (inputs, never written) while this kernel runs; they wait for its results before reading any.
    grid_launch_dependents();
    grid_dependency_wait();     // scores and similarities come from the kernels before this one
    const int u = blockIdx.x;
    const float* a = scores + (size_t)u * S;
    const float* c = sim + (size_t)u * S;
    const int E = (S + NT - 1) / NT;               // tokens per thread, contiguous
    const int lo = min(S, (int)threadIdx.x * E), hi = min(S, lo + E);
    const int R = max(0, S - n_r);                 // first recent position
    const int nh = min(n_h, R);

    // ---- 1. conserved set: recent window + n_h largest scores (ties: lower index)
    uint32_t cut = 0;
    int need = 0;
    if (nh > 0) {
        radix_select(R, nh, [&](int j) { return ~order_key(a[j]); }, [&](int) { return true; }, cut, need, sh);
    }
    {
        int eq = 0;
        if (nh > 0)
            for (int j = lo; j < min(hi, R); ++j) eq += (~order_key(a[j]) == cut);
        int tot;
        int rank = block_exscan(eq, tot, sh);
        for (int j = lo; j < hi; ++j) {
            uint8_t f = 0;
            if (j >= R) f = F_KEEP;
            else if (nh > 0) {
                const uint32_t kk = ~order_key(a[j]);
                if (kk < cut) f = F_KEEP;
                else if (kk == cut) { if (rank < need) f = F_KEEP; ++rank; }
            }
            flags[j] = f;
        }
    }
    __syncthreads();

    int32_t* st = set_start + (size_t)u * (cap + 1);
    int32_t* pv = pivot + (size_t)u * cap;

    // ---- eviction (Section 2.2): the conserved tokens are the output, one state each
    if (set_rule == KVM_SETS_CONSERVED_ONLY) {
        int nk = 0;
        for (int j = lo; j < hi; ++j) nk += (flags[j] & F_KEEP) ? 1 : 0;
        int n_keep;
        int id = block_exscan(nk, n_keep, sh);
        for (int j = lo; j < hi; ++j) {
            const bool k = (flags[j] & F_KEEP) != 0;
            if (k && id < cap) { st[id] = j; pv[id] = j; }
            if (set_id) set_id[(size_t)u * S + j] = k ? id : -1;
            id += k;
        }
        if (threadIdx.x == 0) {
            if (n_keep <= cap) st[n_keep] = S;
            out_len[u] = n_keep;
            if (stats) {
                atomicMax(&stats->max_out_len, n_keep);
                int old = stats->min_out_len;      // 0 means "unset"
                while (old == 0 || n_keep < old) {
                    const int prev = atomicCAS(&stats->min_out_len, old, n_keep);
                    if (prev == old) break;
                    old = prev;
                }
                atomicAdd((unsigned long long*)&stats->sum_out_len, (unsigned long long)n_keep);
            }
        }
        return;
    }

    bool fire = false;
    int tot_near = 0;
    if (set_rule == KVM_SETS_ANCHOR) {
        // ---- anchor reading (Section 3.2): token i, when it ends a group, takes with it the eff(i) tokens
        // before it: its run length (c[] holds it) cut short by the nearest conserved token; conserved
        // tokens take none.  The groups are the chain S-1 -> next(S-1) -> ... with next(i) = i - eff(i) - 1,
        // found by pointer jumping: after round k every chain node within 2^k - 1 steps of S-1 is marked.
        uint16_t* JA = reinterpret_cast<uint16_t*>(flags + ((S + 15) & ~15));     // next(i) + 1; 0 = chain ends
        uint16_t* JB = JA + S;
        int last_keep = -1;
        for (int j = lo; j < hi; ++j) if (flags[j] & F_KEEP) last_keep = j;
        int pk = block_exscan_max(last_keep, sh);            // nearest conserved token before this range
        for (int j = lo; j < hi; ++j) {
            const bool kept = (flags[j] & F_KEEP) != 0;
            const int eff = kept ? 0 : min((int)c[j], j - 1 - pk);
            JA[j] = (uint16_t)(j - eff);                      // next + 1 = j - eff - 1 + 1
            if (kept) pk = j;
        }
        if (threadIdx.x == 0) flags[S - 1] |= F_ANCHOR;
        __syncthreads();
        unsigned* fw = reinterpret_cast<unsigned*>(flags);
        for (int span = 1; span < S; span <<= 1) {
            for (int j = lo; j < hi; ++j) {
                const int nx = JA[j];
                if ((flags[j] & F_ANCHOR) && nx) atomicOr(&fw[(nx - 1) >> 2], (unsigned)F_ANCHOR << (8 * ((nx - 1) & 3)));
                JB[j] = nx ? JA[nx - 1] : (uint16_t)0;
            }
            __syncthreads();
            uint16_t* t = JA; JA = JB; JB = t;
        }
        for (int j = lo; j < hi; ++j)
            if (j == 0 || (flags[j - 1] & F_ANCHOR)) flags[j] |= F_CUT;   // own byte: neighbours read bit F_ANCHOR only
    } else {
    // ---- 2. boundary flags
    int n_hard = 0, n_soft = 0, n_near = 0;
    for (int j = lo; j < hi; ++j) {
        uint8_t f = flags[j];
        const bool hard = (j == 0) || (f & F_KEEP) || (flags[j - 1] & F_KEEP);
        const float cj = c[j];
        if (j > 0 && fabsf(cj - eps) < 1e-3f) ++n_near;
        if (hard) { f |= F_HARD | F_CUT; ++n_hard; }
        else if (!(cj > eps)) { f |= F_SOFT | F_CUT; ++n_soft; }
        flags[j] = f;    // only bits other than F_KEEP change, so neighbours reading F_KEEP are safe
    }
    int tot_hard, tot_soft;
    block_exscan(n_hard, tot_hard, sh);
    block_exscan(n_soft, tot_soft, sh);
    block_exscan(n_near, tot_near, sh);

    // ---- 3. budget rule: keep only the (cap - hard) soft cuts with the smallest similarity
    fire = enforce && (tot_hard + tot_soft > cap);
    if (fire) {
        const int m = max(0, cap - tot_hard);
        uint32_t cut2 = 0;
        int need2 = 0;
        if (m > 0)
            radix_select(S, m, [&](int j) { return order_key(c[j]); }, [&](int j) { return (flags[j] & F_SOFT) != 0; },
                         cut2, need2, sh);
        int eq = 0;
        if (m > 0)
            for (int j = lo; j < hi; ++j) eq += ((flags[j] & F_SOFT) && order_key(c[j]) == cut2);
        int tot;
        int rank = block_exscan(eq, tot, sh);
        for (int j = lo; j < hi; ++j) {
            const uint8_t f = flags[j];
            if (f & F_SOFT) {
                bool stay = false;
                if (m > 0) {
                    const uint32_t kk = order_key(c[j]);
                    if (kk < cut2) stay = true;
                    else if (kk == cut2) { stay = rank < need2; ++rank; }
                }
                if (!stay) flags[j] = f & ~F_CUT;
            }
        }
    }
    }   // neighbour reading
    __syncthreads();

    // ---- 4. scan of the cut flags -> set ids and starts
    int ncut = 0;
    for (int j = lo; j < hi; ++j) ncut += (flags[j] & F_CUT) ? 1 : 0;
    int n_sets;
    const int before = block_exscan(ncut, n_sets, sh);
    {
        int id = before - 1;
        for (int j = lo; j < hi; ++j) {
            if (flags[j] & F_CUT) {
                ++id;
                if (id <= cap) st[id] = j;
            }
            if (set_id) set_id[(size_t)u * S + j] = id;
        }
    }
    if (threadIdx.x == 0) {
        if (n_sets <= cap) st[n_sets] = S;
        out_len[u] = n_sets;
        if (stats) {
            if (fire) atomicAdd(&stats->units_budget_rule, 1);
            if (tot_near) atomicAdd(&stats->near_threshold, tot_near);
            atomicMax(&stats->max_out_len, n_sets);
            int old = stats->min_out_len;      // 0 means "unset"
            while (old == 0 || n_sets < old) {
                const int prev = atomicCAS(&stats->min_out_len, old, n_sets);
                if (prev == old) break;
                old = prev;
            }
            atomicAdd((unsigned long long*)&stats->sum_out_len, (unsigned long long)n_sets);
        }
    }

    // ---- 5. segmented arg-max: pivot of each set (ties: lowest index).  The key is the score (Eq. 6),
    // the token index (last-index pivot of the average-weighted baseline) or the caller's key array.
    const float* pk = pivot_key ? pivot_key + (size_t)u * S : a;
    auto key_of = [&](int j) -> float {
        return pivot_rule == KVM_PIVOT_LAST ? (float)j : (pivot_rule == KVM_PIVOT_KEY ? pk[j] : a[j]);
    };
    // Per thread: `head` = best of the tokens before the first cut in its range
    // (they belong to a set that started earlier), `run` = best since its last cut.
    Best head = {-INFINITY, INT_MAX}, run = {-INFINITY, INT_MAX};
    bool seen_cut = false;
    int id = before - 1;          // set of the token before `lo`
    int first_cut_id = -1;        // id of the set that starts at this thread's first cut
    for (int j = lo; j < hi; ++j) {
        if (flags[j] & F_CUT) {
            if (seen_cut) { if (id < cap) pv[id] = run.i; }       // a set fully inside this range
            else { head = run; first_cut_id = id + 1; }
            seen_cut = true;
            ++id;
            run = {-INFINITY, INT_MAX};
        }
        run = better(run, Best{key_of(j), j});
    }
    if (!seen_cut) head = run;
    // Exclusive segmented scan over threads of (value = tail or whole range, flag = seen_cut).
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    Best x = run;                 // tail if seen_cut, else the whole range (== head)
    int xf = seen_cut ? 1 : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float la = __shfl_up_sync(0xffffffffu, x.a, off);
        const int li = __shfl_up_sync(0xffffffffu, x.i, off);
        const int lf = __shfl_up_sync(0xffffffffu, xf, off);
        if (lane >= off && !xf) { x = better(Best{la, li}, x); xf = lf; }
    }
    __syncthreads();
    if (lane == 31) { sh.warp_a[w] = x.a; sh.warp_p[w] = x.i; sh.warp_f[w] = xf; }
    __syncthreads();
    if (w == 0) {
        Best y = {sh.warp_a[lane], sh.warp_p[lane]};
        int yf = sh.warp_f[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float la = __shfl_up_sync(0xffffffffu, y.a, off);
            const int li = __shfl_up_sync(0xffffffffu, y.i, off);
            const int lf = __shfl_up_sync(0xffffffffu, yf, off);
            if (lane >= off && !yf) { y = better(Best{la, li}, y); yf = lf; }
        }
        // exclusive: shift by one warp
        const float ea = __shfl_up_sync(0xffffffffu, y.a, 1);
        const int ei = __shfl_up_sync(0xffffffffu, y.i, 1);
        sh.warp_a[lane] = lane ? ea : -INFINITY;
        sh.warp_p[lane] = lane ? ei : INT_MAX;
    }
    __syncthreads();
    // carry into this thread = (carry into its warp) (+) (inclusive value of the previous lane)
    const float pa = __shfl_up_sync(0xffffffffu, x.a, 1);
    const int pi = __shfl_up_sync(0xffffffffu, x.i, 1);
    const int pf = __shfl_up_sync(0xffffffffu, xf, 1);
    Best carry = {sh.warp_a[w], sh.warp_p[w]};
    if (lane > 0) carry = pf ? Best{pa, pi} : better(carry, Best{pa, pi});
    // The set that was open when this thread's range began ends at its first cut
    // (or at the end of the sequence, for the thread holding the last token).
    if (lo < hi) {
        if (seen_cut) {
            const int ended = first_cut_id - 1;
            if (ended >= 0 && ended < cap) pv[ended] = better(carry, head).i;
            if (hi == S && id < cap) pv[id] = run.i;
        } else if (hi == S) {
            if (id >= 0 && id < cap) pv[id] = better(carry, head).i;
        }
    }
}

// Sets formed by Algorithm 1 alone (nothing conserved, no budget) over the sequence length:
// 1 + #{j >= 1 : not (sim_j > eps)}, divided by S.  One block per unit.
__global__ void __launch_bounds__(256) set_ratio_kernel(const float* __restrict__ sim, float* __restrict__ ratio,
                                                        int S, float eps) {
    __shared__ int part[8];
    const float* c = sim + (size_t)blockIdx.x * S;
    int n = 0;
    for (int j = 1 + threadIdx.x; j < S; j += 256) n += !(c[j] > eps);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) n += __shfl_xor_sync(0xffffffffu, n, off);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 1;
        for (int w = 0; w < 8; ++w) t += part[w];
        ratio[blockIdx.x] = (float)t / (float)S;
    }
}

}  // namespace

// Largest dynamic shared memory the segment kernel is ever launched with: the anchor reading at KVM_ANCHOR_MAX_SEQ.
size_t segment_max_smem() {
    const size_t a = (size_t)KVM_MAX_SEQ, b = (size_t)5 * KVM_ANCHOR_MAX_SEQ + 16;
    return a > b ? a : b;
}

cudaError_t launch_set_ratio(const Dims& d, const float* sim, float* ratio, cudaStream_t st) {
    set_ratio_kernel<<<d.U, 256, 0, st>>>(sim, ratio, d.S, d.eps);
    return cudaGetLastError();
}

cudaError_t launch_segment(const Dims& d, const float* scores, const float* sim, int32_t* set_id,
                           int32_t* set_start, int32_t* pivot, int32_t* out_len, kvm_stats* stats, cudaStream_t st) {
    // flags [S] bytes; the anchor reading adds two uint16 jump arrays
    const size_t smem = d.set_rule == KVM_SETS_ANCHOR ? (size_t)((d.S + 15) & ~15) + 4 * (size_t)d.S : (size_t)d.S;
    if (smem > 40 * 1024) {   // more dynamic shared memory than the default limit: opt in (cheap, idempotent)
        cudaError_t e = cudaFuncSetAttribute(segment_unit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)segment_max_smem());
        if (e != cudaSuccess) return e;
    }
    return launch_dependent(segment_unit_kernel, dim3(d.U), dim3(NT), smem, st, scores, sim, set_id, set_start, pivot,
                            out_len, stats, d.S, d.cap, d.n_r, d.n_h, d.eps, d.enforce, d.pivot_rule,
                            d.pivot_rule == KVM_PIVOT_KEY ? d.pivot_key : (const float*)nullptr, d.set_rule);
}

}  // namespace kvm
