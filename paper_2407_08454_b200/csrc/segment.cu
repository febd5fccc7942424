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
// Two kernels compute the same thing: segment_unit_kernel for every shape and
// rule (tokens re-read per phase, flags in shared memory, 8-bit radix digits),
// and segment_unit_reg_kernel for the neighbour reading with at most four
// tokens per thread (S <= 4096), which keeps a thread's tokens in registers.
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
    int hist[3][256];       // radix-select histograms, used in rotation (one block barrier per digit)
    int warp_i[2][NW];      // per-warp totals of the block scans, two buffers used alternately
    float warp_a[NW];
    int warp_p[NW];
    int warp_f[NW];
    int tot[4];             // block-wide counters (hard cuts, soft cuts, near-threshold pairs)
};

// Block scans with ONE barrier each: every warp leaves its total in shared memory, and after the barrier every
// warp scans the 32 totals for itself.  Consecutive scans must alternate `buf`: a warp can only reach the scan
// after next (same buffer) once all warps have passed the barrier in between, i.e. finished reading this one.

// Exclusive prefix sum of one int per thread; returns the block total through `total`.
__device__ __forceinline__ int block_exscan(int v, int& total, Shared& sh, int buf) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    if (lane == 31) sh.warp_i[buf][w] = inc;
    __syncthreads();
    const int x = sh.warp_i[buf][lane];
    int xi = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, xi, off);
        if (lane >= off) xi += t;
    }
    total = __shfl_sync(0xffffffffu, xi, 31);
    return __shfl_sync(0xffffffffu, xi - x, w) + inc - v;
}

// Exclusive prefix maximum of one int per thread (identity -1).
__device__ __forceinline__ int block_exscan_max(int v, Shared& sh, int buf) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc = max(inc, t);
    }
    if (lane == 31) sh.warp_i[buf][w] = inc;
    __syncthreads();
    int x = sh.warp_i[buf][lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, x, off);
        if (lane >= off) x = max(x, t);
    }
    const int before_warp = __shfl_sync(0xffffffffu, x, (w + 31) & 31);   // inclusive maximum over warps 0..w-1
    const int prev = __shfl_up_sync(0xffffffffu, inc, 1);
    return max(w ? before_warp : -1, lane ? prev : -1);
}

// Among the tokens j in [lo, hi) of every thread for which valid(j), find the k smallest keys (k >= 1,
// k <= number of valid tokens).  On return every valid token with key < cut is selected, and of the `n_eq`
// tokens with key == cut the first `need` in index order are.
// Four 8-bit digits, most significant first.  A digit costs one block barrier: the histograms rotate through
// three buffers (digit p counts into buffer p mod 3 and clears the one digit p + 2 will use, which nobody has
// read since the barrier before), and every warp finds the digit's bin for itself from the finished histogram
// instead of waiting for one warp to publish it.
template <typename KeyFn, typename ValidFn>
__device__ __forceinline__ void radix_select(int lo, int hi, int k, KeyFn key, ValidFn valid, uint32_t& cut,
                                             int& need, int& n_eq, Shared& sh) {
    const int lane = threadIdx.x & 31;
    if (threadIdx.x < 512) sh.hist[threadIdx.x >> 8][threadIdx.x & 255] = 0;
    __syncthreads();
    uint32_t prefix = 0, mask = 0;
    int k_rem = k, cnt = 0;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const int shift = 24 - 8 * p;
        int* H = sh.hist[p % 3];
        // a thread's tokens are neighbours and often share a bin: count runs, one atomic per run
        int run_bin = -1, run_n = 0;
        for (int j = lo; j < hi; ++j) {
            if (!valid(j)) continue;
            const uint32_t kk = key(j);
            if ((kk & mask) != prefix) continue;
            const int bin = (int)((kk >> shift) & 255u);
            if (bin != run_bin) {
                if (run_n) atomicAdd(&H[run_bin], run_n);
                run_bin = bin;
                run_n = 0;
            }
            ++run_n;
        }
        if (run_n) atomicAdd(&H[run_bin], run_n);
        __syncthreads();
        // lane l owns bins [8l, 8l+8): find the bin where the running count reaches k_rem
        const int4 c0 = reinterpret_cast<const int4*>(H)[lane * 2], c1 = reinterpret_cast<const int4*>(H)[lane * 2 + 1];
        const int c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        int s = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) s += c[t];
        int inc = s;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        int below = inc - s, bin = 0, bin_below = 0, bin_cnt = 0;
        const bool mine = below < k_rem && k_rem <= inc;       // true in exactly one lane
        if (mine) {
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (below < k_rem && k_rem <= below + c[t]) { bin = lane * 8 + t; bin_below = below; bin_cnt = c[t]; }
                below += c[t];
            }
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
        bin = __shfl_sync(0xffffffffu, bin, src);
        bin_below = __shfl_sync(0xffffffffu, bin_below, src);
        cnt = __shfl_sync(0xffffffffu, bin_cnt, src);
        prefix |= (uint32_t)bin << shift;
        mask |= 255u << shift;
        k_rem -= bin_below;
        if (p < 2 && threadIdx.x < 256) sh.hist[(p + 2) % 3][threadIdx.x] = 0;
    }
    cut = prefix;
    need = k_rem;
    n_eq = cnt;
}

struct Best {
    float a;
    int i;
};
// Left operand covers lower indices; ties keep the left (lower index).
__device__ __forceinline__ Best better(Best l, Best r) { return (r.a > l.a) ? r : l; }

__device__ __forceinline__ void record_out_len(kvm_stats* stats, int n) {
    atomicMax(&stats->max_out_len, n);
    int old = stats->min_out_len;      // 0 means "unset"
    while (old == 0 || n < old) {
        const int prev = atomicCAS(&stats->min_out_len, old, n);
        if (prev == old) break;
        old = prev;
    }
    atomicAdd((unsigned long long*)&stats->sum_out_len, (unsigned long long)n);
}

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

    if (threadIdx.x < 4) sh.tot[threadIdx.x] = 0;   // (the barriers of step 1 come before their first use)

    // ---- 1. conserved set: recent window + n_h largest scores (ties: lower index)
    uint32_t cut = 0;
    int need = 0, n_eq = 0;
    if (nh > 0) {
        radix_select(lo, min(hi, R), nh, [&](int j) { return ~order_key(a[j]); }, [&](int) { return true; }, cut,
                     need, n_eq, sh);
    }
    {
        // Tokens whose key equals the cut are taken in index order until `need` are; when all of them are
        // needed (no tie at the cut: the usual case) their ranks do not matter and the scan is skipped.
        int rank = 0;
        if (nh > 0 && need < n_eq) {
            int eq = 0;
            for (int j = lo; j < min(hi, R); ++j) eq += (~order_key(a[j]) == cut);
            int tot;
            rank = block_exscan(eq, tot, sh, 0);
        }
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
        int id = block_exscan(nk, n_keep, sh, 1);
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
                record_out_len(stats, n_keep);
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
        int pk = block_exscan_max(last_keep, sh, 1);            // nearest conserved token before this range
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
    // block totals: warp sums, one shared-memory atomic per warp and counter (integers: any order gives the same sum)
    n_hard = __reduce_add_sync(0xffffffffu, n_hard);
    n_soft = __reduce_add_sync(0xffffffffu, n_soft);
    n_near = __reduce_add_sync(0xffffffffu, n_near);
    if ((threadIdx.x & 31) == 0) {
        if (n_hard) atomicAdd(&sh.tot[0], n_hard);
        if (n_soft) atomicAdd(&sh.tot[1], n_soft);
        if (n_near) atomicAdd(&sh.tot[2], n_near);
    }
    __syncthreads();
    const int tot_hard = sh.tot[0], tot_soft = sh.tot[1];
    tot_near = sh.tot[2];

    // ---- 3. budget rule: keep only the (cap - hard) soft cuts with the smallest similarity
    fire = enforce && (tot_hard + tot_soft > cap);
    if (fire) {
        const int m = max(0, cap - tot_hard);
        uint32_t cut2 = 0;
        int need2 = 0, n_eq2 = 0;
        if (m > 0)
            radix_select(lo, hi, m, [&](int j) { return order_key(c[j]); },
                         [&](int j) { return (flags[j] & F_SOFT) != 0; }, cut2, need2, n_eq2, sh);
        int rank = 0;
        if (m > 0 && need2 < n_eq2) {
            int eq = 0;
            for (int j = lo; j < hi; ++j) eq += ((flags[j] & F_SOFT) && order_key(c[j]) == cut2);
            int tot;
            rank = block_exscan(eq, tot, sh, 1);
        }
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
    // (no barrier: from here on a thread reads only the flags of its own tokens, which it wrote itself)

    // ---- 4. scan of the cut flags -> set ids and starts
    int ncut = 0;
    for (int j = lo; j < hi; ++j) ncut += (flags[j] & F_CUT) ? 1 : 0;
    int n_sets;
    const int before = block_exscan(ncut, n_sets, sh, 0);
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
            record_out_len(stats, n_sets);
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
    if (lane == 31) { sh.warp_a[w] = x.a; sh.warp_p[w] = x.i; sh.warp_f[w] = xf; }
    __syncthreads();
    // every warp scans the 32 warp aggregates for itself; the carry into warp w is the inclusive value of warp w-1
    Best y = {sh.warp_a[lane], sh.warp_p[lane]};
    int yf = sh.warp_f[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float la = __shfl_up_sync(0xffffffffu, y.a, off);
        const int li = __shfl_up_sync(0xffffffffu, y.i, off);
        const int lf = __shfl_up_sync(0xffffffffu, yf, off);
        if (lane >= off && !yf) { y = better(Best{la, li}, y); yf = lf; }
    }
    const float wa = __shfl_sync(0xffffffffu, y.a, (w + 31) & 31);
    const int wi = __shfl_sync(0xffffffffu, y.i, (w + 31) & 31);
    // carry into this thread = (carry into its warp) (+) (inclusive value of the previous lane)
    const float pa = __shfl_up_sync(0xffffffffu, x.a, 1);
    const int pi = __shfl_up_sync(0xffffffffu, x.i, 1);
    const int pf = __shfl_up_sync(0xffffffffu, xf, 1);
    Best carry = w ? Best{wa, wi} : Best{-INFINITY, INT_MAX};
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

// ---------------------------------------------------------------------------------------------------------
// The same step for the neighbour reading when a thread's share is at most EM tokens (S <= EM * 1024): scores,
// similarities, keys and flags stay in registers, every token loop is unrolled, and neighbouring threads
// exchange the one bit they need by shuffle.  With 32 warps on one SM the kernel is bound by instruction issue,
// so what counts is instructions per token; results are identical to segment_unit_kernel's.
struct SharedReg {
    int hist[3][2048];      // one histogram per digit of the radix select
    int warp_i[2][NW];      // per-warp totals of the block scans, two buffers used alternately
    float warp_a[NW];
    int warp_p[NW];
    int warp_f[NW];
    int tot[4];             // block-wide counters (hard cuts, soft cuts, near-threshold pairs)
    int found[3][4];        // per digit: bin, keys below it, keys in it
};

// Exclusive prefix sum of one int per thread with one barrier (see block_exscan above for the two buffers).
__device__ __forceinline__ int block_exscan(int v, int& total, SharedReg& sh, int buf) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    if (lane == 31) sh.warp_i[buf][w] = inc;
    __syncthreads();
    const int x = sh.warp_i[buf][lane];
    int xi = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, xi, off);
        if (lane >= off) xi += t;
    }
    total = __shfl_sync(0xffffffffu, xi, 31);
    return __shfl_sync(0xffffffffu, xi - x, w) + inc - v;
}

// The k smallest of the keys marked in `valid` (bit t = key[t]); results as radix_select's.  Three digits of
// 11, 11 and 10 bits: the block's 1024 threads own two bins each, a block scan over the bin counts finds the
// digit, and the one thread whose bins hold the k-th key publishes it.  (Eight-bit digits with every warp
// scanning 256 bins for itself cost more instructions in total, and instruction issue is what bounds this kernel.)
template <int EM>
__device__ __forceinline__ void radix_select_reg(const uint32_t (&key)[EM], unsigned valid, int k, uint32_t& cut,
                                                 int& need, int& n_eq, SharedReg& sh) {
    static_assert(NT == 1024, "two bins per thread");
    {
        int* h = &sh.hist[0][0];
#pragma unroll
        for (int i = 0; i < 6; ++i) h[i * NT + threadIdx.x] = 0;
    }
    __syncthreads();
    uint32_t prefix = 0, mask = 0;
    int k_rem = k, cnt = 0;
#pragma unroll
    for (int p = 0; p < 3; ++p) {
        const int shift = p == 0 ? 21 : (p == 1 ? 10 : 0);
        const uint32_t dmask = p == 2 ? 1023u : 2047u;
        int* H = sh.hist[p];
        if (p == 0) {
            // the leading digit of neighbouring tokens is often the same: one atomic per run
            int run_bin = -1, run_n = 0;
#pragma unroll
            for (int t = 0; t < EM; ++t) {
                if (!((valid >> t) & 1u)) continue;
                const int bin = (int)(key[t] >> 21);
                if (bin != run_bin) {
                    if (run_n) atomicAdd(&H[run_bin], run_n);
                    run_bin = bin;
                    run_n = 0;
                }
                ++run_n;
            }
            if (run_n) atomicAdd(&H[run_bin], run_n);
        } else {
#pragma unroll
            for (int t = 0; t < EM; ++t)
                if (((valid >> t) & 1u) && (key[t] & mask) == prefix) atomicAdd(&H[(key[t] >> shift) & dmask], 1);
        }
        __syncthreads();
        const int2 h = reinterpret_cast<const int2*>(H)[threadIdx.x];     // bins 2t, 2t+1
        const int s = h.x + h.y;
        int tot;
        const int below = block_exscan(s, tot, sh, p & 1);
        if (below < k_rem && k_rem <= below + s) {                        // true in exactly one thread
            const bool first = k_rem <= below + h.x;
            sh.found[p][0] = 2 * (int)threadIdx.x + (first ? 0 : 1);
            sh.found[p][1] = first ? below : below + h.x;
            sh.found[p][2] = first ? h.x : h.y;
        }
        __syncthreads();
        prefix |= (uint32_t)sh.found[p][0] << shift;
        mask |= dmask << shift;
        k_rem -= sh.found[p][1];
        cnt = sh.found[p][2];
    }
    cut = prefix;
    need = k_rem;
    n_eq = cnt;
}

template <int EM>
__global__ void __launch_bounds__(NT) segment_unit_reg_kernel(const float* __restrict__ scores,
                                                              const float* __restrict__ sim,
                                                              int32_t* __restrict__ set_id,
                                                              int32_t* __restrict__ set_start,
                                                              int32_t* __restrict__ pivot, int32_t* __restrict__ out_len,
                                                              kvm_stats* stats, int S, int cap, int n_r, int n_h,
                                                              float eps, int enforce, int pivot_rule,
                                                              const float* __restrict__ pivot_key) {
    __shared__ SharedReg sh;
    grid_launch_dependents();   // (as in segment_unit_kernel)
    grid_dependency_wait();
    const int u = blockIdx.x;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int E = (S + NT - 1) / NT;               // tokens per thread, contiguous; E <= EM
    const int lo = min(S, (int)threadIdx.x * E);
    const int n = min(E, S - lo);                  // this thread's tokens: lo .. lo+n-1
    const int R = max(0, S - n_r);                 // first recent position
    const int nh = min(n_h, R);
    if (threadIdx.x < 4) sh.tot[threadIdx.x] = 0;  // (barriers of step 1 come before their first use)

    float a[EM], c[EM];
    uint32_t ka[EM];
    const size_t g0 = (size_t)u * S + lo;          // this thread's first token in the [U, S] arrays
    const bool vec = EM == 4 && n == 4 && (g0 & 3) == 0;   // four tokens on a 16-byte boundary: one access per array
    if (vec) {
        const float4 av = *reinterpret_cast<const float4*>(scores + g0), cv = *reinterpret_cast<const float4*>(sim + g0);
        a[0] = av.x; a[1] = av.y; a[2] = av.z; a[3] = av.w;
        c[0] = cv.x; c[1] = cv.y; c[2] = cv.z; c[3] = cv.w;
    } else {
#pragma unroll
        for (int t = 0; t < EM; ++t) {
            a[t] = (t < n) ? scores[g0 + t] : 0.f;
            c[t] = (t < n) ? sim[g0 + t] : 0.f;
        }
    }
#pragma unroll
    for (int t = 0; t < EM; ++t) ka[t] = ~order_key(a[t]);
    const unsigned own = (1u << n) - 1u;                                      // bit t: token lo+t exists
    const unsigned old_m = own & ((1u << max(0, min(n, R - lo))) - 1u);        // ... and lies before the recent window

    // ---- 1. conserved set: recent window + n_h largest scores (ties: lower index)
    uint32_t cut = 0;
    int need = 0, n_eq = 0;
    if (nh > 0) radix_select_reg<EM>(ka, old_m, nh, cut, need, n_eq, sh);
    unsigned keep = own & ~old_m;                                             // the recent window
    if (nh > 0) {
        int rank = 0;
        if (need < n_eq) {        // a tie at the cut: the first `need` of the equal keys in index order
            int eq = 0;
#pragma unroll
            for (int t = 0; t < EM; ++t) eq += (((old_m >> t) & 1u) && ka[t] == cut);
            int tot;
            rank = block_exscan(eq, tot, sh, 0);
        } else {
            rank = INT_MIN;       // every equal key is taken
        }
#pragma unroll
        for (int t = 0; t < EM; ++t) {
            if (!((old_m >> t) & 1u)) continue;
            if (ka[t] < cut) keep |= 1u << t;
            else if (ka[t] == cut) { if (rank < need) keep |= 1u << t; ++rank; }
        }
    }
    // the token before this thread's first: the last token of the thread before (which has all E of its tokens)
    const unsigned last_keep = (keep >> (E - 1)) & 1u;
    if (lane == 31) sh.warp_f[w] = (int)last_keep;
    __syncthreads();
    unsigned prev_keep = __shfl_up_sync(0xffffffffu, last_keep, 1);
    if (lane == 0) prev_keep = w ? (unsigned)sh.warp_f[w - 1] : 0u;

    // ---- 2. boundary flags
    unsigned hardm = 0, softm = 0;
    int n_near = 0;
#pragma unroll
    for (int t = 0; t < EM; ++t) {
        if (!((own >> t) & 1u)) continue;
        const int j = lo + t;
        const unsigned before = t ? (keep >> (t - 1)) & 1u : prev_keep;
        const bool hard = (j == 0) || ((keep >> t) & 1u) || before;
        if (j > 0 && fabsf(c[t] - eps) < 1e-3f) ++n_near;
        if (hard) hardm |= 1u << t;
        else if (!(c[t] > eps)) softm |= 1u << t;
    }
    {
        const int wh = __reduce_add_sync(0xffffffffu, __popc(hardm));
        const int ws = __reduce_add_sync(0xffffffffu, __popc(softm));
        const int wn = __reduce_add_sync(0xffffffffu, n_near);
        if (lane == 0) {
            if (wh) atomicAdd(&sh.tot[0], wh);
            if (ws) atomicAdd(&sh.tot[1], ws);
            if (wn) atomicAdd(&sh.tot[2], wn);
        }
    }
    __syncthreads();
    const int tot_hard = sh.tot[0], tot_soft = sh.tot[1], tot_near = sh.tot[2];

    // ---- 3. budget rule: keep only the (cap - hard) soft cuts with the smallest similarity
    const bool fire = enforce && (tot_hard + tot_soft > cap);
    unsigned cutm = hardm | softm;
    if (fire) {
        const int m = max(0, cap - tot_hard);
        unsigned stay = 0;
        if (m > 0) {
            uint32_t kc[EM];
#pragma unroll
            for (int t = 0; t < EM; ++t) kc[t] = order_key(c[t]);
            uint32_t cut2 = 0;
            int need2 = 0, n_eq2 = 0;
            radix_select_reg<EM>(kc, softm, m, cut2, need2, n_eq2, sh);
            int rank = INT_MIN;
            if (need2 < n_eq2) {
                int eq = 0;
#pragma unroll
                for (int t = 0; t < EM; ++t) eq += (((softm >> t) & 1u) && kc[t] == cut2);
                int tot;
                rank = block_exscan(eq, tot, sh, 1);
            }
#pragma unroll
            for (int t = 0; t < EM; ++t) {
                if (!((softm >> t) & 1u)) continue;
                if (kc[t] < cut2) stay |= 1u << t;
                else if (kc[t] == cut2) { if (rank < need2) stay |= 1u << t; ++rank; }
            }
        }
        cutm = hardm | stay;
    }

    // ---- 4. scan of the cut flags -> set ids and starts
    int32_t* st = set_start + (size_t)u * (cap + 1);
    int32_t* pv = pivot + (size_t)u * cap;
    int n_sets;
    const int before = block_exscan(__popc(cutm), n_sets, sh, 0);
    {
        int id = before - 1, ids[EM];
#pragma unroll
        for (int t = 0; t < EM; ++t) {
            if (((own & cutm) >> t) & 1u) {
                ++id;
                if (id <= cap) st[id] = lo + t;
            }
            ids[t] = id;
        }
        if (set_id) {
            if (vec) {
                *reinterpret_cast<int4*>(set_id + g0) = make_int4(ids[0], ids[1], ids[2], ids[3]);
            } else {
#pragma unroll
                for (int t = 0; t < EM; ++t)
                    if (t < n) set_id[g0 + t] = ids[t];
            }
        }
    }
    if (threadIdx.x == 0) {
        if (n_sets <= cap) st[n_sets] = S;
        out_len[u] = n_sets;
        if (stats) {
            if (fire) atomicAdd(&stats->units_budget_rule, 1);
            if (tot_near) atomicAdd(&stats->near_threshold, tot_near);
            record_out_len(stats, n_sets);
        }
    }

    // ---- 5. segmented arg-max: pivot of each set (ties: lowest index), as in segment_unit_kernel
    float key[EM];
#pragma unroll
    for (int t = 0; t < EM; ++t) {
        key[t] = a[t];
        if (pivot_rule == KVM_PIVOT_LAST) key[t] = (float)(lo + t);
        else if (pivot_rule == KVM_PIVOT_KEY && t < n) key[t] = pivot_key[g0 + t];
    }
    Best head = {-INFINITY, INT_MAX}, run = {-INFINITY, INT_MAX};
    bool seen_cut = false;
    int id = before - 1;          // set of the token before `lo`
    int first_cut_id = -1;        // id of the set that starts at this thread's first cut
#pragma unroll
    for (int t = 0; t < EM; ++t) {
        if (!((own >> t) & 1u)) continue;
        if ((cutm >> t) & 1u) {
            if (seen_cut) { if (id < cap) pv[id] = run.i; }       // a set fully inside this range
            else { head = run; first_cut_id = id + 1; }
            seen_cut = true;
            ++id;
            run = {-INFINITY, INT_MAX};
        }
        run = better(run, Best{key[t], lo + t});
    }
    if (!seen_cut) head = run;
    Best x = run;                 // tail if seen_cut, else the whole range (== head)
    int xf = seen_cut ? 1 : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float la = __shfl_up_sync(0xffffffffu, x.a, off);
        const int li = __shfl_up_sync(0xffffffffu, x.i, off);
        const int lf = __shfl_up_sync(0xffffffffu, xf, off);
        if (lane >= off && !xf) { x = better(Best{la, li}, x); xf = lf; }
    }
    if (lane == 31) { sh.warp_a[w] = x.a; sh.warp_p[w] = x.i; sh.warp_f[w] = xf; }
    __syncthreads();
    Best y = {sh.warp_a[lane], sh.warp_p[lane]};
    int yf = sh.warp_f[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float la = __shfl_up_sync(0xffffffffu, y.a, off);
        const int li = __shfl_up_sync(0xffffffffu, y.i, off);
        const int lf = __shfl_up_sync(0xffffffffu, yf, off);
        if (lane >= off && !yf) { y = better(Best{la, li}, y); yf = lf; }
    }
    const float wa = __shfl_sync(0xffffffffu, y.a, (w + 31) & 31);
    const int wi = __shfl_sync(0xffffffffu, y.i, (w + 31) & 31);
    const float pa = __shfl_up_sync(0xffffffffu, x.a, 1);
    const int pi = __shfl_up_sync(0xffffffffu, x.i, 1);
    const int pf = __shfl_up_sync(0xffffffffu, xf, 1);
    Best carry = w ? Best{wa, wi} : Best{-INFINITY, INT_MAX};
    if (lane > 0) carry = pf ? Best{pa, pi} : better(carry, Best{pa, pi});
    if (n > 0) {
        const bool last = (lo + n == S);
        if (seen_cut) {
            const int ended = first_cut_id - 1;
            if (ended >= 0 && ended < cap) pv[ended] = better(carry, head).i;
            if (last && id < cap) pv[id] = run.i;
        } else if (last) {
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
    if (d.set_rule == KVM_SETS_ADJACENT && d.S <= 4 * NT)
        return launch_dependent(segment_unit_reg_kernel<4>, dim3(d.U), dim3(NT), 0, st, scores, sim, set_id, set_start,
                                pivot, out_len, stats, d.S, d.cap, d.n_r, d.n_h, d.eps, d.enforce, d.pivot_rule,
                                d.pivot_rule == KVM_PIVOT_KEY ? d.pivot_key : (const float*)nullptr);
    return launch_dependent(segment_unit_kernel, dim3(d.U), dim3(NT), smem, st, scores, sim, set_id, set_start, pivot,
                            out_len, stats, d.S, d.cap, d.n_r, d.n_h, d.eps, d.enforce, d.pivot_rule,
                            d.pivot_rule == KVM_PIVOT_KEY ? d.pivot_key : (const float*)nullptr, d.set_rule);
}

}  // namespace kvm
