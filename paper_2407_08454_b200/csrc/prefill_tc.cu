// Causal attention over the whole prompt on the 5th-generation tensor cores (bf16 inputs):
//   O_i = sum_{j<=i} softmax_j(c q_i.k_j) v_j,   lse_i = ln sum_{j<=i} exp(c q_i.k_j)          Eq. 1
// This is the attention a prefill runs anyway; its row log-sum-exp is exactly what the score step's row pass
// computes, so a caller that runs this kernel hands `lse` to kvm_compress_with_lse and pays for no row pass.
//
// A work item is one 128-row query tile of one query head with the key/value tiles 0..it it attends to.  Per
// key tile ("step") two tcgen05.mma chains run: S = Q K^T into a 128-column TMEM accumulator, and O += P V into
// another, with P = exp(S - reference) written to shared memory as bf16 by the softmax warps in the layout the
// tensor core reads (128-byte rows, 128-byte swizzle) and V read with its head dimension contiguous (the layout
// it has in memory).  Two groups of four softmax warps take alternate steps, each with its own S accumulator, P
// tile, O accumulator, reference maximum and row sum, so that one group's exponentials run under the other
// group's products; the two partial results of a row are joined when the item ends, by the group that took the
// item's first step (groups swap from item to item: step j of item n belongs to group (j + n) & 1), which reads
// the other group's accumulator first and hands it back at once, so that the other group's first step of the next
// item runs beside the join.  The logits stay two steps ahead of the P V products across item boundaries (the Q
// tile is released when the item's last Q K^T has been issued).  A softmax thread owns one
// query row = one TMEM lane: it holds the 128 logits of a step in registers (the accumulator is handed back at
// once), and multiplies its row of O by exp(old - new reference) only when the maximum has grown by more than
// 8 (log2 units) since the reference was set, so that most steps touch O not at all.
//
// One CTA per SM, persistent:  warps 0-7 softmax (group = warp / 4),  warp 8 producer of the Q and K tiles (TMA,
// 128-byte swizzle; K and V tiles in rings of two),  warp 9 one thread issues the Q K^T MMAs and owns tensor memory,  warp 10 one
// thread issues the P V MMAs (two issuing threads: neither product's waits hold the other's issue up),  warp 11
// producer of the V tiles (the third warpgroup gives registers up to the softmax warpgroups).  Items are dealt
// longest first, boustrophedon.  Every wait on an mbarrier is bounded; a wait that runs out raises a flag, every
// role leaves its loops, the rows in hand are written as NaN, kvm_stats.status is set when given, tensor memory
// is freed.  (The test build of the library, never shipped, shortens the limit and makes the producer leave out one
// V tile, so that this path can be exercised: KVM_TEST_WAIT_LIMIT_CLOCKS, KVM_TEST_DROP_B_STAGE.)
#include <mutex>

#include "tc_common.cuh"

namespace kvm {
namespace {

using namespace tc;

constexpr int TILE = 128;
constexpr int KCHUNK = 64;
constexpr int NKV = 2;                  // ring depth of the K tiles and of the V tiles
constexpr int NGRP = 2;                 // softmax groups taking alternate steps
constexpr int NSOFT = 4 * NGRP;         // softmax warps: one per TMEM lane quarter and group
constexpr int NTHREADS = (NSOFT + 4) * 32;   // three warpgroups: two of softmax warps, one with producer, MMA issue and two idle warps
// Registers: the launch gives every thread 168 (65536 / 384); the softmax warpgroups then take 208 each and the
// third warpgroup keeps 56 (2 x 128 x 208 + 128 x 56 = 60416 <= 384 x 168 = 64512).
constexpr int REGS_SOFTMAX = 208, REGS_OTHER = 56;
constexpr uint32_t CHUNK_BYTES = TILE * 128;            // [128 rows x 64 bf16]
constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
constexpr float RESCALE_STEP = 8.f;     // the reference maximum follows the running maximum in steps of at least this
constexpr uint32_t S_COLS = TILE, O_COL0 = NGRP * S_COLS;  // TMEM columns: S of group 0 | S of group 1 | O 0 | O 1

struct __align__(8) Bars {
    uint64_t q_full, q_empty;
    uint64_t k_full[NKV], k_empty[NKV], v_full[NKV], v_empty[NKV];
    uint64_t s_full[NGRP], s_empty[NGRP];
    uint64_t p_full[NGRP], pv_done[NGRP], o_empty[NGRP];
    uint64_t part_full, part_empty;     // the handing group's row state at item end: written / read
};
struct alignas(16) Shared {
    Bars bar;
    uint32_t tmem_base;
    int abort_flag;
    float part_m[TILE], part_l[TILE];   // the handing group's row state at item end (through part_full / part_empty)
};

struct Sched {
    int P, c, NH, T;
    // (32-bit arithmetic: the launcher refuses shapes whose item count does not fit; a 64-bit division here costs
    // every role several hundred clocks at every item boundary)
    __device__ __forceinline__ bool item(int n, int& head, int& tile) const {
        const unsigned k = (unsigned)n * (unsigned)P + (unsigned)((n & 1) ? (P - 1 - c) : c);
        if (k >= (unsigned)NH * (unsigned)T) return false;
        const unsigned r = k / (unsigned)NH;
        head = (int)(k - r * (unsigned)NH);
        tile = T - 1 - (int)r;
        return true;
    }
};

template <int KCH>
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_attend_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ O,
                      float* __restrict__ lse, kvm_stats* stats, int B, int Hq, int Hkv, int S, float scale2) {
    constexpr int D = KCH * KCHUNK;
    constexpr uint32_t TILE_BYTES = KCH * CHUNK_BYTES;     // a Q, K or V tile
    constexpr uint32_t P_BYTES = 2 * CHUNK_BYTES;          // P: [2 key chunks][128 rows][128 B]
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* sQ = aligned;
    uint8_t* sK = sQ + TILE_BYTES;
    uint8_t* sV = sK + NKV * TILE_BYTES;
    uint8_t* sP = sV + NKV * TILE_BYTES;                   // one P tile per group
    Shared& sh = *reinterpret_cast<Shared*>(sP + NGRP * P_BYTES);
    volatile int* abort_flag = &sh.abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = Hq / Hkv;
    const int T = (S + TILE - 1) / TILE;
    const Sched sc{(int)gridDim.x, (int)blockIdx.x, B * Hq, T};

    if (threadIdx.x == 0) {
        mbar_init(&sh.bar.q_full, 1); mbar_init(&sh.bar.q_empty, 1);
        for (int i = 0; i < NKV; ++i) {
            mbar_init(&sh.bar.k_full[i], 1); mbar_init(&sh.bar.k_empty[i], 1);
            mbar_init(&sh.bar.v_full[i], 1); mbar_init(&sh.bar.v_empty[i], 1);
        }
        for (int i = 0; i < NGRP; ++i) {
            mbar_init(&sh.bar.s_full[i], 1); mbar_init(&sh.bar.s_empty[i], 4);
            mbar_init(&sh.bar.p_full[i], 4); mbar_init(&sh.bar.pv_done[i], 1);
        }
        for (int i = 0; i < NGRP; ++i) mbar_init(&sh.bar.o_empty[i], 4);
        mbar_init(&sh.bar.part_full, 4); mbar_init(&sh.bar.part_empty, 4);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == NSOFT + 1) tmem_alloc(&sh.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp >= NSOFT) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_OTHER));
      if (warp == NSOFT) {
        // ============================== producer of the Q and K tiles ==============================
        // (The V tiles have a producer of their own: a V tile's slot comes free a step or two after the K tile's
        // of the same step, and one thread loading both in turn would hold the next K tile back behind that wait.)
        if (lane == 0) {
            uint32_t kv = 0;                                  // K tiles loaded so far
            bool ok = true;
            int head, tile;
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                ok = mbar_wait(&sh.bar.q_empty, (n & 1) ^ 1, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&sh.bar.q_full, TILE_BYTES);
#pragma unroll
                for (int kc = 0; kc < KCH; ++kc)
                    tma_load_3d(sQ + kc * CHUNK_BYTES, &map_q, &sh.bar.q_full, kc * KCHUNK, tile * TILE, head);
                const int kvhead = (head / Hq) * Hkv + (head % Hq) / G;
                for (int j = 0; j <= tile; ++j, ++kv) {
                    const int s = kv % NKV;
                    ok = mbar_wait(&sh.bar.k_empty[s], ((kv / NKV) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&sh.bar.k_full[s], TILE_BYTES);
#pragma unroll
                    for (int kc = 0; kc < KCH; ++kc)
                        tma_load_3d(sK + s * TILE_BYTES + kc * CHUNK_BYTES, &map_k, &sh.bar.k_full[s], kc * KCHUNK,
                                    j * TILE, kvhead);
                }
            }
            // Copies already issued complete on their own; before shared memory is given back, let them land
            // (bounded: each try_wait suspends for a while by itself).
            if (*abort_flag)
                for (uint32_t it = 0; it < (1u << 14); ++it) mbar_try(&sh.bar.q_full, 0);
        }
      } else if (warp == NSOFT + 3) {
        // ============================== producer of the V tiles ==============================
        if (lane == 0) {
            uint32_t kv = 0;                                  // V tiles loaded so far
            bool ok = true;
            int head, tile;
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                const int kvhead = (head / Hq) * Hkv + (head % Hq) / G;
                for (int j = 0; j <= tile; ++j, ++kv) {
#ifdef KVM_TEST_DROP_B_STAGE
                    if (kv == (uint32_t)(KVM_TEST_DROP_B_STAGE)) continue;   // test build only: this V tile never arrives
#endif
                    const int s = kv % NKV;
                    ok = mbar_wait(&sh.bar.v_empty[s], ((kv / NKV) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&sh.bar.v_full[s], TILE_BYTES);
#pragma unroll
                    for (int kc = 0; kc < KCH; ++kc)
                        tma_load_3d(sV + s * TILE_BYTES + kc * CHUNK_BYTES, &map_v, &sh.bar.v_full[s], kc * KCHUNK,
                                    j * TILE, kvhead);
                }
            }
            if (*abort_flag)
                for (uint32_t it = 0; it < (1u << 14); ++it) mbar_try(&sh.bar.v_full[0], 0);
        }
      } else if (warp == NSOFT + 1) {
        // ============================== MMA issue: S = Q K^T ==============================
        // Step j of item n belongs to group (j + n) & 1.  This thread runs ahead of the P V products as far as the
        // two S accumulators allow (a group's next S is issued as soon as the group has taken the last one into
        // registers), across item boundaries too: Q is released as soon as the item's last Q K^T has been issued,
        // so the next Q tile and the next item's first S tiles arrive while the last products drain.  (Its
        // commits cover its own MMAs only: the two products are issued by two threads.)
        if (lane == 0) {
            constexpr uint32_t IDESC_S = idesc_bf16(TILE);
            const uint64_t desc_q = smem_desc(base);
            const uint64_t desc_k0 = smem_desc(base + TILE_BYTES);
            uint32_t ks_cnt = 0;                             // K tiles consumed so far
            uint32_t s_cnt[NGRP] = {0, 0};                   // per group: S tiles produced
            bool ok = true;
            int head, tile;
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                ok = mbar_wait(&sh.bar.q_full, n & 1, abort_flag);
                for (int j = 0; ok && j <= tile; ++j) {
                    const int g = (j + n) & 1;
                    const int s = ks_cnt % NKV;
                    ok = mbar_wait(&sh.bar.k_full[s], (ks_cnt / NKV) & 1, abort_flag) &&
                         mbar_wait(&sh.bar.s_empty[g], (s_cnt[g] & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t dk = desc_k0 + (uint64_t)s * (TILE_BYTES >> 4);
#pragma unroll
                    for (int kc = 0; kc < KCH; ++kc)
#pragma unroll
                        for (int ks = 0; ks < KCHUNK / 16; ++ks)
                            umma_bf16(tmem_base + g * S_COLS, desc_q + ((kc * CHUNK_BYTES + ks * 32) >> 4),
                                      dk + ((kc * CHUNK_BYTES + ks * 32) >> 4), IDESC_S, (kc | ks) ? 1u : 0u);
                    umma_commit(&sh.bar.k_empty[s]);
                    umma_commit(&sh.bar.s_full[g]);
                    ++ks_cnt; ++s_cnt[g];
                }
                if (ok) umma_commit(&sh.bar.q_empty);        // every product that reads this Q tile has been issued
            }
        }
      } else if (warp == NSOFT + 2) {
        // ============================== MMA issue: O += P V ==============================
        if (lane == 0) {
            constexpr uint32_t IDESC_O = idesc_bf16(D, true);
            const uint32_t v_addr0 = base + TILE_BYTES + NKV * TILE_BYTES;
            const uint64_t desc_p0 = smem_desc(v_addr0 + NKV * TILE_BYTES);
            uint32_t vs_cnt = 0;                             // V tiles consumed so far
            uint32_t pv_cnt[NGRP] = {0, 0};                  // per group: P V products issued
            bool ok = true;
            int head, tile;
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                for (int j = 0; ok && j <= tile; ++j) {
                    const int g = (j + n) & 1;
                    if (j < 2) ok = mbar_wait(&sh.bar.o_empty[g], (n & 1) ^ 1, abort_flag);   // the last item's O of this group has been read
                    const int s = vs_cnt % NKV;
                    ok = ok && mbar_wait(&sh.bar.p_full[g], pv_cnt[g] & 1, abort_flag) &&
                         mbar_wait(&sh.bar.v_full[s], (vs_cnt / NKV) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t dv0 = smem_desc_mn(v_addr0 + s * TILE_BYTES, CHUNK_BYTES);   // 16 keys further: + 2 KB
                    const uint64_t dp = desc_p0 + (uint64_t)g * (P_BYTES >> 4);
#pragma unroll
                    for (int kk = 0; kk < TILE / 16; ++kk)          // 16 keys per MMA
                        umma_bf16(tmem_base + O_COL0 + g * S_COLS, dp + (((kk / 4) * CHUNK_BYTES + (kk % 4) * 32) >> 4),
                                  dv0 + (uint64_t)((kk * 16 * 128) >> 4), IDESC_O, ((j >> 1) | kk) ? 1u : 0u);
                    umma_commit(&sh.bar.v_empty[s]);
                    umma_commit(&sh.bar.pv_done[g]);         // the group's P may be overwritten, its O read or rescaled
                    ++vs_cnt; ++pv_cnt[g];
                }
            }
        }
      }
    } else {
        // ============================== softmax ==============================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
        const int grp = warp >> 2, lq = warp & 3;
        const int row = lq * 32 + lane;                      // query row of the tile = TMEM lane
        const uint32_t t_lane = tmem_base + ((uint32_t)(lq * 32) << 16);
        const uint32_t t_s = t_lane + grp * S_COLS, t_o = t_lane + O_COL0 + grp * S_COLS;
        uint8_t* prow = sP + grp * P_BYTES + row * 128;
        uint32_t s_cnt = 0, pv_cnt = 0;                      // this group's steps so far
        uint32_t pv_other = 0;                               // the other group's (the joining group reads both results)
        bool ok = true;
        int head, tile;
        for (int n = 0; ok && sc.item(n, head, tile); ++n) {
            float m = -INFINITY, l = 0.f;                    // reference maximum (log2 units) and sum relative to it
            const int j_first = (grp + n) & 1;               // this group's first step of the item
            for (int j = j_first; j <= tile; j += NGRP) {
                ok = mbar_wait(&sh.bar.s_full[grp], s_cnt & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t vr[TILE];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld32_issue(t_s + q * 32, vr + q * 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.bar.s_empty[grp]);   // the accumulator goes back at once
                ++s_cnt;
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_fence(vr + q * 32);
                float v[TILE];
#pragma unroll
                for (int c = 0; c < TILE; ++c) v[c] = __uint_as_float(vr[c]);
                if (j == tile) {                             // diagonal tile: keys after the query do not exist for it
#pragma unroll
                    for (int c = 0; c < TILE; ++c)
                        if (c > row) v[c] = -INFINITY;
                }
                float mx = v[0];
#pragma unroll
                for (int c = 1; c + 1 < TILE; c += 2) mx = fmax3(mx, v[c], v[c + 1]);
                mx = fmaxf(mx, v[TILE - 1]) * scale2;
                // the reference moves only when the maximum has outgrown it by RESCALE_STEP: exp2(x - m) stays
                // below 2^RESCALE_STEP, and O is rescaled rarely
                float alpha = 1.f;
                const bool first = j == j_first;             // the group's first step of the item
                const bool grow = mx > m + RESCALE_STEP;
                if (first) m = mx;
                else if (grow) { alpha = ex2(m - mx); m = mx; }
                const bool rescale = !first && __any_sync(0xffffffffu, grow);
                // p = 2^(x - m), summed in fp32, rounded to bf16 for the tensor core
                const uint64_t sc2 = pack2(scale2, scale2), nm2 = pack2(-m, -m);
                float sum[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pk[TILE / 2];
#pragma unroll
                for (int c = 0; c < TILE; c += 2) {
                    float x0, x1;
                    unpack2(ffma2(pack2(v[c], v[c + 1]), sc2, nm2), x0, x1);
                    const float e0 = ex2(x0), e1 = ex2(x1);
                    sum[(c >> 1) & 3] += e0 + e1;
                    pk[c >> 1] = Vec<__nv_bfloat16>::pack2(e0, e1);
                }
                l = l * alpha + ((sum[0] + sum[1]) + (sum[2] + sum[3]));
                // the group's previous P V has to be done before its P is overwritten or its O rescaled
                ok = mbar_wait(&sh.bar.pv_done[grp], (pv_cnt & 1) ^ 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (rescale) {
                    tc_fence_after();
#pragma unroll
                    for (int q = 0; q < D / 32; ++q) {
                        uint32_t orr[32];
                        tmem_ld32_issue(t_o + q * 32, orr);
                        tmem_ld_wait();
                        tmem_ld_fence(orr);
#pragma unroll
                        for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                        tmem_st32(t_o + q * 32, orr);
                    }
                    tmem_st_wait();
                }
                // P row: 16-byte piece c of key chunk kc sits at piece c ^ (row & 7) of the row's 128 bytes
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int kc = c >> 3, piece = c & 7;
                    *reinterpret_cast<uint4*>(prow + kc * CHUNK_BYTES + ((piece ^ (row & 7)) << 4)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                }
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.bar.p_full[grp]);
                ++pv_cnt;
            }
            const int n_own = tile >= j_first ? (tile - j_first) / 2 + 1 : 0;
            const int n_other = tile + 1 - n_own;            // steps the other group takes in this item
            pv_other += n_other;
            // ---- item end: one group hands its row state to the other, which joins the two partial results:
            //      O = (O_a 2^(m_a - M) + O_b 2^(m_b - M)) / (l_a 2^(m_a - M) + l_b 2^(m_b - M)),  M = max(m_a, m_b)
            // The joining group is the one that took the item's first step (group n & 1), so the other one is
            // free for the next item's first step while the join runs.
            if (grp != (n & 1)) {
                // (every item, also one in which this group had no step: the two groups count items alike)
                ok = ok && mbar_wait(&sh.bar.part_empty, (n & 1) ^ 1, abort_flag);   // the last item's has been read
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                sh.part_m[row] = m;
                sh.part_l[row] = l;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.bar.part_full);
                continue;
            }
            if (ok) {
                ok = mbar_wait(&sh.bar.part_full, n & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
            }
            const float m1 = ok ? sh.part_m[row] : -INFINITY, l1 = ok ? sh.part_l[row] : 0.f;
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(&sh.bar.part_empty);
            const int gi = tile * TILE + row;
            if (ok) {
                ok = mbar_wait(&sh.bar.pv_done[grp], (pv_cnt & 1) ^ 1, abort_flag);
                if (ok && n_other > 0) ok = mbar_wait(&sh.bar.pv_done[grp ^ 1], (pv_other & 1) ^ 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
            }
            ok = ok && (*abort_flag == 0);
            __nv_bfloat16* orow = O + ((size_t)head * S + gi) * D;
            if (ok) {
                tc_fence_after();
                const float M = fmaxf(m, m1);
                const float w0 = n_own > 0 ? ex2(m - M) : 0.f, w1 = n_other > 0 ? ex2(m1 - M) : 0.f;
                const float L = l * w0 + l1 * w1;
                const float f0 = w0 / L, f1 = w1 / L;
                // the other group's accumulator first, whole, so that it goes back at once: that group is
                // already at work on the next item
                // (a group without a step in this item has a stale accumulator: it is read all the same, so that
                // the registers are not conditional, and replaced by zeros)
                uint32_t o1[D];
#pragma unroll
                for (int q = 0; q < D / 32; ++q) tmem_ld32_issue(t_lane + O_COL0 + (grp ^ 1) * S_COLS + q * 32, o1 + q * 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.bar.o_empty[grp ^ 1]);
#pragma unroll
                for (int q = 0; q < D / 32; ++q) tmem_ld_fence(o1 + q * 32);
                const bool has0 = n_own > 0, has1 = n_other > 0;
#pragma unroll
                for (int q = 0; q < D / 32; ++q) {
                    uint32_t o0[32];
                    tmem_ld32_issue(t_o + q * 32, o0);
                    tmem_ld_wait();
                    tmem_ld_fence(o0);
                    if (gi < S) {
#pragma unroll
                        for (int c = 0; c < 32; c += 8) {
                            float f[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const float a0 = has0 ? __uint_as_float(o0[c + e]) : 0.f;
                                const float a1 = has1 ? __uint_as_float(o1[q * 32 + c + e]) : 0.f;
                                f[e] = fmaf(a1, f1, a0 * f0);
                            }
                            *reinterpret_cast<uint4*>(orow + q * 32 + c) = Vec<__nv_bfloat16>::pack(f);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.bar.o_empty[grp]);
                if (gi < S) lse[(size_t)head * S + gi] = (M + log2f(L)) * LN2;
            } else if (gi < S) {
                // a wait gave up: what this row would have received is marked, not made up
                for (int c = 0; c < D; c += 8)
                    *reinterpret_cast<uint4*>(orow + c) = make_uint4(0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u);
                lse[(size_t)head * S + gi] = NAN;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && sh.abort_flag && stats) stats->status = KVM_E_DEVICE_TIMEOUT;
    if (warp == NSOFT + 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

template <int KCH>
cudaError_t launch_t(const Dims& d, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     __nv_bfloat16* O, float* lse, kvm_stats* stats, cudaStream_t st) {
    const size_t smem = 1024 + (size_t)(1 + 2 * NKV) * KCH * CHUNK_BYTES + NGRP * 2 * CHUNK_BYTES + sizeof(Shared);
    static std::mutex mu;
    static int sms_of[KVM_MAX_DEVICES] = {};
    cudaError_t e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if (dev < 0 || dev >= KVM_MAX_DEVICES) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!sms_of[dev]) {
            e = cudaFuncSetAttribute(prefill_attend_kernel<KCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
            sms_of[dev] = sms;
        }
        sms = sms_of[dev];
    }
    const int T = (d.S + TILE - 1) / TILE;
    const long long items = (long long)d.B * d.Hq * T;
    if (items + sms >= (1ll << 31)) return cudaErrorInvalidValue;   // the schedule counts items in 32 bits
    const int grid = (int)(items < sms ? items : sms);
    prefill_attend_kernel<KCH><<<grid, NTHREADS, smem, st>>>(mq, mk, mv, O, lse, stats, d.B, d.Hq, d.Hkv, d.S,
                                                            d.scale * LOG2E);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_attend(const Dims& d, const void* Q, const void* K, const void* V, void* O, float* lse,
                                  kvm_stats* stats, cudaStream_t st) {
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, Q, d.B * d.Hq, d.S, d.D) || !make_map(&mk, K, d.B * d.Hkv, d.S, d.D) ||
        !make_map(&mv, V, d.B * d.Hkv, d.S, d.D))
        return cudaErrorNotSupported;
    __nv_bfloat16* Ob = reinterpret_cast<__nv_bfloat16*>(O);
    return d.D == 128 ? launch_t<2>(d, mq, mk, mv, Ob, lse, stats, st) : launch_t<1>(d, mq, mk, mv, Ob, lse, stats, st);
}

}  // namespace kvm
