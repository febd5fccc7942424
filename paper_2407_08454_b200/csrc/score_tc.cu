// Aggregated attention scores on the 5th-generation tensor cores (bf16 inputs).
//
//   pass 1 (row pass)     lse_i = ln sum_{j<=i} exp(c q_i.k_j)                     Eq. 1, causal
//   pass 2 (column pass)  a_j   = (1/G) sum_g sum_{i>=j} exp(c q^g_i.k_j - lse^g_i)  Algorithm 2 / Eq. 6, Section 5.2
//
// Both passes are the same machine.  A work item owns one 128-row "A" tile that
// stays in shared memory (a query tile in pass 1, a key tile in pass 2) and
// streams the 128-row "B" tiles it interacts with under the causal mask (key
// tiles 0..it, resp. query tiles jt..T-1 of each of the G query heads).  Each
// step multiplies the A tile with two B tiles at once: a 128x256xD tcgen05.mma
// chain (the shape at which one CTA's tensor core runs at full rate) into a
// 256-column TMEM accumulator whose lanes are the A rows.  In pass 1 a thread therefore owns a
// query row and keeps its running max / sum; in pass 2 the product is computed
// transposed (A = keys), so a thread owns a key and adds up its column of the
// attention map in registers, with no cross-lane reduction.
//
// Pass 2 needs exp(c s_ij - lse_i) with lse varying along the accumulator's columns.  Instead of
// fetching lse per column in the epilogue, pass 1 stores e_i = -lse_i / c as three bf16 terms
// (hi + mid + lo, 24 significant bits) in a 16-channel side tensor, and pass 2 appends one more
// K = 16 MMA per step: A' = ones in the three channels, B' = that side tensor.  The tensor core,
// which is far from busy here, then delivers q.k - lse/c directly and the epilogue is a bare
// multiply, exponential and add per logit.
//
// One CTA per SM, persistent, warp-specialised:
//   warps 0-15 epilogue: two groups of 8 take alternate steps; a warp reads TMEM lanes
//              32*(w%4).. and one column half, does exp2 on the SFUs, keeps row/column state;
//              steps that no mask touches (all but an item's diagonal and ragged tiles) run
//              straight-line code, the others a general path
//   warp  16   producer: TMA (cp.async.bulk.tensor, 128B swizzle) into a 2-stage ring of B pairs
//   warp  17   MMA issue: one thread issues tcgen05.mma / tcgen05.commit; owns TMEM
// Work items are dealt in descending length, boustrophedon over the CTAs, which
// keeps the static schedule within 2 % of a greedy one.
//
// Every wait on an mbarrier is bounded.  A wait that runs out raises a flag in
// shared memory; from then on every role stops touching tensor memory and
// barriers' payloads, finishes its loops without waiting, the outputs of the
// affected items are poisoned with NaN, kvm_stats.status is set when given,
// tensor memory is freed and the kernel returns.
//
// Two compile-time switches exist for the test of that give-up path and are never set in the
// library that ships: KVM_TEST_WAIT_LIMIT_CLOCKS shortens the limit of every wait, and
// KVM_TEST_DROP_B_STAGE = k makes the producer leave out its k-th B stage (barrier not armed,
// copies not issued), so that the MMA warp's wait for it runs out.
#include <cuda.h>

#include <mutex>

#include "similarity_core.cuh"
#include "tc_common.cuh"

namespace kvm {
namespace {

using namespace tc;

constexpr int TILE = 128;            // rows of an A or B tile = MMA M = MMA N
constexpr int KCHUNK = 64;           // bf16 elements per 128-byte swizzle row
constexpr int NSTAGE = 2;            // ring of B pairs (two 128-row tiles each)
constexpr int NSLOT = 4;             // item-end buffers in rotation
constexpr int NACC = 2;              // TMEM accumulator ring (2 x 256 columns = all 512)
constexpr int ACC_COLS = 2 * TILE;   // accumulator columns per step
constexpr int PCH = 16;              // channels of the lse side tensor (one K = 16 MMA slice; 3 are used)
constexpr uint32_t PTILE_BYTES = TILE * PCH * 2;   // 4 KB: 128 rows x 32 B
constexpr int NEPI_WARPS = 16;           // 4 TMEM lane quarters x 2 groups x 2 column halves
constexpr int QCOLS = TILE / 4;          // columns of one TMEM load (a "quarter" of a sub-tile)
constexpr int QPW = 2;                   // quarters of a 128-column sub-tile a warp owns
constexpr int NSIM_WARPS = 2;           // neighbour-key similarities on the side (one of the two passes)
constexpr int SIM_RUN = 8;              // consecutive tokens per lane group and round trip
constexpr int NTHREADS = (NEPI_WARPS + 2 + NSIM_WARPS) * 32;
constexpr float LOG2E = 1.4426950408889634f;

constexpr uint32_t IDESC_N128 = tc::idesc_bf16(TILE), IDESC_N256 = tc::idesc_bf16(2 * TILE);

// ------------------------------------------------------------------ per-chunk arithmetic of the two passes
// A chunk is 32 consecutive accumulator columns of this thread's row, already masked with -inf where the
// causal mask or the sequence end excludes them.  The exponentials' results are added one by one: packing them
// into pairs for a packed add costs a register move per result, which is more than the add it saves.
//
// Row pass: fold the chunk into the running maximum m and sum l (log2 units: x = v * scale2).
__device__ __forceinline__ void chunk_row_pass(const float (&v)[QCOLS], float& m, float& l, float scale2, uint64_t sc2) {
    float mx[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        mx[c] = fmax3(v[c], v[c + 4], v[c + 8]);
        mx[c] = fmax3(mx[c], v[c + 12], v[c + 16]);
        mx[c] = fmax3(mx[c], v[c + 20], v[c + 24]);
        mx[c] = fmaxf(mx[c], v[c + 28]);
    }
    const float mtile = fmaxf(fmax3(mx[0], mx[1], mx[2]), mx[3]);
    const float mnew = fmaxf(m, mtile * scale2);
    if (mnew > -INFINITY) {
        // packed multiply-add for the exponents (the accumulator registers come in adjacent pairs)
        const uint64_t nm2 = pack2(-mnew, -mnew);
        float sum[8] = {l * ex2(m - mnew), 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < QCOLS; c += 2) {
            float x0, x1;
            unpack2(ffma2(pack2(v[c], v[c + 1]), sc2, nm2), x0, x1);
            sum[c & 7] += ex2(x0);
            sum[(c + 1) & 7] += ex2(x1);
        }
        l = ((sum[0] + sum[1]) + (sum[2] + sum[3])) + ((sum[4] + sum[5]) + (sum[6] + sum[7]));
        m = mnew;
    }
}
// Column pass: the accumulator already holds q.k - lse/c; scale, exponentiate, add to eight partial sums.
__device__ __forceinline__ void chunk_col_pass(const float (&v)[QCOLS], float (&acc)[8], uint64_t sc2) {
#pragma unroll
    for (int c = 0; c < QCOLS; c += 2) {
        float x0, x1;
        unpack2(fmul2(pack2(v[c], v[c + 1]), sc2), x0, x1);
        acc[c & 7] += ex2(x0);
        acc[(c + 1) & 7] += ex2(x1);
    }
}

// ------------------------------------------------------------------ static schedule
struct Sched {
    int P, c, NH, T, G, pass;
    // n-th item of this CTA -> (head or unit, tile).  Items are sorted by descending length
    // (pass 1: query tile T-1 first; pass 2: key tile 0 first) and dealt boustrophedon.
    // (32-bit arithmetic: NH * T + P stays far below 2^31 for any tensors that fit a GPU, and the launcher
    // refuses the rest; a 64-bit division here costs every role several hundred clocks at every item boundary)
    __device__ __forceinline__ bool item(int n, int& head, int& tile) const {
        const unsigned k = (unsigned)n * (unsigned)P + (unsigned)((n & 1) ? (P - 1 - c) : c);
        if (k >= (unsigned)NH * (unsigned)T) return false;
        const unsigned r = k / (unsigned)NH;
        head = (int)(k - r * (unsigned)NH);
        tile = (pass == 1) ? (T - 1 - (int)r) : (int)r;
        return true;
    }
    __device__ __forceinline__ int ntiles(int tile) const { return (pass == 1) ? tile + 1 : G * (T - tile); }
};

// Walks a CTA's steps (pairs of B tiles) across its items; (bg, bt) = query head within the group and
// query tile of the step's first B tile in pass 2, advanced without divisions.
struct StepIter {
    int n, t0, head, tile, nt, bg, bt;
    uint32_t cnt;
    bool valid;
    __device__ __forceinline__ void load(const Sched& sc) {
        valid = sc.item(n, head, tile);
        nt = valid ? sc.ntiles(tile) : 0;
        t0 = 0; bg = 0; bt = tile;
    }
    __device__ __forceinline__ void init(const Sched& sc) { n = 0; cnt = 0; load(sc); }
    __device__ __forceinline__ void next(const Sched& sc) {
        if (!valid) return;
        ++cnt;
        t0 += 2;
        if (t0 >= nt) { ++n; load(sc); return; }
        if (sc.pass == 2) {
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (++bt == sc.T) { bt = tile; ++bg; }
        }
    }
};

struct __align__(8) Barriers {
    uint64_t full_a[2], empty_a[2];
    uint64_t full_b[NSTAGE], empty_b[NSTAGE];
    uint64_t acc_full[NACC], acc_empty[NACC];
};

struct alignas(16) Shared {
    Barriers bar;
    uint32_t tmem_base;
    int abort_flag;
    // Partial sums of the four warp sets at item end, in NSLOT buffers used in rotation (item n uses n mod
    // NSLOT; see the item end), and how many of the four warps that own a lane quarter's rows have delivered
    // theirs.  (The row pass also needs the partial maxima and keeps both arrays where the column pass keeps
    // its side tiles, which the row pass does not have.)
    float part_l[NSLOT][4][TILE];
    int arrived[NSLOT][4];
};

template <int KCH, int PASS>
__global__ void __launch_bounds__(NTHREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_p, __nv_bfloat16* __restrict__ lsep_out,
                float* __restrict__ scores, kvm_stats* stats, int B, int Hq, int Hkv, int S,
                float scale2, const __nv_bfloat16* __restrict__ Ksim, float* __restrict__ sim_out) {
    constexpr int pass = PASS;
    extern __shared__ uint8_t smem_raw[];
    constexpr uint32_t CHUNK_BYTES = TILE * 128;            // one [128 rows x 64 bf16] TMA box
    constexpr uint32_t TILE_BYTES = KCH * CHUNK_BYTES;      // an A tile: [KCH][128 rows][128 B]
    constexpr uint32_t PAIR_CHUNK = 2 * CHUNK_BYTES;        // a B pair: [KCH][256 rows][128 B]
    constexpr uint32_t PAIR_BYTES = KCH * PAIR_CHUNK;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* sA = aligned;                                  // 2 A tiles
    uint8_t* sB = aligned + 2 * TILE_BYTES;                 // NSTAGE B pairs
    uint8_t* sP = sB + NSTAGE * PAIR_BYTES;                 // NSTAGE pairs of lse side tiles (pass 2)
    uint8_t* sOnes = sP + NSTAGE * 2 * PTILE_BYTES;         // constant A' tile: ones in the used channels
    Shared& sh = *reinterpret_cast<Shared*>(sOnes + PTILE_BYTES);
    volatile int* abort_flag = &sh.abort_flag;
    static_assert(2 * NSLOT * 4 * TILE * sizeof(float) <= NSTAGE * 2 * PTILE_BYTES, "the row pass's item-end buffers fit the side tiles' space");
    float* part_m = reinterpret_cast<float*>(sP);                                   // [NSLOT][4][TILE], row pass only
    float* part_l = (pass == 1) ? part_m + NSLOT * 4 * TILE : &sh.part_l[0][0][0];     // [NSLOT][4][TILE]

    grid_dependency_wait();     // the column pass reads what the row pass (or the lse conversion) wrote
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = Hq / Hkv;
    const int T = (S + TILE - 1) / TILE;
    Sched sc{(int)gridDim.x, (int)blockIdx.x, pass == 1 ? B * Hq : B * Hkv, T, G, pass};

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.bar.full_a[i], 1); mbar_init(&sh.bar.empty_a[i], 1); }
        for (int i = 0; i < NSTAGE; ++i) { mbar_init(&sh.bar.full_b[i], 1); mbar_init(&sh.bar.empty_b[i], 1); }
        for (int i = 0; i < NACC; ++i) { mbar_init(&sh.bar.acc_full[i], 1); mbar_init(&sh.bar.acc_empty[i], NEPI_WARPS / 2); }
        sh.abort_flag = 0;
        for (int i = 0; i < NSLOT * 4; ++i) (&sh.arrived[0][0])[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (pass == 2 && threadIdx.x < PTILE_BYTES / 16) {
        // every 16-byte chunk of every row = bf16 {1, 1, 1, 0, 0, 0, 0, 0}: the same under any swizzle; the B'
        // side tensor is zero outside channels 0..2, so the ones of the second chunk multiply zeros
        reinterpret_cast<uint4*>(sOnes)[threadIdx.x] = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core's reads
    }
    if (warp == NEPI_WARPS + 1) tmem_alloc(&sh.tmem_base, NACC * ACC_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    // An item's B tiles are consumed two at a time ("steps"): one 128 x 256 MMA chain per step
    // (128 x 128 for an odd last tile).  `cnt` counts steps of this CTA across items.
    if (warp == NEPI_WARPS) {
        // ============================== producer ==============================
        if (lane == 0) {
            const CUtensorMap* mapA = (pass == 1) ? &map_q : &map_k;
            const CUtensorMap* mapB = (pass == 1) ? &map_k : &map_q;
            uint32_t cnt = 0;
            bool ok = true;
            int head, tile;
            int last_a[2] = {-1, -1}, last_b[NSTAGE];      // parity of the last load issued per buffer (-1: none)
            for (int s = 0; s < NSTAGE; ++s) last_b[s] = -1;
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                const int ab = n & 1;
                ok = mbar_wait(&sh.bar.empty_a[ab], ((n >> 1) & 1) ^ 1, abort_flag);
                if (!ok) break;
                last_a[ab] = (n >> 1) & 1;
                mbar_expect_tx(&sh.bar.full_a[ab], TILE_BYTES);
#pragma unroll
                for (int kc = 0; kc < KCH; ++kc)
                    tma_load_3d(sA + ab * TILE_BYTES + kc * CHUNK_BYTES, mapA, &sh.bar.full_a[ab], kc * KCHUNK,
                                tile * TILE, head);
                const int nt = sc.ntiles(tile);
                const int b = head / (pass == 1 ? Hq : Hkv), hh = head % (pass == 1 ? Hq : Hkv);
                int bhead = (pass == 1) ? b * Hkv + hh / G : b * Hq + hh * G;   // B tile cursor, advanced incrementally
                int btile = (pass == 1) ? 0 : tile;
                for (int t = 0; t < nt; t += 2, ++cnt) {
                    const int s = cnt % NSTAGE;
                    const int nh = (t + 1 < nt) ? 2 : 1;
                    ok = mbar_wait(&sh.bar.empty_b[s], ((cnt / NSTAGE) & 1) ^ 1, abort_flag);
                    if (!ok) break;
#ifdef KVM_TEST_DROP_B_STAGE
                    if (cnt == (uint32_t)(KVM_TEST_DROP_B_STAGE)) continue;   // test build only: this stage never arrives
#endif
                    last_b[s] = (cnt / NSTAGE) & 1;
                    mbar_expect_tx(&sh.bar.full_b[s], nh * (TILE_BYTES + (pass == 2 ? PTILE_BYTES : 0u)));
                    for (int h = 0; h < nh; ++h) {
#pragma unroll
                        for (int kc = 0; kc < KCH; ++kc)
                            tma_load_3d(sB + s * PAIR_BYTES + kc * PAIR_CHUNK + h * CHUNK_BYTES, mapB,
                                        &sh.bar.full_b[s], kc * KCHUNK, btile * TILE, bhead);
                        if (pass == 2)
                            tma_load_3d(sP + (s * 2 + h) * PTILE_BYTES, &map_p, &sh.bar.full_b[s], 0, btile * TILE,
                                        bhead);
                        if (++btile == T && pass == 2) { btile = tile; ++bhead; }   // next query head of the group
                    }
                }
            }
            // Copies already issued complete on their own; before shared memory is given
            // back, wait (bounded) for the ones nobody consumed.
            if (*abort_flag) {
                for (int s = 0; s < NSTAGE; ++s)
                    for (uint32_t it = 0; last_b[s] >= 0 && it < (1u << 16); ++it)
                        if (mbar_try(&sh.bar.full_b[s], (uint32_t)last_b[s])) break;
                for (int s = 0; s < 2; ++s)
                    for (uint32_t it = 0; last_a[s] >= 0 && it < (1u << 16); ++it)
                        if (mbar_try(&sh.bar.full_a[s], (uint32_t)last_a[s])) break;
            }
        }
    } else if (warp == NEPI_WARPS + 1) {
        // ============================== MMA issue ==============================
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            int head, tile;
            // descriptors differ from a buffer's first one only in the 16-byte-unit start address
            const uint64_t desc_a[2] = {smem_desc(base), smem_desc(base + TILE_BYTES)};
            const uint64_t desc_b0 = smem_desc(base + 2 * TILE_BYTES);
            const uint64_t desc_p0 = smem_desc_sw32(base + 2 * TILE_BYTES + NSTAGE * PAIR_BYTES);
            const uint64_t desc_ones = smem_desc_sw32(base + 2 * TILE_BYTES + NSTAGE * PAIR_BYTES + NSTAGE * 2 * PTILE_BYTES);
            for (int n = 0; ok && sc.item(n, head, tile); ++n) {
                const int ab = n & 1;
                ok = mbar_wait(&sh.bar.full_a[ab], (n >> 1) & 1, abort_flag);
                if (!ok) break;
                const int nt = sc.ntiles(tile);
                for (int t = 0; t < nt; t += 2, ++cnt) {
                    const int s = cnt % NSTAGE, as = cnt % NACC;
                    ok = mbar_wait(&sh.bar.full_b[s], (cnt / NSTAGE) & 1, abort_flag) &&
                         mbar_wait(&sh.bar.acc_empty[as], ((cnt / NACC) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t idesc = (t + 1 < nt) ? IDESC_N256 : IDESC_N128;
                    const uint64_t da = desc_a[ab], db = desc_b0 + (uint64_t)s * (PAIR_BYTES >> 4);
                    const uint32_t d = tmem_base + as * ACC_COLS;
#pragma unroll
                    for (int kc = 0; kc < KCH; ++kc)
#pragma unroll
                        for (int ks = 0; ks < KCHUNK / 16; ++ks)
                            umma_bf16(d, da + ((kc * CHUNK_BYTES + ks * 32) >> 4), db + ((kc * PAIR_CHUNK + ks * 32) >> 4),
                                      idesc, (kc | ks) ? 1u : 0u);
                    if (pass == 2)                         // + ones x (-lse/c): one more K = 16 slice
                        umma_bf16(d, desc_ones, desc_p0 + (uint64_t)s * ((2 * PTILE_BYTES) >> 4), idesc, 1u);
                    umma_commit(&sh.bar.empty_b[s]);       // B stage reusable once these MMAs retire
                    umma_commit(&sh.bar.acc_full[as]);     // accumulator ready for the epilogue
                }
                if (ok) umma_commit(&sh.bar.empty_a[ab]);  // A tile reusable
            }
        }
    } else if (warp >= NEPI_WARPS + 2) {
        // ============================== similarity on the side ==============================
        // Eq. 2 needs nothing but K, and the epilogue warps leave issue slots and memory bandwidth unused:
        // the key rows are dealt to these warps of all CTAs in runs of SIM_RUN tokens.
        if (sim_out) {
            constexpr int D = KCH * KCHUNK, LPR = D / 8, GPW = 32 / LPR;
            const int runs = (S + SIM_RUN - 1) / SIM_RUN;
            // (32-bit arithmetic: B * Hkv * runs is far below 2^31 for tensors that fit a GPU — the launcher
            // checks B * Hq * T — and a 64-bit division per run would cost a third of the run's own work)
            const unsigned n_runs = (unsigned)(B * Hkv) * (unsigned)runs;
            const int gl = lane % LPR, gbase = lane / LPR * LPR;
            const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << gbase);
            const unsigned stride = gridDim.x * NSIM_WARPS * GPW;
            for (unsigned g = (blockIdx.x * NSIM_WARPS + (warp - NEPI_WARPS - 2)) * GPW + lane / LPR;
                 g < n_runs; g += stride) {
                const unsigned u = g / (unsigned)runs;
                const int j0 = (int)(g - u * (unsigned)runs) * SIM_RUN;
                simcore::run<__nv_bfloat16, D, SIM_RUN>(Ksim + (size_t)u * S * D, sim_out + (size_t)u * S, j0,
                                                        min(j0 + SIM_RUN, S), gl, gbase, gmask);
            }
        }
    } else {
        // ============================== epilogue ==============================
        // Two groups of warps take alternate steps (group g always reads accumulator stage g), so that one
        // group's waits, TMEM loads and bookkeeping overlap the other group's exponentials.  Within a group a
        // warp owns TMEM lane quarter lq and QPW 32-column quarters of each 128-column sub-tile, fetched LDQ
        // quarters at a time; the accumulator is handed back as soon as the step's last fetch has landed.
        const int lq = warp & 3;                             // TMEM lane quarter this warp may read
        const int grp = (warp >> 2) & 1;                     // steps with (cnt & 1) == grp
        const int part = warp >> 3;                          // which share of a sub-tile's columns (0 when 8 warps)
        const int pidx = warp >> 2;                          // partial-state slot of this warp's rows
        const int row = lq * 32 + lane;                      // A row = TMEM lane
        const uint32_t t_lane = tmem_base + ((uint32_t)(lq * 32) << 16) + grp * ACC_COLS + part * (QPW * QCOLS);
        const uint64_t sc2 = pack2(scale2, scale2);
        bool ok = true;
        StepIter it;
        it.init(sc);
        uint32_t own = 0;                                    // own steps processed (accumulator phase)
        const bool ragged = (S & (TILE - 1)) != 0;
        while (it.valid) {
            const int n = it.n, head = it.head, tile = it.tile;
            float m = -INFINITY, l = 0.f;                    // pass 1 state
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // pass 2 state: eight partial sums
            for (; it.valid && it.n == n; it.next(sc)) {
                if ((int)(it.cnt & 1u) != grp) continue;
                const int nh = (it.t0 + 1 < it.nt) ? 2 : 1;
                ok = mbar_wait(&sh.bar.acc_full[grp], own & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (ok) tc_fence_after();
                const int bt0 = (pass == 1) ? it.t0 : it.bt;                        // B tiles of the two sub-tiles
                const int bt1 = (pass == 1) ? it.t0 + 1 : (it.bt + 1 == T ? tile : it.bt + 1);
                bool interior = ok && nh == 2 && bt0 != tile && bt1 != tile;
                if (pass == 2 && ragged) interior = interior && bt0 != T - 1 && bt1 != T - 1;
                if (interior) {
                    // no mask anywhere in this step: straight-line code
#pragma unroll
                    for (int ch = 0; ch < 2 * QPW; ++ch) {
                        uint32_t vr[QCOLS];
                        tmem_ld32_issue(t_lane + (ch / QPW) * TILE + (ch % QPW) * QCOLS, vr);
                        tmem_ld_wait();
                        if (ch == 2 * QPW - 1) {              // last read of this accumulator: release it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sh.bar.acc_empty[grp]);
                        }
                        tmem_ld_fence(vr);
                        float v[QCOLS];
#pragma unroll
                        for (int c = 0; c < QCOLS; ++c) v[c] = __uint_as_float(vr[c]);
                        if (pass == 1) chunk_row_pass(v, m, l, scale2, sc2);
                        else chunk_col_pass(v, acc, sc2);
                    }
                } else {
                    int btile = bt0;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h >= nh) break;
                        const bool diag = (btile == tile);
#pragma unroll
                        for (int k = 0; k < QPW; ++k) {
                            const int cq = part * QPW + k;       // column quarter of this chunk within the sub-tile
                            // On the diagonal tile whole quarters are masked (skip) or fully valid.
                            const bool skip = !ok || (diag && ((pass == 1) ? (cq > lq) : (cq < lq)));
                            const bool mask = diag && (cq == lq);
                            uint32_t vr[QCOLS];
                            if (!skip) { tmem_ld32_issue(t_lane + h * TILE + k * QCOLS, vr); tmem_ld_wait(); }
                            if (h == nh - 1 && k == QPW - 1) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&sh.bar.acc_empty[grp]);
                            }
                            if (skip) continue;
                            tmem_ld_fence(vr);
                            float v[QCOLS];
#pragma unroll
                            for (int c = 0; c < QCOLS; ++c) v[c] = __uint_as_float(vr[c]);
                            if (pass == 1) {
                                if (mask) {
#pragma unroll
                                    for (int c = 0; c < QCOLS; ++c)
                                        if (c > lane) v[c] = -INFINITY;      // key after query
                                }
                                chunk_row_pass(v, m, l, scale2, sc2);
                            } else {
                                const int ncol = S - btile * TILE - cq * QCOLS;   // live columns of this chunk (queries < S)
                                if (mask || ncol < QCOLS) {
#pragma unroll
                                    for (int c = 0; c < QCOLS; ++c)
                                        if ((mask && c < lane) || c >= ncol) v[c] = -INFINITY;   // query before key, or past the end
                                }
                                chunk_col_pass(v, acc, sc2);
                            }
                        }
                        btile = bt1;
                    }
                }
                ++own;
            }
            // ---- item end: the four warps that own a row (2 groups x 2 column halves) each leave their partial
            // state in shared memory; whichever of them comes last combines the four in a fixed order (so the
            // result does not depend on who does it) and stores.  Nobody waits: the group that had the item's
            // last step is a step behind the other one, which goes straight on to the next item.
            // (Buffers: the MMA thread needs a group's accumulator back before it can issue that group's step after
            // next, and it issues in order; so a warp is at most three steps ahead of a warp of the other group
            // that has handed its accumulator back but not yet finished its step and its item end.  With
            // single-step items three steps are three items: four buffers, so that item n - 4 has been
            // combined, and its count cleared, when item n's states are written.)
            const int slot = n % NSLOT;
            const float mine = (pass == 1) ? l : ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
            constexpr int NPART = NEPI_WARPS / 4;            // partial states per row (one per warp that owns it)
            static_assert(NPART == 4, "four warps own a row");
            float* pm = part_m + slot * 4 * TILE + row;       // + q * TILE: warp set q
            float* pl = part_l + slot * 4 * TILE + row;
            if (pass == 1) pm[pidx * TILE] = m;
            pl[pidx * TILE] = mine;
            __syncwarp();
            int before = 0;
            if (lane == 0) {
                __threadfence_block();
                before = atomicAdd(&sh.arrived[slot][lq], 1);
            }
            before = __shfl_sync(0xffffffffu, before, 0);
            if (before == NPART - 1) {
                __threadfence_block();
                if (lane == 0) sh.arrived[slot][lq] = 0;     // for item n + NSLOT
                // (read after all four have delivered: a warp whose wait ran out raised the flag before it came here)
                const bool bad = (*abort_flag != 0);
                const int gi = tile * TILE + row;
                if (gi < S) {
                    if (pass == 1) {
                        const float m0 = pm[0];
                        float M = m0;
#pragma unroll
                        for (int q = 1; q < NPART; ++q) M = fmaxf(M, pm[q * TILE]);
                        float L = (m0 > -INFINITY) ? pl[0] * ex2(m0 - M) : 0.f;
#pragma unroll
                        for (int q = 1; q < NPART; ++q) {
                            const float mq = pm[q * TILE], lq_ = pl[q * TILE];
                            if (mq > -INFINITY) L += lq_ * ex2(mq - M);
                        }
                        // e = -lse / c in the accumulator's units (lse in log2 units is M + log2 L), as hi + mid + lo
                        const float e = bad ? NAN : -(M + log2f(L)) / scale2;
                        const __nv_bfloat16 eh = __float2bfloat16_rn(e);
                        const float r1 = e - __bfloat162float(eh);
                        const __nv_bfloat16 em = __float2bfloat16_rn(r1);
                        const __nv_bfloat16 el = __float2bfloat16_rn(r1 - __bfloat162float(em));
                        uint4* dst = reinterpret_cast<uint4*>(lsep_out + ((size_t)head * S + gi) * PCH);
                        dst[0] = make_uint4((uint32_t)__bfloat16_as_ushort(eh) | ((uint32_t)__bfloat16_as_ushort(em) << 16),
                                            (uint32_t)__bfloat16_as_ushort(el), 0u, 0u);
                        dst[1] = make_uint4(0u, 0u, 0u, 0u);
                    } else {
                        float tot = pl[0];
#pragma unroll
                        for (int q = 1; q < NPART; ++q) tot += pl[q * TILE];
                        scores[(size_t)head * S + gi] = bad ? NAN : tot / (float)G;
                    }
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && sh.abort_flag && stats) stats->status = KVM_E_DEVICE_TIMEOUT;
    if (warp == NEPI_WARPS + 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, NACC * ACC_COLS);
    }
}

// ------------------------------------------------------------------ host side
// [heads, S, 16] bf16 side tensor of pass 2: boxes of [1, 128 rows, 16 channels] (32-byte rows), 32-byte swizzle.
bool make_map_side(CUtensorMap* map, const void* ptr, int heads, int S) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)PCH, (cuuint64_t)S, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)PCH * 2, (cuuint64_t)S * PCH * 2};
    cuuint32_t box[3] = {PCH, TILE, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Caller-supplied natural-log lse -> the side tensor pass 2 multiplies in (e = -lse * log2(e) / scale2 as hi+mid+lo).
__global__ void __launch_bounds__(256) lse_split_kernel(const float* __restrict__ lse, __nv_bfloat16* __restrict__ side,
                                                        long long rows, float neg_log2e_over_scale2) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const float e = lse[i] * neg_log2e_over_scale2;
    const __nv_bfloat16 eh = __float2bfloat16_rn(e);
    const float r1 = e - __bfloat162float(eh);
    const __nv_bfloat16 em = __float2bfloat16_rn(r1);
    const __nv_bfloat16 el = __float2bfloat16_rn(r1 - __bfloat162float(em));
    uint4* dst = reinterpret_cast<uint4*>(side + (size_t)i * PCH);
    dst[0] = make_uint4((uint32_t)__bfloat16_as_ushort(eh) | ((uint32_t)__bfloat16_as_ushort(em) << 16),
                        (uint32_t)__bfloat16_as_ushort(el), 0u, 0u);
    dst[1] = make_uint4(0u, 0u, 0u, 0u);
}

// The row pass's side tensor back to a natural-log lse per query row: lse = -(hi + mid + lo) * scale2 * ln 2.
__global__ void __launch_bounds__(256) side_to_lse_kernel(const __nv_bfloat16* __restrict__ side, float* __restrict__ lse,
                                                          long long rows, float neg_scale2_ln2) {
    grid_dependency_wait();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const uint2 raw = __ldcg(reinterpret_cast<const uint2*>(side + (size_t)i * PCH));
    const float hi = __uint_as_float(raw.x << 16), mid = __uint_as_float(raw.x & 0xffff0000u);
    const float lo = __uint_as_float(raw.y << 16);
    lse[i] = ((hi + mid) + lo) * neg_scale2_ln2;
}

template <int KCH>
cudaError_t launch_t(const Dims& d, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mp,
                     const float* lse_in, __nv_bfloat16* side, float* scores, kvm_stats* stats, cudaStream_t st,
                     const __nv_bfloat16* Ksim, float* sim_out, float* lse_out) {
    const size_t smem = 1024 + (size_t)(2 + 2 * NSTAGE) * KCH * TILE * 128 + (size_t)(2 * NSTAGE + 1) * PTILE_BYTES +
                        sizeof(Shared);
    // the shared-memory opt-in and the SM count are looked up once per device and kernel instantiation
    static std::mutex mu;
    static int sms_of[KVM_MAX_DEVICES] = {};
    cudaError_t e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if (dev < 0 || dev >= KVM_MAX_DEVICES) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!sms_of[dev]) {
            e = cudaFuncSetAttribute(score_tc_kernel<KCH, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            e = cudaFuncSetAttribute(score_tc_kernel<KCH, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
            sms_of[dev] = sms;
        }
        sms = sms_of[dev];
    }
    const int T = (d.S + TILE - 1) / TILE;
    const float scale2 = d.scale * LOG2E;
    // the schedule counts items, and the similarity warps their runs of tokens, in 32 bits
    if ((long long)d.B * d.Hq * T + sms >= (1ll << 31)) return cudaErrorInvalidValue;
    if ((long long)d.B * d.Hkv * ((d.S + SIM_RUN - 1) / SIM_RUN) + (long long)sms * 64 >= (1ll << 31)) return cudaErrorInvalidValue;
    if (!lse_in) {
        const long long items = (long long)d.B * d.Hq * T;
        const int grid = (int)(items < sms ? items : sms);
        // (the kernel begins with the dependency wait, so it may be scheduled while whatever precedes it drains)
        e = launch_dependent(score_tc_kernel<KCH, 1>, dim3(grid), dim3(NTHREADS), smem, st, mq, mk, mp, side,
                             (float*)nullptr, stats, d.B, d.Hq, d.Hkv, d.S, scale2, Ksim, scores ? (float*)nullptr : sim_out);
        if (e != cudaSuccess) return e;
    } else {
        const long long rows = (long long)d.B * d.Hq * d.S;
        lse_split_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(lse_in, side, rows, -LOG2E / scale2);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (lse_out) {                                    // the caller wants the row pass's result in the clear
        const long long rows = (long long)d.B * d.Hq * d.S;
        e = launch_dependent(side_to_lse_kernel, dim3((unsigned)((rows + 255) / 256)), dim3(256), 0, st,
                             (const __nv_bfloat16*)side, lse_out, rows, -scale2 * 0.6931471805599453f);
        if (e != cudaSuccess) return e;
    }
    if (!scores) return cudaSuccess;                  // row pass only
    const long long items = (long long)d.U * T;
    const int grid = (int)(items < sms ? items : sms);
    return launch_dependent(score_tc_kernel<KCH, 2>, dim3(grid), dim3(NTHREADS), smem, st, mq, mk, mp,
                            (__nv_bfloat16*)nullptr, scores, stats, d.B, d.Hq, d.Hkv, d.S, scale2, Ksim,
                            sim_out);
}

}  // namespace

// Bytes of scratch per query row that the tensor-core path needs (the lse side tensor).
size_t score_tc_scratch_bytes_per_row() { return (size_t)PCH * 2; }

// sim_out (nullable): when given, the spare warps of the column pass (of the row pass when scores is NULL and
// the column pass does not run) also write the neighbour-key similarities [U,S] there, so the caller needs no
// similarity kernel.  (Measured on a 32-head, 4096-token layer: 0.9 us less per call beside the column pass
// than beside the row pass; the spare warps share two of the four schedulers with the epilogue warps of two
// TMEM lane quarters, which then lag the others, and an accumulator goes back when its slowest warp is done.)
// scores may be NULL (row pass only); lse_out (nullable) receives the natural-log row log-sum-exp [B,Hq,S].
cudaError_t launch_score_tc(const Dims& d, const void* Q, const void* K, const float* lse_in, float* lse_ws,
                            float* scores, kvm_stats* stats, cudaStream_t st, float* sim_out, float* lse_out) {
    CUtensorMap mq, mk, mp;
    __nv_bfloat16* side = reinterpret_cast<__nv_bfloat16*>(lse_ws);
    if (!make_map(&mq, Q, d.B * d.Hq, d.S, d.D) || !make_map(&mk, K, d.B * d.Hkv, d.S, d.D) ||
        !make_map_side(&mp, side, d.B * d.Hq, d.S))
        return cudaErrorNotSupported;
    const __nv_bfloat16* Ks = reinterpret_cast<const __nv_bfloat16*>(K);
    return d.D == 128 ? launch_t<2>(d, mq, mk, mp, lse_in, side, scores, stats, st, Ks, sim_out, lse_out)
                      : launch_t<1>(d, mq, mk, mp, lse_in, side, scores, stats, st, Ks, sim_out, lse_out);
}

}  // namespace kvm
