// TEST INFRASTRUCTURE -- NOT A PRODUCT PATH.
//
// Plain fp64 CPU statement of KVMerger's prefill-time KV-cache compression
// (Wang, Jin, Yu, Zhang, "Model Tells You Where to Merge", arXiv 2407.08454),
// written from the paper's definitions, one step per function, in the paper's
// order.  It exists to check the CUDA library and to be timed as a CPU
// baseline.  It shares no code with the CUDA path and nothing in the library
// may call it.
//
// Inputs are fp32 arrays holding the storage-dtype values exactly (bf16 and
// fp32 both widen to fp32 without loss); all arithmetic is fp64.
// A "unit" is one (batch entry, KV head) pair; units are independent.
// Indices are 0-based.
//
// Parity pins (tests/test_oracle_*.py): every function below is pinned by
// closed forms, invariants, library routines or brute force (kvmo_prefill_attend:
// a library softmax row by row, the row-sum invariant, its last row against
// kvmo_attend and its log-sum-exp against kvmo_scores).  Parity unpinned BY THE PAPER (no
// printed example; pinned only by brute force, monotonicity and invariants):
// the budget rule in kvmo_boundaries; the per-set bandwidth of kvmo_merge's
// weight_rule 3 (a reading of Eq. 4, which is circular as printed).
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

int kvmo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Capacity and conserved-set sizes from the ratios of Section 5.1
// ("Implementation details"): C = floor(budget*S), n_r = floor(recent*S),
// n_h = floor(heavy*S).
void kvmo_sizes(int32_t S, double budget, double recent, double heavy,
                int32_t* C, int32_t* n_r, int32_t* n_h) {
    *C = (int32_t)std::floor(budget * (double)S);
    *n_r = (int32_t)std::floor(recent * (double)S);
    *n_h = (int32_t)std::floor(heavy * (double)S);
}

// Eq. 1 (causal, decoder-only) and the aggregated attention score of
// Algorithm 2 / Eq. 6: for every query head q^g of the group of KV head h,
//   s_ij = scale * <q_i, k_j>,  j <= i
//   A_ij = exp(s_ij - m_i) / l_i,  m_i = max_j s_ij,  l_i = sum_j exp(s_ij - m_i)
//   a_j  = (1/G) sum_g sum_{i >= j} A^g_ij        (GQA: mean of the G maps, Section 5.2)
// Q [B,Hq,S,D], K [B,Hkv,S,D]; scores [B,Hkv,S]; lse (nullable) [B,Hq,S] = m_i + ln l_i.
void kvmo_scores(int32_t B, int32_t Hq, int32_t Hkv, int32_t S, int32_t D, double scale,
                 const float* Q, const float* K, double* scores, double* lse) {
    const int32_t G = Hq / Hkv;
    const int64_t U = (int64_t)B * Hkv;
    for (int64_t u = 0; u < U; ++u) {
        const int64_t b = u / Hkv, h = u % Hkv;
        const float* Ku = K + (size_t)u * S * D;
        double* a = scores + (size_t)u * S;
        for (int32_t j = 0; j < S; ++j) a[j] = 0.0;
        for (int32_t g = 0; g < G; ++g) {
            const int64_t qh = b * Hq + h * G + g;
            const float* Qh = Q + (size_t)qh * S * D;
            int nthreads = 1;
#ifdef _OPENMP
            nthreads = omp_get_max_threads();
#endif
            // Column sums are accumulated per thread and added in thread order.
            std::vector<std::vector<double>> part(nthreads, std::vector<double>(S, 0.0));
#pragma omp parallel
            {
                int tid = 0;
#ifdef _OPENMP
                tid = omp_get_thread_num();
#endif
                std::vector<double> s(S);
                double* acc = part[tid].data();
#pragma omp for schedule(static, 8)
                for (int32_t i = 0; i < S; ++i) {
                    const float* q = Qh + (size_t)i * D;
                    double m = -INFINITY;
                    for (int32_t j = 0; j <= i; ++j) {
                        const float* k = Ku + (size_t)j * D;
                        double dot = 0.0;
#pragma omp simd reduction(+ : dot)
                        for (int32_t t = 0; t < D; ++t) dot += (double)q[t] * (double)k[t];
                        s[j] = scale * dot;
                        if (s[j] > m) m = s[j];
                    }
                    double l = 0.0;
                    for (int32_t j = 0; j <= i; ++j) l += std::exp(s[j] - m);
                    for (int32_t j = 0; j <= i; ++j) acc[j] += std::exp(s[j] - m) / l;
                    if (lse) lse[(size_t)qh * S + i] = m + std::log(l);
                }
            }
            for (int t = 0; t < nthreads; ++t)
                for (int32_t j = 0; j < S; ++j) a[j] += part[t][j];
        }
        for (int32_t j = 0; j < S; ++j) a[j] /= (double)G;
    }
}

// Conserved set (Section 4.1, last paragraph; Section 4.2 "recent tokens"):
// the last n_r positions, plus the n_h largest aggregated scores among the
// other positions (ties -> lower index).  keep [U,S] (0/1).
void kvmo_keep(int64_t U, int32_t S, int32_t n_r, int32_t n_h, const double* scores, uint8_t* keep) {
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < U; ++u) {
        const double* a = scores + (size_t)u * S;
        uint8_t* kp = keep + (size_t)u * S;
        const int32_t R = std::max(0, S - n_r);  // first recent position
        for (int32_t j = 0; j < S; ++j) kp[j] = (j >= R) ? 1 : 0;
        std::vector<int32_t> idx(R);
        for (int32_t j = 0; j < R; ++j) idx[j] = j;
        std::stable_sort(idx.begin(), idx.end(), [&](int32_t x, int32_t y) { return a[x] > a[y]; });
        for (int32_t t = 0; t < std::min(n_h, R); ++t) kp[idx[t]] = 1;
    }
}

// Eq. 2 restricted to the neighbour pairs Algorithm 1 consumes (|i-j| = 1):
// sim_j = <k_{j-1}, k_j> / (|k_{j-1}| |k_j|), j >= 1; 0 if a norm is 0; sim_0 = 0.
void kvmo_similarity(int64_t U, int32_t S, int32_t D, const float* K, double* sim) {
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < U; ++u) {
        const float* Ku = K + (size_t)u * S * D;
        double* c = sim + (size_t)u * S;
        c[0] = 0.0;
        for (int32_t j = 1; j < S; ++j) {
            const float* x = Ku + (size_t)(j - 1) * D;
            const float* y = Ku + (size_t)j * D;
            double xy = 0.0, xx = 0.0, yy = 0.0;
            for (int32_t t = 0; t < D; ++t) {
                xy += (double)x[t] * (double)y[t];
                xx += (double)x[t] * (double)x[t];
                yy += (double)y[t] * (double)y[t];
            }
            c[j] = (xx > 0.0 && yy > 0.0) ? xy / (std::sqrt(xx) * std::sqrt(yy)) : 0.0;
        }
    }
}

// Algorithm 1 as a boundary flag per token: token j starts a new merging set
// unless it is grouped with its left neighbour, which needs sim_j > eps
// (strict) and neither token conserved (conserved states take no part in
// merging, so each is a set of its own and ends the run on both sides).
//   hard_j = (j == 0) | keep_j | keep_{j-1};   soft_j = !hard_j & !(sim_j > eps)
// Budget rule (a reading; the paper fixes eps and lets the ratio result, and
// says the ratio can be set by adjusting the threshold): if the flags exceed
// the capacity C, the threshold is lowered for this unit just enough, i.e.
// only the (C - n_hard) soft boundaries with the smallest similarity stay
// (ties -> lower index).  b [U,S] (0/1); fired (nullable) [U].
void kvmo_boundaries(int64_t U, int32_t S, int32_t C, double eps, int32_t enforce_budget,
                     const double* sim, const uint8_t* keep, uint8_t* b, int32_t* fired) {
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < U; ++u) {
        const double* c = sim + (size_t)u * S;
        const uint8_t* kp = keep + (size_t)u * S;
        uint8_t* bu = b + (size_t)u * S;
        std::vector<int32_t> soft;
        int32_t n_hard = 0;
        for (int32_t j = 0; j < S; ++j) {
            const bool hard = (j == 0) || kp[j] || kp[j - 1];
            const bool grouped = !hard && (c[j] > eps);
            bu[j] = grouped ? 0 : 1;
            if (hard) ++n_hard;
            else if (!grouped) soft.push_back(j);
        }
        int32_t f = 0;
        if (enforce_budget && n_hard + (int32_t)soft.size() > C) {
            f = 1;
            const int32_t m = std::max(0, C - n_hard);
            std::stable_sort(soft.begin(), soft.end(), [&](int32_t x, int32_t y) { return c[x] < c[y]; });
            for (size_t t = (size_t)m; t < soft.size(); ++t) bu[soft[t]] = 0;
        }
        if (fired) fired[u] = f;
    }
}

// Layer-wise compression ratio of Section 3.2 (Figure 3(b)): the number of
// groups the set identification forms on its own -- walking the sequence and
// grouping a state with its neighbour while their similarity exceeds eps, with
// nothing conserved and no budget -- over the number of states.  ratio [U].
void kvmo_layer_ratio(int64_t U, int32_t S, double eps, const double* sim, double* ratio) {
    for (int64_t u = 0; u < U; ++u) {
        int32_t groups = 0;
        int32_t i = S - 1;                       // from the last token to the first
        while (i >= 0) {
            ++groups;
            int32_t j = i - 1;
            while (j >= 0 && sim[(size_t)u * S + j + 1] > eps) --j;   // sim_{j+1} pairs tokens j and j+1
            i = j;
        }
        ratio[u] = (double)groups / (double)S;
    }
}

// Set identification as Section 3.2 words it ("anchor" reading): starting from
// the last token, a key state gathers the consecutive states before it whose
// similarity TO IT exceeds eps; the first state that fails (or is conserved, or
// the start of the sequence) ends the group, and the walk goes on from there.
// A conserved state is a group of its own.  (Algorithm 1 compares
// neighbours instead; both readings give consecutive, disjoint, covering sets.)
//   cos(a, b) = <a,b> / (|a||b|), 0 if a norm is 0, computed in fp64.
// b [U,S] (0/1) = boundary flags (1 at the first token of every group);
// run (nullable) [U,S] = for EVERY token i, the number of consecutive
// predecessors whose similarity to k_i exceeds eps, ignoring conserved tokens
// (the quantity the walk consults at its anchors).
// run_in (nullable) [U,S]: run lengths decided elsewhere (e.g. in fp32 by the code under test); when given,
// the walk consults them instead of evaluating cosines, so that only integer logic is left.
void kvmo_boundaries_anchor(int64_t U, int32_t S, int32_t D, double eps, const float* K, const uint8_t* keep,
                            uint8_t* b, int32_t* run, const int32_t* run_in) {
#pragma omp parallel for schedule(static, 1)
    for (int64_t u = 0; u < U; ++u) {
        const float* Ku = K + (size_t)u * S * D;
        const uint8_t* kp = keep + (size_t)u * S;
        auto cosine = [&](int32_t i, int32_t j) {
            double dot = 0.0, ni = 0.0, nj = 0.0;
            for (int32_t t = 0; t < D; ++t) {
                const double a = Ku[(size_t)i * D + t], c = Ku[(size_t)j * D + t];
                dot += a * c; ni += a * a; nj += c * c;
            }
            return (ni > 0.0 && nj > 0.0) ? dot / (std::sqrt(ni) * std::sqrt(nj)) : 0.0;
        };
        if (run)
            for (int32_t i = 0; i < S; ++i) {
                int32_t j = i - 1;
                while (j >= 0 && cosine(i, j) > eps) --j;
                run[(size_t)u * S + i] = i - 1 - j;
            }
        for (int32_t j = 0; j < S; ++j) b[(size_t)u * S + j] = 0;
        int32_t i = S - 1;
        while (i >= 0) {
            int32_t j = i - 1;
            if (!kp[i]) {
                if (run_in) {
                    int32_t left = run_in[(size_t)u * S + i];
                    while (j >= 0 && !kp[j] && left > 0) { --j; --left; }
                } else {
                    while (j >= 0 && !kp[j] && cosine(i, j) > eps) --j;
                }
            }
            b[(size_t)u * S + j + 1] = 1;       // the group is tokens j+1 .. i
            i = j;
        }
    }
}

// Definition 4.1's partition: consecutive, disjoint sets covering the sequence.
// set_id_j = (number of flags at positions <= j) - 1; set s = [set_start[s], set_start[s+1]).
// set_id [U,S]; set_start [U,cap+1]; out_len [U].  Entries past out_len are untouched.
void kvmo_sets(int64_t U, int32_t S, int32_t cap, const uint8_t* b,
               int32_t* set_id, int32_t* set_start, int32_t* out_len) {
    for (int64_t u = 0; u < U; ++u) {
        const uint8_t* bu = b + (size_t)u * S;
        int32_t n = 0;
        for (int32_t j = 0; j < S; ++j) {
            if (bu[j]) {
                if (n <= cap) set_start[(size_t)u * (cap + 1) + n] = j;
                ++n;
            }
            set_id[(size_t)u * S + j] = n - 1;
        }
        if (n <= cap) set_start[(size_t)u * (cap + 1) + n] = S;
        out_len[u] = n;
    }
}

// Algorithm 2, pivot step (Eq. 6): p_s = argmax_{j in set s} a_j, ties -> lowest j.
void kvmo_pivots(int64_t U, int32_t S, int32_t cap, const double* scores,
                 const int32_t* set_start, const int32_t* out_len, int32_t* pivot) {
    for (int64_t u = 0; u < U; ++u) {
        const double* a = scores + (size_t)u * S;
        const int32_t* st = set_start + (size_t)u * (cap + 1);
        for (int32_t s = 0; s < out_len[u]; ++s) {
            int32_t p = st[s];
            for (int32_t j = st[s] + 1; j < st[s + 1]; ++j)
                if (a[j] > a[p]) p = j;
            pivot[(size_t)u * cap + s] = p;
        }
    }
}

// Pivot of the average-weighted baseline (Section 4.2, first experiment): the
// state with the maximum index within each merging set.
void kvmo_pivots_last(int64_t U, int32_t cap, const int32_t* set_start, const int32_t* out_len, int32_t* pivot) {
    for (int64_t u = 0; u < U; ++u) {
        const int32_t* st = set_start + (size_t)u * (cap + 1);
        for (int32_t s = 0; s < out_len[u]; ++s) pivot[(size_t)u * cap + s] = st[s + 1] - 1;
    }
}

// Algorithm 2, weights and merge (Eq. 4, Eq. 5, Definition 4.2), fixed sigma:
//   g_j = exp(-|k_p - k_j|^2 / (2 sigma^2)),  w_j = g_j / sum_{t in set} g_t   (g_p = 1)
//   K*_s = sum_j w_j k_j;   V*_s = (|set| if scale_v else 1) * sum_j w_j v_j
// weight_rule 0 is the paper's method.  1 = average-weighted merging (Section
// 4.2's baseline): g_j = 1, so w_j = 1/|set|.  2 = the sigma -> 0 limit named
// after Eq. 5: nothing but the pivot survives, g_j = [j == p].
// 3 = a bandwidth per merging set (PARITY UNPINNED: Eq. 4 defines sigma through
// the weights that depend on it; this is one non-circular reading, not the
// paper's statement): sigma_s^2 = mean_{j in set} |k_p - k_j|^2 / 2, i.e.
// g_j = exp(-|k_p - k_j|^2 / mean_t |k_p - k_t|^2), and g_j = 1 when that mean is 0.
// K_out, V_out [U,cap,D] fp64 (rows >= out_len untouched); weights (nullable) [U,S].
void kvmo_merge(int64_t U, int32_t S, int32_t D, int32_t cap, double sigma, int32_t scale_v, int32_t weight_rule,
                const float* K, const float* V, const int32_t* set_start, const int32_t* pivot,
                const int32_t* out_len, double* K_out, double* V_out, double* weights) {
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < U; ++u) {
        const float* Ku = K + (size_t)u * S * D;
        const float* Vu = V + (size_t)u * S * D;
        const int32_t* st = set_start + (size_t)u * (cap + 1);
        std::vector<double> g(S);
        for (int32_t s = 0; s < out_len[u]; ++s) {
            const int32_t lo = st[s], hi = st[s + 1], p = pivot[(size_t)u * cap + s];
            const float* kp = Ku + (size_t)p * D;
            double gsum = 0.0, two_sigma2 = 2.0 * sigma * sigma;
            if (weight_rule == 3) {
                double total = 0.0;
                for (int32_t j = lo; j < hi; ++j) {
                    const float* kj = Ku + (size_t)j * D;
                    for (int32_t t = 0; t < D; ++t) {
                        const double df = (double)kp[t] - (double)kj[t];
                        total += df * df;
                    }
                }
                two_sigma2 = total / (double)(hi - lo);      // 2 sigma_s^2 = mean squared distance to the pivot
            }
            for (int32_t j = lo; j < hi; ++j) {
                const float* kj = Ku + (size_t)j * D;
                double d2 = 0.0;
                for (int32_t t = 0; t < D; ++t) {
                    const double df = (double)kp[t] - (double)kj[t];
                    d2 += df * df;
                }
                if (weight_rule == 1) g[j] = 1.0;
                else if (weight_rule == 2) g[j] = (j == p) ? 1.0 : 0.0;
                else if (weight_rule == 3 && !(two_sigma2 > 0.0)) g[j] = 1.0;
                else g[j] = std::exp(-d2 / two_sigma2);
                gsum += g[j];
            }
            double* ko = K_out + ((size_t)u * cap + s) * D;
            double* vo = V_out + ((size_t)u * cap + s) * D;
            for (int32_t t = 0; t < D; ++t) { ko[t] = 0.0; vo[t] = 0.0; }
            const double vmul = scale_v ? (double)(hi - lo) : 1.0;
            for (int32_t j = lo; j < hi; ++j) {
                const double w = g[j] / gsum;
                if (weights) weights[(size_t)u * S + j] = w;
                const float* kj = Ku + (size_t)j * D;
                const float* vj = Vu + (size_t)j * D;
                for (int32_t t = 0; t < D; ++t) {
                    ko[t] += w * (double)kj[t];
                    vo[t] += vmul * w * (double)vj[t];
                }
            }
        }
    }
}

// Eviction for comparison (Section 2.2; the heavy-hitter scheme the paper
// measures against in Section 4.2 and Section 5): only the conserved tokens --
// the n_h largest aggregated scores and the n_r most recent -- stay, unchanged
// and in token order; everything else is dropped.  out_pos [U,cap] = the kept
// token indices; K_out, V_out [U,cap,D]; out_len [U] = number kept (<= cap required).
void kvmo_evict(int64_t U, int32_t S, int32_t D, int32_t cap, const uint8_t* keep, const float* K, const float* V,
                int32_t* out_len, int32_t* out_pos, double* K_out, double* V_out) {
    for (int64_t u = 0; u < U; ++u) {
        int32_t n = 0;
        for (int32_t j = 0; j < S; ++j) {
            if (!keep[(size_t)u * S + j]) continue;
            if (n < cap) {
                out_pos[(size_t)u * cap + n] = j;
                for (int32_t t = 0; t < D; ++t) {
                    K_out[((size_t)u * cap + n) * D + t] = (double)K[((size_t)u * S + j) * D + t];
                    V_out[((size_t)u * cap + n) * D + t] = (double)V[((size_t)u * S + j) * D + t];
                }
            }
            ++n;
        }
        out_len[u] = n;
    }
}

// One decode step of Eq. 1 over a cache that may be compressed: for query head
// h of batch entry b (KV head h / G), with the first len[u] of `rows` cache rows,
//   A_t = softmax(scale * q_t K^T),   O_t = A_t V.
// q [B,Hq,D]; K, V [B,Hkv,rows,D]; len [B*Hkv] (nullable: all rows); out [B,Hq,D].
// No rows -> O_t = 0.
void kvmo_attend(int32_t B, int32_t Hq, int32_t Hkv, int32_t rows, int32_t D, double scale,
                 const float* q, const float* K, const float* V, const int32_t* len, double* out) {
    const int32_t G = Hq / Hkv;
    for (int32_t b = 0; b < B; ++b)
        for (int32_t h = 0; h < Hq; ++h) {
            const int64_t u = (int64_t)b * Hkv + h / G;
            const int32_t n = len ? len[u] : rows;
            const float* qt = q + ((size_t)b * Hq + h) * D;
            const float* Ku = K + (size_t)u * rows * D;
            const float* Vu = V + (size_t)u * rows * D;
            double* o = out + ((size_t)b * Hq + h) * D;
            for (int32_t t = 0; t < D; ++t) o[t] = 0.0;
            if (n <= 0) continue;
            std::vector<double> s(n);
            double m = -INFINITY;
            for (int32_t j = 0; j < n; ++j) {
                double dot = 0.0;
                for (int32_t t = 0; t < D; ++t) dot += (double)qt[t] * (double)Ku[(size_t)j * D + t];
                s[j] = scale * dot;
                m = std::max(m, s[j]);
            }
            double l = 0.0;
            for (int32_t j = 0; j < n; ++j) { s[j] = std::exp(s[j] - m); l += s[j]; }
            for (int32_t j = 0; j < n; ++j)
                for (int32_t t = 0; t < D; ++t) o[t] += (s[j] / l) * (double)Vu[(size_t)j * D + t];
        }
}

// Eq. 1 for every position of the prompt at once (the prefill): for query head h (KV head h / G) and
// position i, O_i = sum_{j <= i} softmax_j(scale * <q_i, k_j>) v_j over the causal prefix, and the row's
// log-sum-exp lse_i = ln sum_{j <= i} exp(scale * <q_i, k_j>) (the quantity kvmo_scores also returns).
// Q [B,Hq,S,D], K/V [B,Hkv,S,D]; out [B,Hq,S,D]; lse (nullable) [B,Hq,S].
void kvmo_prefill_attend(int32_t B, int32_t Hq, int32_t Hkv, int32_t S, int32_t D, double scale, const float* Q,
                         const float* K, const float* V, double* out, double* lse) {
    const int32_t G = Hq / Hkv;
    for (int64_t qh = 0; qh < (int64_t)B * Hq; ++qh) {
        const int64_t b = qh / Hq, h = qh % Hq;
        const int64_t u = b * Hkv + h / G;
        const float* Qh = Q + (size_t)qh * S * D;
        const float* Ku = K + (size_t)u * S * D;
        const float* Vu = V + (size_t)u * S * D;
#pragma omp parallel for schedule(static, 8)
        for (int32_t i = 0; i < S; ++i) {
            std::vector<double> s(i + 1);
            double m = -INFINITY;
            for (int32_t j = 0; j <= i; ++j) {
                double dot = 0.0;
                for (int32_t t = 0; t < D; ++t) dot += (double)Qh[(size_t)i * D + t] * (double)Ku[(size_t)j * D + t];
                s[j] = scale * dot;
                m = std::max(m, s[j]);
            }
            double l = 0.0;
            for (int32_t j = 0; j <= i; ++j) { s[j] = std::exp(s[j] - m); l += s[j]; }
            double* o = out + ((size_t)qh * S + i) * D;
            for (int32_t t = 0; t < D; ++t) o[t] = 0.0;
            for (int32_t j = 0; j <= i; ++j)
                for (int32_t t = 0; t < D; ++t) o[t] += (s[j] / l) * (double)Vu[(size_t)j * D + t];
            if (lse) lse[(size_t)qh * S + i] = m + std::log(l);
        }
    }
}

// Definition 2.1's criterion |O_t - O_t*|, read as the Euclidean norm per
// attention head; ref = |O_t| for a relative figure.  O, O_star [n,D]; err, ref [n].
void kvmo_perturbation(int64_t n, int32_t D, const double* O, const double* O_star, double* err, double* ref) {
    for (int64_t i = 0; i < n; ++i) {
        double e = 0.0, r = 0.0;
        for (int32_t t = 0; t < D; ++t) {
            const double d = O[(size_t)i * D + t] - O_star[(size_t)i * D + t];
            e += d * d;
            r += O[(size_t)i * D + t] * O[(size_t)i * D + t];
        }
        err[i] = std::sqrt(e);
        ref[i] = std::sqrt(r);
    }
}

// The whole path for one layer, steps in the paper's order.  All outputs are
// caller-allocated; cap = C when enforce_budget, else S.
// Variants (all 0 = the paper's method): pivot_rule 1 = last index of the set,
// 2 = arg-max of pivot_key [U,S] (iid random numbers give the random-pivot
// ablation of Section 5.3); weight_rule as in kvmo_merge; set_rule 2 = the anchor
// reading of the set identification (kvmo_boundaries_anchor); set_rule 1 = eviction
// (kvmo_evict; set_id is -1 for dropped tokens, set_start[s] = the kept token).
void kvmo_compress(int32_t B, int32_t Hq, int32_t Hkv, int32_t S, int32_t D, double scale,
                   int32_t cap, int32_t n_r, int32_t n_h, double eps, double sigma,
                   int32_t scale_v, int32_t enforce_budget,
                   int32_t pivot_rule, int32_t weight_rule, int32_t set_rule, const double* pivot_key,
                   const float* Q, const float* K, const float* V,
                   double* scores, uint8_t* keep, double* sim, uint8_t* b,
                   int32_t* set_id, int32_t* set_start, int32_t* out_len, int32_t* pivot,
                   double* K_out, double* V_out) {
    const int64_t U = (int64_t)B * Hkv;
    kvmo_scores(B, Hq, Hkv, S, D, scale, Q, K, scores, nullptr);
    kvmo_keep(U, S, n_r, n_h, scores, keep);
    kvmo_similarity(U, S, D, K, sim);
    if (set_rule == 1) {
        kvmo_evict(U, S, D, cap, keep, K, V, out_len, pivot, K_out, V_out);
        for (int64_t u = 0; u < U; ++u) {
            int32_t n = 0;
            for (int32_t j = 0; j < S; ++j) {
                const bool k = keep[(size_t)u * S + j] != 0;
                b[(size_t)u * S + j] = k;
                set_id[(size_t)u * S + j] = k ? n : -1;
                if (k && n <= cap) set_start[(size_t)u * (cap + 1) + n] = j;
                n += k;
            }
            if (n <= cap) set_start[(size_t)u * (cap + 1) + n] = S;
        }
        return;
    }
    if (set_rule == 2) kvmo_boundaries_anchor(U, S, D, eps, K, keep, b, nullptr, nullptr);   // no budget rule: cap must be S
    else kvmo_boundaries(U, S, cap, eps, enforce_budget, sim, keep, b, nullptr);
    kvmo_sets(U, S, cap, b, set_id, set_start, out_len);
    if (pivot_rule == 1) kvmo_pivots_last(U, cap, set_start, out_len, pivot);
    else kvmo_pivots(U, S, cap, pivot_rule == 2 ? pivot_key : scores, set_start, out_len, pivot);
    kvmo_merge(U, S, D, cap, sigma, scale_v, weight_rule, K, V, set_start, pivot, out_len, K_out, V_out, nullptr);
}

}  // extern "C"
