// C ABI of the kvm library: host-side validation, workspace carving, dispatch.
// All checks run before anything is enqueued; nothing here allocates device memory or synchronises.
#include <math.h>
#include <string.h>

#include <mutex>

#include "common.cuh"

namespace kvm {
namespace {

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

int derive(const kvm_params* p, Dims& d) {
    if (!p) return KVM_E_NULL;
    if (p->dtype != KVM_BF16 && p->dtype != KVM_F32) return KVM_E_DTYPE;
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->seq < 1) return KVM_E_SHAPE;
    if (p->n_q_heads % p->n_kv_heads != 0) return KVM_E_SHAPE;
    if (p->head_dim != 64 && p->head_dim != 128) return KVM_E_SHAPE;
    if (p->seq > KVM_MAX_SEQ) return KVM_E_SHAPE;
    if ((long long)p->batch * p->n_q_heads > 65535) return KVM_E_SHAPE;
    if (!(p->budget > 0.f && p->budget <= 1.f)) return KVM_E_PARAM;
    if (!isfinite(p->sim_threshold)) return KVM_E_PARAM;
    if (!isfinite(p->softmax_scale)) return KVM_E_PARAM;
    if (p->causal != 1) return KVM_E_UNSUPPORTED;
    const bool half_budget = p->budget >= 0.425f;
    const float recent = p->recent_ratio < 0.f ? (half_budget ? 0.17f : 0.08f) : p->recent_ratio;
    const float heavy = p->heavy_ratio < 0.f ? (half_budget ? 0.12f : 0.02f) : p->heavy_ratio;
    if (!(recent >= 0.f && recent <= 1.f) || !(heavy >= 0.f && heavy <= 1.f)) return KVM_E_PARAM;
    d.B = p->batch; d.Hq = p->n_q_heads; d.Hkv = p->n_kv_heads; d.G = d.Hq / d.Hkv;
    d.S = p->seq; d.D = p->head_dim; d.U = d.B * d.Hkv; d.dtype = p->dtype;
    const int C = (int)floor((double)p->budget * (double)d.S);
    d.n_r = (int)floor((double)recent * (double)d.S);
    d.n_h = (int)floor((double)heavy * (double)d.S);
    d.enforce = p->enforce_budget ? 1 : 0;
    d.cap = d.enforce ? C : d.S;
    if (p->pivot_rule < KVM_PIVOT_MAX_SCORE || p->pivot_rule > KVM_PIVOT_KEY) return KVM_E_PARAM;
    if (p->weight_rule < KVM_WEIGHT_GAUSSIAN || p->weight_rule > KVM_WEIGHT_SET_SIGMA) return KVM_E_PARAM;
    if (p->set_rule < KVM_SETS_ADJACENT || p->set_rule > KVM_SETS_ANCHOR) return KVM_E_PARAM;
    if (p->set_rule == KVM_SETS_ANCHOR && (p->enforce_budget || p->seq > KVM_ANCHOR_MAX_SEQ)) return KVM_E_UNSUPPORTED;
    d.pivot_rule = p->pivot_rule; d.weight_rule = p->weight_rule; d.set_rule = p->set_rule;
    d.pivot_key = p->pivot_key;
    if (p->set_rule != KVM_SETS_CONSERVED_ONLY && p->weight_rule == KVM_WEIGHT_GAUSSIAN &&
        (!(p->sigma > 0.f) || !isfinite(p->sigma)))
        return KVM_E_PARAM;
    if (d.set_rule == KVM_SETS_CONSERVED_ONLY) {
        d.pivot_rule = KVM_PIVOT_MAX_SCORE; d.weight_rule = KVM_WEIGHT_PIVOT_ONLY; d.pivot_key = nullptr;
        if ((long long)d.cap < (long long)d.n_r + d.n_h) return KVM_E_PARAM;   // the kept tokens must fit
    } else {
        if (d.pivot_rule == KVM_PIVOT_KEY && !d.pivot_key) return KVM_E_NULL;
        // (pivot_key is read with scalar loads: no alignment beyond a float's is asked of it)
        if (d.pivot_rule == KVM_PIVOT_KEY && ((uintptr_t)d.pivot_key & 3u)) return KVM_E_ALIGN;
        // the forced cuts alone (first token, recent window, each heavy hitter and its right neighbour) must fit
        if (d.enforce && (long long)d.cap < 1LL + d.n_r + 2LL * d.n_h) return KVM_E_PARAM;
    }
    if (d.cap < 1) return KVM_E_PARAM;
    d.scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)d.D);
    d.eps = p->sim_threshold;
    d.sigma = p->sigma;
    d.scale_v = p->scale_v_by_set_size ? 1 : 0;
    return KVM_OK;
}

inline size_t score_row_bytes(const Dims& d) {
    return d.dtype == KVM_BF16 ? score_tc_scratch_bytes_per_row() : sizeof(float);
}

struct Workspace {
    float* lse;         // row-pass output: [B,Hq,S] fp32 (fp32 path) or [B,Hq,S,16] bf16 side tensor (bf16 path)
    float* scores;      // [U,S]
    float* sim;         // [U,S]
    int32_t* set_start; // [U,cap+1]
    int32_t* set_id;    // [U,S]
    float* merge_part;  // partial sums of sets that cross token tiles
    float* attend_part; // per-chunk online-softmax states of the decode-step attention
    size_t bytes;
};

Workspace carve(const Dims& d, void* base) {
    Workspace w;
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off += align_up(n); return (char*)base + o; };
    w.lse = (float*)take((size_t)d.B * d.Hq * d.S * score_row_bytes(d));
    w.scores = (float*)take((size_t)d.U * d.S * sizeof(float));
    w.sim = (float*)take((size_t)d.U * d.S * sizeof(float));
    w.set_start = (int32_t*)take((size_t)d.U * (d.cap + 1) * sizeof(int32_t));
    w.set_id = (int32_t*)take((size_t)d.U * d.S * sizeof(int32_t));
    w.merge_part = (float*)take(merge_scratch_floats(d) * sizeof(float));
    w.attend_part = (float*)take(attend_scratch_floats(d) * sizeof(float));
    w.bytes = off;
    return w;
}

inline bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

int check_ws(const Dims& d, void* ws, size_t ws_bytes, Workspace& w) {
    if (!ws) return KVM_E_WORKSPACE;
    if (misaligned(ws)) return KVM_E_ALIGN;
    w = carve(d, ws);
    if (ws_bytes < w.bytes) return KVM_E_WORKSPACE;
    return KVM_OK;
}

// sim_out (nullable): where the neighbour-key similarities are wanted.  *sim_done tells whether the score
// step produced them on the side (bf16 path) or the caller still has to launch the similarity kernel.
cudaError_t run_score(const Dims& d, const void* Q, const void* K, const float* lse_in, float* scores,
                      const Workspace& w, kvm_stats* stats, cudaStream_t st, float* sim_out = nullptr,
                      bool* sim_done = nullptr) {
    // bf16: tensor cores (tcgen05); fp32: plain FMA, since tensor-core input rounding cannot hold the score tolerance
    if (d.dtype == KVM_BF16) {
        if (sim_done) *sim_done = sim_out != nullptr;
        return launch_score_tc(d, Q, K, lse_in, w.lse, scores, stats, st, sim_out);
    }
    if (sim_done) *sim_done = false;
    return launch_score_simt(d, Q, K, lse_in, w.lse, scores, st);
}

}  // namespace
}  // namespace kvm

using namespace kvm;

extern "C" {

int kvm_version(void) { return KVM_VERSION; }

const char* kvm_status_string(int s) {
    switch (s) {
        case KVM_OK: return "ok";
        case KVM_E_NULL: return "a required pointer is NULL";
        case KVM_E_SHAPE: return "unsupported shape";
        case KVM_E_DTYPE: return "unknown dtype";
        case KVM_E_PARAM: return "parameter out of range or capacity too small for the conserved tokens";
        case KVM_E_ALIGN: return "pointer not 16-byte aligned";
        case KVM_E_WORKSPACE: return "workspace missing or too small";
        case KVM_E_UNSUPPORTED: return "unsupported request";
        case KVM_E_CUDA: return "CUDA runtime error";
        case KVM_E_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
        case KVM_E_STATIC_LIMIT:
            return "batch * n_q_heads * seq exceeds the built-in scratch of kvm_score_static (KVM_STATIC_SCORE_ROWS rows in fp32, an eighth of that in bf16)";
        default: return "unknown status";
    }
}

int kvm_sizes(const kvm_params* p, int32_t* cap, int32_t* n_recent, int32_t* n_heavy) {
    Dims d;
    const int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (cap) *cap = d.cap;
    if (n_recent) *n_recent = d.n_r;
    if (n_heavy) *n_heavy = d.n_h;
    return KVM_OK;
}

int kvm_workspace_bytes(const kvm_params* p, size_t* bytes) {
    Dims d;
    const int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!bytes) return KVM_E_NULL;
    *bytes = carve(d, nullptr).bytes;
    return KVM_OK;
}

int kvm_score(const kvm_params* p, const void* Q, const void* K, const float* lse_in, float* scores, void* ws,
              size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!Q || !K || !scores) return KVM_E_NULL;
    if (misaligned(Q) || misaligned(K) || misaligned(scores) || (lse_in && misaligned(lse_in))) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    return run_score(d, Q, K, lse_in, scores, w, nullptr, (cudaStream_t)cuda_stream) == cudaSuccess ? KVM_OK
                                                                                                    : KVM_E_CUDA;
}

int kvm_row_lse(const kvm_params* p, const void* Q, const void* K, float* lse_out, void* ws, size_t ws_bytes,
                void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!Q || !K || !lse_out) return KVM_E_NULL;
    if (misaligned(Q) || misaligned(K) || misaligned(lse_out)) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (d.dtype == KVM_BF16)
        return launch_score_tc(d, Q, K, nullptr, w.lse, nullptr, nullptr, st, nullptr, lse_out) == cudaSuccess
                   ? KVM_OK
                   : KVM_E_CUDA;
    // fp32 path: its row pass leaves the natural-log lse in the workspace as it is
    if (launch_score_simt(d, Q, K, nullptr, w.lse, nullptr, st) != cudaSuccess) return KVM_E_CUDA;
    return cudaMemcpyAsync(lse_out, w.lse, (size_t)d.B * d.Hq * d.S * sizeof(float), cudaMemcpyDeviceToDevice, st) ==
                   cudaSuccess
               ? KVM_OK
               : KVM_E_CUDA;
}

int kvm_segment(const kvm_params* p, const void* K, const float* scores, int32_t* set_id, int32_t* set_start,
                int32_t* pivot, int32_t* out_len, float* sim_out, kvm_stats* stats, void* ws, size_t ws_bytes,
                void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!K || !scores || !set_start || !pivot || !out_len) return KVM_E_NULL;
    if (misaligned(K) || misaligned(scores)) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* sim = sim_out ? sim_out : w.sim;
    if (d.set_rule == KVM_SETS_ANCHOR) {
        // (the workspace's set-id region is free until the segment kernel writes it: scratch for the key norms)
        if (launch_anchor_runs(d, K, sim, (float*)w.set_id, st) != cudaSuccess) return KVM_E_CUDA;
    } else if (d.set_rule == KVM_SETS_ADJACENT || sim_out) {
        if (launch_similarity(d, K, sim, st) != cudaSuccess) return KVM_E_CUDA;
    }
    if (launch_segment(d, scores, sim, set_id, set_start, pivot, out_len, stats, st) != cudaSuccess)
        return KVM_E_CUDA;
    return KVM_OK;
}

int kvm_layer_ratio(const kvm_params* p, const void* K, float* ratio, float* sim_out, void* ws, size_t ws_bytes,
                    void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!K || !ratio) return KVM_E_NULL;
    if (misaligned(K)) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* sim = sim_out ? sim_out : w.sim;
    if (launch_similarity(d, K, sim, st) != cudaSuccess) return KVM_E_CUDA;
    return launch_set_ratio(d, sim, ratio, st) == cudaSuccess ? KVM_OK : KVM_E_CUDA;
}

int kvm_prefill_attend(const kvm_params* p, const void* Q, const void* K, const void* V, void* O, float* lse,
                       kvm_stats* stats, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (d.dtype != KVM_BF16) return KVM_E_UNSUPPORTED;
    if (!Q || !K || !V || !O || !lse) return KVM_E_NULL;
    if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return KVM_E_ALIGN;
    return launch_prefill_attend(d, Q, K, V, O, lse, stats, (cudaStream_t)cuda_stream) == cudaSuccess ? KVM_OK
                                                                                                     : KVM_E_CUDA;
}

int kvm_attend(const kvm_params* p, const void* q, const void* K, const void* V, int32_t rows, const int32_t* len,
               float* out, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!q || !K || !V || !out) return KVM_E_NULL;
    if (rows < 1 || rows > d.S) return KVM_E_SHAPE;
    if (misaligned(q) || misaligned(K) || misaligned(V) || misaligned(out)) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    return launch_attend(d, q, K, V, rows, len, out, w.attend_part, (cudaStream_t)cuda_stream) == cudaSuccess
               ? KVM_OK
               : KVM_E_CUDA;
}

int kvm_output_perturbation(const kvm_params* p, const void* q, const void* K, const void* V, const void* K_c,
                            const void* V_c, const int32_t* len_c, float* out_full, float* out_comp, float* err,
                            float* ref, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!q || !K || !V || !K_c || !V_c || !len_c || !out_full || !out_comp || !err || !ref) return KVM_E_NULL;
    if (misaligned(q) || misaligned(K) || misaligned(V) || misaligned(K_c) || misaligned(V_c) ||
        misaligned(out_full) || misaligned(out_comp))
        return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (launch_attend(d, q, K, V, d.S, nullptr, out_full, w.attend_part, st) != cudaSuccess) return KVM_E_CUDA;
    if (launch_attend(d, q, K_c, V_c, d.cap, len_c, out_comp, w.attend_part, st) != cudaSuccess) return KVM_E_CUDA;
    return launch_perturbation(d, out_full, out_comp, err, ref, st) == cudaSuccess ? KVM_OK : KVM_E_CUDA;
}

int kvm_merge_compact(const kvm_params* p, const void* K, const void* V, const int32_t* set_start,
                      const int32_t* pivot, const int32_t* out_len, void* K_out, void* V_out, int32_t* out_size,
                      void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!K || !V || !set_start || !pivot || !out_len || !K_out || !V_out) return KVM_E_NULL;
    if (misaligned(K) || misaligned(V) || misaligned(K_out) || misaligned(V_out)) return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (d.weight_rule == KVM_WEIGHT_PIVOT_ONLY)
        return launch_gather(d, K, V, set_start, pivot, out_len, K_out, V_out, out_size, st) == cudaSuccess
                   ? KVM_OK
                   : KVM_E_CUDA;
    if (launch_token_sets(d, set_start, out_len, w.set_id, st) != cudaSuccess) return KVM_E_CUDA;
    // (the similarity and score regions of the workspace are free here: scratch for the per-set bandwidths)
    return launch_merge(d, K, V, set_start, pivot, w.set_id, out_len, K_out, V_out, out_size, w.merge_part, w.sim,
                        w.scores, nullptr, st) ==
                   cudaSuccess
               ? KVM_OK
               : KVM_E_CUDA;
}

int kvm_compress(const kvm_params* p, const void* Q, const void* K, const void* V, void* K_out, void* V_out,
                 int32_t* out_len, int32_t* out_pos, float* scores_out, kvm_stats* stats, void* ws,
                 size_t ws_bytes, void* cuda_stream) {
    return kvm_compress_with_lse(p, Q, K, V, nullptr, K_out, V_out, out_len, out_pos, scores_out, stats, ws,
                                 ws_bytes, cuda_stream);
}

int kvm_compress_with_lse(const kvm_params* p, const void* Q, const void* K, const void* V, const float* lse_in,
                          void* K_out, void* V_out, int32_t* out_len, int32_t* out_pos, float* scores_out,
                          kvm_stats* stats, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!Q || !K || !V || !K_out || !V_out || !out_len || !out_pos) return KVM_E_NULL;
    if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(K_out) || misaligned(V_out) ||
        (scores_out && misaligned(scores_out)) || (lse_in && misaligned(lse_in)))
        return KVM_E_ALIGN;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* scores = scores_out ? scores_out : w.scores;
    const bool want_sim = d.set_rule == KVM_SETS_ADJACENT;
    bool sim_done = false;
    if (run_score(d, Q, K, lse_in, scores, w, stats, st, want_sim ? w.sim : nullptr, &sim_done) != cudaSuccess)
        return KVM_E_CUDA;
    if (want_sim && !sim_done)
        if (launch_similarity(d, K, w.sim, st) != cudaSuccess) return KVM_E_CUDA;
    if (d.set_rule == KVM_SETS_ANCHOR)
        if (launch_anchor_runs(d, K, w.sim, (float*)w.set_id, st) != cudaSuccess) return KVM_E_CUDA;
    if (launch_segment(d, scores, w.sim, w.set_id, w.set_start, out_pos, out_len, stats, st) != cudaSuccess)
        return KVM_E_CUDA;
    if (d.weight_rule == KVM_WEIGHT_PIVOT_ONLY)
        return launch_gather(d, K, V, w.set_start, out_pos, out_len, K_out, V_out, nullptr, st) == cudaSuccess
                   ? KVM_OK
                   : KVM_E_CUDA;
    if (launch_merge(d, K, V, w.set_start, out_pos, w.set_id, out_len, K_out, V_out, nullptr, w.merge_part, w.sim,
                     w.scores, stats, st) !=
        cudaSuccess)
        return KVM_E_CUDA;
    return KVM_OK;
}

int kvm_compress_layers(const kvm_params* p, int32_t n_layers, const float* sim_thresholds, const void* const* Q,
                        const void* const* K, const void* const* V, void* const* K_out, void* const* V_out,
                        int32_t* const* out_len, int32_t* const* out_pos, kvm_stats* stats, void* ws,
                        size_t ws_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (n_layers < 1) return KVM_E_SHAPE;
    if (!Q || !K || !V || !K_out || !V_out || !out_len || !out_pos) return KVM_E_NULL;
    Workspace w;
    if ((rc = check_ws(d, ws, ws_bytes, w)) != KVM_OK) return rc;
    for (int32_t l = 0; l < n_layers; ++l) {       // everything is checked before the first layer is enqueued
        if (!Q[l] || !K[l] || !V[l] || !K_out[l] || !V_out[l] || !out_len[l] || !out_pos[l]) return KVM_E_NULL;
        if (misaligned(Q[l]) || misaligned(K[l]) || misaligned(V[l]) || misaligned(K_out[l]) || misaligned(V_out[l]))
            return KVM_E_ALIGN;
        if (sim_thresholds && !isfinite(sim_thresholds[l])) return KVM_E_PARAM;
    }
    for (int32_t l = 0; l < n_layers; ++l) {
        kvm_params pl = *p;
        if (sim_thresholds) pl.sim_threshold = sim_thresholds[l];
        rc = kvm_compress(&pl, Q[l], K[l], V[l], K_out[l], V_out[l], out_len[l], out_pos[l], nullptr, stats, ws,
                          ws_bytes, cuda_stream);
        if (rc != KVM_OK) return rc;
    }
    return KVM_OK;
}

int kvm_host_staging_bytes(const kvm_params* p, size_t* bytes) {
    Dims d;
    const int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!bytes) return KVM_E_NULL;
    const size_t e = d.dtype == KVM_BF16 ? 2 : 4;
    size_t off = 0;
    off += align_up((size_t)d.B * d.Hq * d.S * d.D * e);        // Q
    off += 2 * align_up((size_t)d.U * d.S * d.D * e);           // K, V
    off += 2 * align_up((size_t)d.U * d.cap * d.D * e);         // K_out, V_out
    off += align_up((size_t)d.U * sizeof(int32_t));             // out_len
    off += align_up((size_t)d.U * d.cap * sizeof(int32_t));     // out_pos
    off += carve(d, nullptr).bytes;
    *bytes = off;
    return KVM_OK;
}

// Streams and events of kvm_compress_host's copy/compute pipeline: created once per device on first use,
// kept until the process exits.
namespace {

constexpr int kHostChunksMax = 4;     // measured on a C1 layer: 2 groups 2.34 ms, 3 2.25, 4 2.23, 6 2.24, 8 2.29
constexpr int kPipeDevices = 64;

struct HostPipe {
    bool ready = false;
    cudaStream_t compute = nullptr, d2h = nullptr;
    cudaEvent_t start = nullptr, end = nullptr, h2d[kHostChunksMax] = {}, done[kHostChunksMax] = {};
};
HostPipe g_pipe[kPipeDevices];
std::mutex g_pipe_mu;      // held while a call enqueues: calls on one device share the events

HostPipe* host_pipe_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kPipeDevices) return nullptr;
    HostPipe& hp = g_pipe[dev];
    if (hp.ready) return &hp;
    bool ok = cudaStreamCreateWithFlags(&hp.compute, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.end, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kHostChunksMax; ++i)
        ok = cudaEventCreateWithFlags(&hp.h2d[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    hp.ready = true;
    return &hp;
}

}  // namespace

int kvm_compress_host(const kvm_params* p, const void* Q, const void* K, const void* V, void* K_out, void* V_out,
                      int32_t* out_len, int32_t* out_pos, void* dev, size_t dev_bytes, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!Q || !K || !V || !K_out || !V_out || !out_len || !out_pos) return KVM_E_NULL;
    size_t need = 0;
    kvm_host_staging_bytes(p, &need);
    if (!dev || dev_bytes < need) return KVM_E_WORKSPACE;
    if (misaligned(dev)) return KVM_E_ALIGN;
    const size_t e = d.dtype == KVM_BF16 ? 2 : 4;
    const size_t rowQ = (size_t)d.G * d.S * d.D * e, rowK = (size_t)d.S * d.D * e;       // bytes per unit
    const size_t rowO = (size_t)d.cap * d.D * e, rowP = (size_t)d.cap * sizeof(int32_t);
    char* b = (char*)dev;
    size_t off = 0;
    auto take = [&](size_t n) { char* q = b + off; off += align_up(n); return q; };
    char* dQ = take(rowQ * d.U); char* dK = take(rowK * d.U); char* dV = take(rowK * d.U);
    char* dKo = take(rowO * d.U); char* dVo = take(rowO * d.U);
    char* dL = take((size_t)d.U * sizeof(int32_t)); char* dP = take(rowP * d.U);
    char* ws = b + off;
    const size_t ws_bytes = dev_bytes - off;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    // Units are independent and contiguous in every tensor, so the layer is cut into groups of units and
    // the three stages run as a pipeline: host-to-device copies on the caller's stream, kernels on a second
    // stream, device-to-host copies on a third.  The caller's stream waits for the last copy out.
    std::lock_guard<std::mutex> lock(g_pipe_mu);
    HostPipe* hp = host_pipe_for_current_device();
    if (!hp) return KVM_E_CUDA;
    const int nch = d.U < kHostChunksMax ? d.U : kHostChunksMax;
    const int per = (d.U + nch - 1) / nch;
    auto ok = [](cudaError_t err) { return err == cudaSuccess; };
    // a group of units as a layer of its own: one batch entry, nu KV heads
    auto group_params = [&](int u0, int nu) {
        kvm_params pc = *p;
        pc.batch = 1;
        pc.n_kv_heads = nu;
        pc.n_q_heads = nu * d.G;
        if (pc.pivot_key) pc.pivot_key += (size_t)u0 * d.S;
        return pc;
    };
    // every group is validated before anything is enqueued, so a refusal leaves no copy in flight
    for (int u0 = 0; u0 < d.U; u0 += per) {
        const kvm_params pc = group_params(u0, (d.U - u0 < per) ? d.U - u0 : per);
        Dims dc;
        size_t need_c = 0;
        if ((rc = derive(&pc, dc)) != KVM_OK) return rc;
        if ((rc = kvm_workspace_bytes(&pc, &need_c)) != KVM_OK) return rc;
        if (need_c > ws_bytes) return KVM_E_WORKSPACE;
    }
    if (!ok(cudaEventRecord(hp->start, st)) || !ok(cudaStreamWaitEvent(hp->compute, hp->start, 0)) ||
        !ok(cudaStreamWaitEvent(hp->d2h, hp->start, 0)))
        return KVM_E_CUDA;
    // From here on work is in flight on the library's streams: whatever happens, the caller's stream is made
    // to wait for all of it before the call returns, so that an error return never leaves copies writing the
    // caller's buffers behind its back.
    int status = KVM_OK;
    for (int c = 0, u0 = 0; u0 < d.U && status == KVM_OK; ++c, u0 += per) {
        const int nu = (d.U - u0 < per) ? d.U - u0 : per;
        const kvm_params pc = group_params(u0, nu);
        if (!ok(cudaMemcpyAsync(dQ + rowQ * u0, (const char*)Q + rowQ * u0, rowQ * nu, cudaMemcpyHostToDevice, st)) ||
            !ok(cudaMemcpyAsync(dK + rowK * u0, (const char*)K + rowK * u0, rowK * nu, cudaMemcpyHostToDevice, st)) ||
            !ok(cudaMemcpyAsync(dV + rowK * u0, (const char*)V + rowK * u0, rowK * nu, cudaMemcpyHostToDevice, st)) ||
            !ok(cudaEventRecord(hp->h2d[c], st)) || !ok(cudaStreamWaitEvent(hp->compute, hp->h2d[c], 0))) {
            status = KVM_E_CUDA;
            break;
        }
        rc = kvm_compress(&pc, dQ + rowQ * u0, dK + rowK * u0, dV + rowK * u0, dKo + rowO * u0, dVo + rowO * u0,
                          (int32_t*)dL + u0, (int32_t*)(dP + rowP * u0), nullptr, nullptr, ws, ws_bytes, hp->compute);
        if (rc != KVM_OK) {
            status = rc;
            break;
        }
        if (!ok(cudaEventRecord(hp->done[c], hp->compute)) || !ok(cudaStreamWaitEvent(hp->d2h, hp->done[c], 0)) ||
            !ok(cudaMemcpyAsync((char*)K_out + rowO * u0, dKo + rowO * u0, rowO * nu, cudaMemcpyDeviceToHost, hp->d2h)) ||
            !ok(cudaMemcpyAsync((char*)V_out + rowO * u0, dVo + rowO * u0, rowO * nu, cudaMemcpyDeviceToHost, hp->d2h)) ||
            !ok(cudaMemcpyAsync(out_len + u0, (int32_t*)dL + u0, (size_t)nu * sizeof(int32_t), cudaMemcpyDeviceToHost,
                                hp->d2h)) ||
            !ok(cudaMemcpyAsync((char*)out_pos + rowP * u0, dP + rowP * u0, rowP * nu, cudaMemcpyDeviceToHost, hp->d2h)))
            status = KVM_E_CUDA;
    }
    // join: the copy-out stream follows the compute stream, the caller's stream follows the copy-out stream
    if (!ok(cudaEventRecord(hp->done[0], hp->compute)) || !ok(cudaStreamWaitEvent(hp->d2h, hp->done[0], 0)) ||
        !ok(cudaEventRecord(hp->end, hp->d2h)) || !ok(cudaStreamWaitEvent(st, hp->end, 0)))
        return KVM_E_CUDA;
    return status;
}

// ---------------------------------------------------------------------------
// kvm_score without a caller workspace, for callers that may not allocate.
// The scratch is part of the library image; see the declaration in kvm.h.
namespace {

constexpr int kMaxDevices = KVM_MAX_DEVICES;

// The row pass's output for up to KVM_STATIC_SCORE_ROWS fp32 rows.  In HOST code this name is only a stand-in
// for the device symbol; its device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_score_scratch[(size_t)KVM_STATIC_SCORE_ROWS * sizeof(float)];

void* g_static_ptr[kMaxDevices];   // device address of the array, per device; set once

// One-time set-up for the current device.  Returns nullptr if the runtime refuses.
void* static_scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void* ptr = __atomic_load_n(&g_static_ptr[dev], __ATOMIC_ACQUIRE);
    if (ptr) return ptr;
    if (cudaGetSymbolAddress(&ptr, g_static_score_scratch) != cudaSuccess || !ptr) return nullptr;
    __atomic_store_n(&g_static_ptr[dev], ptr, __ATOMIC_RELEASE);   // racing first calls store the same value
    return ptr;
}

}  // namespace

int kvm_score_static(const kvm_params* p, const void* Q, const void* K, float* scores, void* cuda_stream) {
    Dims d;
    int rc = derive(p, d);
    if (rc != KVM_OK) return rc;
    if (!Q || !K || !scores) return KVM_E_NULL;
    if (misaligned(Q) || misaligned(K) || misaligned(scores)) return KVM_E_ALIGN;
    // the row pass leaves 4 bytes per query row for fp32 tensors and 32 bytes for bf16 ones
    if ((unsigned long long)d.B * d.Hq * d.S * score_row_bytes(d) > (unsigned long long)KVM_STATIC_SCORE_ROWS * sizeof(float))
        return KVM_E_STATIC_LIMIT;
    unsigned char* base = (unsigned char*)static_scratch_for_current_device();
    if (!base) return KVM_E_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // The array keeps the previous call's contents.  Nothing in it has to start at zero: the row pass rewrites
    // every row this call's column pass reads.
    Workspace w;
    w.lse = (float*)base;
    w.scores = nullptr;
    w.sim = nullptr;
    w.set_start = nullptr;
    w.set_id = nullptr;
    w.merge_part = nullptr;
    w.attend_part = nullptr;
    w.bytes = sizeof(g_static_score_scratch);
    return run_score(d, Q, K, nullptr, scores, w, nullptr, st) == cudaSuccess ? KVM_OK : KVM_E_CUDA;
}

}  // extern "C"
