/*
 * kvm -- prefill-time KV-cache compression by adaptive merging (KVMerger,
 * arXiv 2407.08454) for NVIDIA B200 (sm_100a).  C ABI.
 *
 * Per attention layer and per (batch entry, KV head) "unit" the library
 *   1. sums the causal attention map softmax(Q K^T * scale) over queries, giving
 *      one aggregated score per key (Eq. 1; Algorithm 2; Eq. 6; for grouped-query
 *      attention the maps of a KV head's query heads are averaged, Section 5.2);
 *   2. measures the cosine similarity of neighbouring keys (Eq. 2) and cuts the
 *      sequence into merging sets of consecutive tokens (Algorithm 1,
 *      Definition 4.1); the most recent tokens and the keys with the largest
 *      scores are conserved, i.e. never merged (Sections 4.1, 4.2, 5.1);
 *   3. picks each set's pivot, the key with the largest score (Eq. 6);
 *   4. merges each set's keys and values into one state with Gaussian-kernel
 *      weights around the pivot (Eq. 4, Eq. 5, Definition 4.2) and writes the
 *      states densely, in token order.
 *
 * Conventions for every entry point
 *   - Unless a parameter says "host", tensor pointers are DEVICE pointers owned by
 *     the caller, contiguous row-major in the stated shape and 16-byte aligned.
 *     Inputs are never written.
 *   - The library allocates no device memory and, kvm_compress_host's streams
 *     aside, keeps no state between calls.  Scratch
 *     space is the caller's `ws` buffer of at least kvm_workspace_bytes() bytes;
 *     its contents are undefined afterwards.  Calls that share a workspace must
 *     be ordered on one stream.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream) and the call returns without synchronising.
 *   - Return value: KVM_OK, or a negative kvm_status found on the host before
 *     anything was enqueued (KVM_E_CUDA: a launch or copy was refused by the
 *     runtime).  Conditions found on the device are reported through kvm_stats.
 *   - U = batch * n_kv_heads units; G = n_q_heads / n_kv_heads; S = seq;
 *     D = head_dim; cap = output capacity in rows per unit =
 *     floor(budget * S) when enforce_budget, else S.
 */
#ifndef KVM_H_
#define KVM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVM_VERSION 101

enum kvm_dtype { KVM_BF16 = 0, KVM_F32 = 1 };

enum kvm_status {
    KVM_OK = 0,
    KVM_E_NULL = -1,        /* a required pointer is NULL */
    KVM_E_SHAPE = -2,       /* sizes not positive, heads not divisible, head_dim not 64/128, seq too long */
    KVM_E_DTYPE = -3,       /* dtype is not a kvm_dtype */
    KVM_E_PARAM = -4,       /* ratio/threshold/bandwidth/rule out of range, or capacity too small for the conserved set */
    KVM_E_ALIGN = -5,       /* a tensor pointer is not 16-byte aligned */
    KVM_E_WORKSPACE = -6,   /* ws is NULL or smaller than kvm_workspace_bytes() */
    KVM_E_UNSUPPORTED = -7, /* valid request this build cannot run (e.g. non-causal) */
    KVM_E_CUDA = -8,        /* the CUDA runtime refused a launch, a copy or a driver lookup */
    KVM_E_DEVICE_TIMEOUT = -9, /* only ever appears in kvm_stats.status: a bounded device wait gave up */
    KVM_E_STATIC_LIMIT = -10 /* kvm_score_static: the problem does not fit the built-in scratch (see KVM_STATIC_SCORE_ROWS) */
};

/* The paper's problem statement as a plain struct (Section 2.4; hyper-parameters of Section 5.1). */
typedef struct kvm_params {
    int32_t batch, n_q_heads, n_kv_heads, seq, head_dim; /* head_dim 64 or 128; seq <= KVM_MAX_SEQ */
    int32_t dtype;               /* kvm_dtype of Q, K, V and of K_out, V_out */
    float budget;                /* (0,1]: cache budget, 0.50 or 0.35 in the paper */
    float recent_ratio;          /* share of S conserved as most recent tokens; < 0: preset 0.17 (budget >= 0.425) else 0.08 */
    float heavy_ratio;           /* share of S conserved for largest scores;    < 0: preset 0.12 (budget >= 0.425) else 0.02 */
    float sim_threshold;         /* epsilon of Algorithm 1; neighbours group when similarity > epsilon (strict); paper: 0.75 */
    float sigma;                 /* Gaussian bandwidth of Eq. 4, > 0 (only KVM_WEIGHT_GAUSSIAN reads it); the paper's best fixed value is 5 */
    float softmax_scale;         /* <= 0: 1/sqrt(head_dim) as in Eq. 1 */
    int32_t causal;              /* must be 1 */
    int32_t scale_v_by_set_size; /* 1: value weights are multiplied by the set size (text after Eq. 5); 0: plain weighted mean */
    int32_t enforce_budget;      /* 1: at most floor(budget*S) sets per unit (see kvm_segment); 0: capacity is S */
    /* Variants the paper describes beside its method.  All zero = the method itself. */
    int32_t pivot_rule;          /* kvm_pivot_rule */
    int32_t weight_rule;         /* kvm_weight_rule */
    int32_t set_rule;            /* kvm_set_rule */
    const float* pivot_key;      /* device [U, S] fp32, finite, 4-byte aligned; read only when pivot_rule == KVM_PIVOT_KEY, else NULL */
} kvm_params;

/* How the pivot of a merging set is chosen. */
enum kvm_pivot_rule {
    KVM_PIVOT_MAX_SCORE = 0, /* largest aggregated attention score (Eq. 6) */
    KVM_PIVOT_LAST = 1,      /* the set's maximum token index (the average-weighted baseline of Section 4.2) */
    KVM_PIVOT_KEY = 2        /* largest pivot_key, ties to the lowest index; iid random keys give the random-pivot
                                ablation of Section 5.3.  The conserved set still comes from the attention scores. */
};
/* How a set's states are weighted. */
enum kvm_weight_rule {
    KVM_WEIGHT_GAUSSIAN = 0,  /* Eq. 4, Eq. 5 with the fixed sigma */
    KVM_WEIGHT_AVERAGE = 1,   /* every state 1/|set| (average-weighted merging, Section 4.2); sigma is ignored */
    KVM_WEIGHT_PIVOT_ONLY = 2, /* the sigma -> 0 limit noted after Eq. 5: the pivot's own K and V rows, nothing
                                  merged in (V still times the set size when scale_v_by_set_size) */
    KVM_WEIGHT_SET_SIGMA = 3   /* a bandwidth per merging set.  Eq. 4 defines sigma through the weights that depend
                                  on it; this rule is one non-circular reading, not the paper's statement:
                                  2 sigma_s^2 = mean over the set of |k_p - k_j|^2, so g_j = exp(-|k_p - k_j|^2 / mean)
                                  (every g_j = 1 when the mean is 0).  sigma is ignored. */
};
/* Which states reach the output. */
enum kvm_set_rule {
    KVM_SETS_ADJACENT = 0,       /* Algorithm 1: every token belongs to a merging set */
    KVM_SETS_CONSERVED_ONLY = 1, /* eviction as in the heavy-hitter schemes of Section 2.2: only the conserved tokens
                                    (largest scores + most recent) stay, unchanged, in token order; pivot_rule,
                                    weight_rule, sim_threshold and sigma are ignored, out_len = n_recent + n_heavy,
                                    which must fit the capacity; set_id is -1 for dropped tokens and
                                    set_start[s] = pivot[s] = the s-th kept token */
    KVM_SETS_ANCHOR = 2          /* the set identification as Section 3.2 words it: walking from the last token, a
                                    state gathers the consecutive states before it whose similarity TO IT exceeds
                                    sim_threshold (Algorithm 1 compares neighbours instead).  Conserved
                                    tokens stand alone.  No budget rule: enforce_budget must be 0 (capacity S), and
                                    seq <= KVM_ANCHOR_MAX_SEQ.  kvm_segment's sim_out then receives, per token, the
                                    number of predecessors it would gather as a group's last state. */
};

#define KVM_MAX_SEQ 65536
#define KVM_ANCHOR_MAX_SEQ 40960 /* longest sequence for KVM_SETS_ANCHOR (its walk lives in shared memory) */

/* Device-side report, filled by kvm_segment / kvm_compress when given.  Zero it before the call. */
typedef struct kvm_stats {
    int32_t status;            /* KVM_OK or KVM_E_DEVICE_TIMEOUT */
    int32_t units_budget_rule; /* units in which the budget rule removed boundaries */
    int32_t near_threshold;    /* neighbour pairs with |similarity - epsilon| < 1e-3 */
    int32_t min_out_len, max_out_len; /* over units (min starts at 0 meaning "unset") */
    int64_t sum_out_len;
} kvm_stats;

/* Derived sizes for a parameter set: capacity rows per unit, recent count, heavy-hitter count. Host only. */
int kvm_sizes(const kvm_params* p, int32_t* cap, int32_t* n_recent, int32_t* n_heavy);

/* Bytes of scratch every entry point below accepts for these parameters. Host only. */
int kvm_workspace_bytes(const kvm_params* p, size_t* bytes);

/*
 * Aggregated attention scores (Eq. 1 restricted to the causal part; column sums
 * as in Algorithm 2 / Eq. 6; mean over the G query heads of a KV head, Section 5.2).
 *   Q [batch, n_q_heads, S, D], K [batch, n_kv_heads, S, D] in p->dtype.
 *   lse_in: NULL, or [batch, n_q_heads, S] fp32 natural-log row log-sum-exp of
 *           the scaled causal logits (e.g. from the prefill attention kernel);
 *           when given, the row pass is skipped.
 *   scores: [batch, n_kv_heads, S] fp32, written.
 * bf16 runs on tensor cores with fp32 accumulation and fp32 softmax; fp32 runs in fp32 FMA.
 */
int kvm_score(const kvm_params* p, const void* Q, const void* K, const float* lse_in,
              float* scores, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The row pass of kvm_score alone: the natural-log row log-sum-exp of the scaled causal logits (Eq. 1's softmax
 * normaliser), lse_out [batch, n_q_heads, S] fp32, written.  It is what kvm_score and kvm_compress_with_lse accept
 * as lse_in, so a caller that compresses the same layer several times (other budgets, thresholds or rules) pays
 * for the row pass once.
 */
int kvm_row_lse(const kvm_params* p, const void* Q, const void* K, float* lse_out, void* ws, size_t ws_bytes,
                void* cuda_stream);

/*
 * Merging-set identification and pivots (Eq. 2, Algorithm 1, Definition 4.1, Eq. 6).
 *   K [batch, n_kv_heads, S, D]; scores [batch, n_kv_heads, S] fp32.
 *   Conserved tokens: the last n_recent positions and, among the others, the
 *   n_heavy largest scores (ties: lower index).  Token j starts a set when j = 0,
 *   when j or j-1 is conserved, or when cos(k_{j-1}, k_j) > epsilon is false.
 *   Budget rule (enforce_budget): if that gives more than cap sets, only the
 *   cap - (forced cuts) similarity cuts with the smallest similarity are kept
 *   (ties: lower index), which equals lowering epsilon for that unit.
 *   Outputs (all written for rows < out_len only):
 *     set_id    NULL or [U, S] i32     set index of each token
 *     set_start [U, cap+1] i32         first token of each set; set_start[out_len] = S
 *     pivot     [U, cap] i32           token with the largest score in the set (ties: lowest index)
 *     out_len   [U] i32                number of sets
 *     sim_out   NULL or [U, S] fp32    cos(k_{j-1}, k_j), entry 0 is 0
 *     stats     NULL or device kvm_stats
 */
int kvm_segment(const kvm_params* p, const void* K, const float* scores,
                int32_t* set_id, int32_t* set_start, int32_t* pivot, int32_t* out_len,
                float* sim_out, kvm_stats* stats, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Gaussian-kernel weighted merge and compaction (Eq. 4 with fixed sigma, Eq. 5,
 * Definition 4.2, Algorithm 2).  For set s with tokens [set_start[s], set_start[s+1])
 * and pivot p:  g_j = exp(-|k_p - k_j|^2 / (2 sigma^2)),  K_out[s] = sum g_j k_j / sum g_j,
 * V_out[s] = n_s * sum g_j v_j / sum g_j (n_s omitted when !scale_v_by_set_size).
 * fp32 accumulation, one round-to-nearest-even conversion at the store; a set of
 * one token is copied bit for bit.
 *   K, V [U, S, D]; set_start [U, cap+1]; pivot [U, cap]; out_len [U] (device).
 *   K_out, V_out [U, cap, D] in p->dtype; rows >= out_len are left untouched.
 *   out_size: NULL or [U, cap] i32, the size of each set.
 */
int kvm_merge_compact(const kvm_params* p, const void* K, const void* V,
                      const int32_t* set_start, const int32_t* pivot, const int32_t* out_len,
                      void* K_out, void* V_out, int32_t* out_size,
                      void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The whole path for one layer: kvm_score, kvm_segment, kvm_merge_compact chained
 * on the stream with intermediates in the workspace.
 * (No allocation, no synchronisation, no host-side state: the call can be captured
 * into a CUDA graph and replayed.)
 *   out_pos    [U, cap] i32   pivot token index of each output row (ascending)
 *   scores_out NULL or [U, S] fp32
 *   stats      NULL or device kvm_stats
 */
int kvm_compress(const kvm_params* p, const void* Q, const void* K, const void* V,
                 void* K_out, void* V_out, int32_t* out_len, int32_t* out_pos,
                 float* scores_out, kvm_stats* stats, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * kvm_compress for callers that already hold the row log-sum-exp of the layer's causal attention (a fused
 * prefill attention kernel produces it as a by-product): lse_in [batch, n_q_heads, S] fp32, natural log, of
 * the logits scaled by softmax_scale.  The row pass of the score step is skipped, which halves the score
 * step's work (Eq. 1 is evaluated once per query-key pair instead of twice).  lse_in NULL = kvm_compress.
 */
int kvm_compress_with_lse(const kvm_params* p, const void* Q, const void* K, const void* V, const float* lse_in,
                          void* K_out, void* V_out, int32_t* out_len, int32_t* out_pos, float* scores_out,
                          kvm_stats* stats, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * kvm_compress for callers whose tensors live in HOST memory (pinned memory
 * makes the copies asynchronous).  Q, K, V, K_out, V_out, out_len, out_pos are
 * host pointers with the shapes of kvm_compress; `dev` is a caller-owned device
 * buffer of at least kvm_host_staging_bytes() bytes that holds the staged tensors
 * and the workspace.  Copies in, compresses, copies all cap rows out.  The layer
 * is cut into groups of units that flow through a three-stage pipeline (copy in
 * on `cuda_stream`, kernels and copy out on two streams of the library's own), so
 * that the copies in both directions overlap each other and the kernels;
 * `cuda_stream` waits for the last copy out, and the caller synchronises it before
 * reading.  The first call on a device creates the two streams and a handful of
 * events, which live until the process exits (the one piece of state the library
 * keeps); calls are serialised by a host mutex while they enqueue.
 */
int kvm_host_staging_bytes(const kvm_params* p, size_t* bytes);
int kvm_compress_host(const kvm_params* p, const void* Q, const void* K, const void* V,
                      void* K_out, void* V_out, int32_t* out_len, int32_t* out_pos,
                      void* dev, size_t dev_bytes, void* cuda_stream);

/*
 * Layer-wise compression ratio of the set identification alone (Section 3.2, Figure 3(b)): per unit,
 * (number of merging sets Algorithm 1 forms with nothing conserved and no budget) / S, for the
 * threshold p->sim_threshold.  Lowering the threshold lowers the ratio; the paper proposes choosing a
 * threshold per layer from this statistic, which callers do by giving each layer's kvm_compress call its
 * own sim_threshold.
 *   K [batch, n_kv_heads, S, D]; ratio [U] fp32 (device), written; sim_out NULL or [U, S] fp32.
 * budget, recent_ratio, heavy_ratio, sigma and the rules of p are not used.
 */
int kvm_layer_ratio(const kvm_params* p, const void* K, float* ratio, float* sim_out,
                    void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * A stack of layers with one similarity threshold each (Section 3.2: the layer-wise compression ratios can be set
 * by adjusting the threshold layer by layer): n_layers calls of kvm_compress, layer l with sim_threshold =
 * sim_thresholds[l] (p->sim_threshold for all layers when sim_thresholds is NULL), enqueued one after the other on
 * the stream; the workspace is shared, the layers' tensors are not.
 *   Q, K, V, K_out, V_out, out_len, out_pos: HOST arrays of n_layers device pointers, each as in kvm_compress
 *   sim_thresholds: NULL or a HOST array of n_layers floats (read before the call returns)
 *   stats: NULL or one device kvm_stats that accumulates over the layers
 * Every layer's arguments are checked before anything is enqueued.
 */
int kvm_compress_layers(const kvm_params* p, int32_t n_layers, const float* sim_thresholds, const void* const* Q,
                        const void* const* K, const void* const* V, void* const* K_out, void* const* V_out,
                        int32_t* const* out_len, int32_t* const* out_pos, kvm_stats* stats, void* ws,
                        size_t ws_bytes, void* cuda_stream);

/*
 * Causal attention over the whole prompt (Eq. 1 for every position: O_i = softmax_{j<=i}(q_i K^T * scale) V), the
 * attention a prefill runs in any case, together with each row's natural-log log-sum-exp.  The compression is
 * applied at the end of the prefill (Section 4, Figure 4): a caller that computes its prefill attention here hands
 * `lse` to kvm_compress_with_lse (or kvm_score's lse_in) and the score step then needs no row pass of its own.
 * Query head h of batch entry b reads KV head h / G.
 *   Q    [batch, n_q_heads, S, D], K, V [batch, n_kv_heads, S, D]: device, bf16 (KVM_E_UNSUPPORTED otherwise),
 *        16-byte aligned, not written
 *   O    [batch, n_q_heads, S, D] bf16 (device), written: fp32 accumulation, one rounding at the store; the
 *        probabilities enter the second product rounded to bf16, as in the tensor-core attention kernels in use
 *   lse  [batch, n_q_heads, S] fp32 (device), written: ln sum_{j<=i} exp(scale * q_i.k_j)
 *   stats NULL or a device kvm_stats: status = KVM_E_DEVICE_TIMEOUT if a bounded wait inside the kernel gave up
 *        (the rows in hand at that moment are then NaN, rows of later work items are not written)
 * Tensor cores (tcgen05); no workspace.  Only the shape, dtype and softmax_scale of p are used.  Enqueues on the
 * stream and returns; errors found on the host are returned before anything is enqueued.
 */
int kvm_prefill_attend(const kvm_params* p, const void* Q, const void* K, const void* V, void* O, float* lse,
                       kvm_stats* stats, void* cuda_stream);

/*
 * One decode step of attention (Eq. 1: O_t = softmax(q_t K^T * scale) V) over a cache whose units may hold
 * different numbers of rows, e.g. the output of kvm_compress.  Query head h of batch entry b reads KV head h / G.
 *   q    [batch, n_q_heads, D] in p->dtype
 *   K, V [batch, n_kv_heads, rows, D] in p->dtype, 1 <= rows <= S
 *   len  NULL (every unit holds `rows` rows) or device [U] i32: rows of each unit that are valid
 *   out  [batch, n_q_heads, D] fp32, written; a unit with no rows gives zeros
 * fp32 arithmetic.  Only the shape, dtype and softmax_scale of p are used.
 */
int kvm_attend(const kvm_params* p, const void* q, const void* K, const void* V, int32_t rows, const int32_t* len,
               float* out, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The criterion of Definition 2.1 for one decode step: attention outputs over the full cache (K, V
 * [U, S, D]) and over the compressed one (K_c, V_c [U, cap, D] with len_c [U], as kvm_compress leaves
 * them for the same p), and per (batch, query head) err = |O_t - O_t*|_2 and ref = |O_t|_2.
 *   out_full, out_comp [batch, n_q_heads, D] fp32; err, ref [batch, n_q_heads] fp32; all written.
 */
int kvm_output_perturbation(const kvm_params* p, const void* q, const void* K, const void* V, const void* K_c,
                            const void* V_c, const int32_t* len_c, float* out_full, float* out_comp, float* err,
                            float* ref, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * kvm_score for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of kvm_score, same arithmetic.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * serving engine that handed its whole memory pool to another allocator at
 * start-up, in a plugin that is not allowed to grow the process's footprint, or
 * on a latency path where an allocation (which may synchronise the device) is
 * not acceptable -- and that has no spare buffer to lend as a workspace.
 *
 * Instead of a caller workspace, the row log-sum-exp scratch lives in a fixed
 * array built into the library image: KVM_STATIC_SCORE_ROWS floats (4 MiB).  Every
 * GPU on which the CUDA runtime loads the library's device code holds that array
 * from then (at the latest from this function's first call there) until the process
 * exits, whether or not the function is called again.
 *
 *   - Same Q, K, scores and stream arguments as kvm_score; no lse_in, no ws.
 *   - batch * n_q_heads * seq must not exceed KVM_STATIC_SCORE_ROWS for fp32 tensors and
 *     KVM_STATIC_SCORE_ROWS / 8 for bf16 tensors (their row pass leaves 32 bytes per row), otherwise
 *     KVM_E_STATIC_LIMIT is returned and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (a
 *     one-time host-side set-up, done with that device current).  Make that first
 *     call outside any stream capture.
 *   - All calls on one device share the one array and it keeps whatever the last
 *     call left there.  Nothing in it has to start at zero (the row pass rewrites
 *     every row before the column pass reads it), but two calls whose kernels
 *     overlap on the GPU (different streams, no ordering between them) write and
 *     read the same rows and give wrong scores: order such calls on one stream or
 *     with events.
 *   - Calls no cudaMalloc/cudaFree and no allocating library routine.
 */
#define KVM_STATIC_SCORE_ROWS (1 << 20)
int kvm_score_static(const kvm_params* p, const void* Q, const void* K, float* scores, void* cuda_stream);

const char* kvm_status_string(int status);
int kvm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVM_H_ */
