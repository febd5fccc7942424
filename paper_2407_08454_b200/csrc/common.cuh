// Shared declarations of the kvm CUDA library (internal; the public ABI is include/kvm.h).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvm.h"

namespace kvm {

constexpr int KVM_MAX_DEVICES = 64;   // per-device host-side caches are arrays of this size

// Validated, derived problem sizes handed to every launcher.
struct Dims {
    int B, Hq, Hkv, G, S, D, U;
    int cap, n_r, n_h;
    int dtype;  // kvm_dtype
    float scale, eps, sigma;
    int scale_v, enforce;
    int pivot_rule, weight_rule, set_rule;   // kvm_pivot_rule, kvm_weight_rule, kvm_set_rule
    const float* pivot_key;                  // [U,S] when pivot_rule == KVM_PIVOT_KEY
};

// 16-byte vector <-> fp32 lanes.  Vec<T>::N elements of T per 16 bytes.
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
        // bf16 -> fp32 is a 16-bit left shift
        f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);  // round to nearest even
        return *reinterpret_cast<uint32_t*>(&v);
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
    }
};

__device__ __forceinline__ uint4 ldg16(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }

// Programmatic dependent launch: a kernel launched with launch_dependent() may be scheduled while the kernel
// before it on the stream is still draining; it must call grid_dependency_wait() before it touches anything that
// kernel wrote (the wait returns once the earlier grid has completed and its writes are visible; it is a no-op for
// a kernel launched the ordinary way).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the kernel launched after this one (with launch_dependent) be scheduled once every block of this grid has
// called it or exited; that kernel still waits for this grid's completion in its grid_dependency_wait().
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Launchers (each enqueues on the stream and returns the launch status).
cudaError_t launch_score_simt(const Dims& d, const void* Q, const void* K, const float* lse_in, float* lse_ws,
                              float* scores, cudaStream_t st);
cudaError_t launch_score_tc(const Dims& d, const void* Q, const void* K, const float* lse_in, float* lse_ws,
                            float* scores, kvm_stats* stats, cudaStream_t st, float* sim_out = nullptr,
                            float* lse_out = nullptr);
size_t score_tc_scratch_bytes_per_row();
cudaError_t launch_prefill_attend(const Dims& d, const void* Q, const void* K, const void* V, void* O, float* lse,
                                  kvm_stats* stats, cudaStream_t st);
cudaError_t launch_similarity(const Dims& d, const void* K, float* sim, cudaStream_t st);
cudaError_t launch_segment(const Dims& d, const float* scores, const float* sim, int32_t* set_id,
                           int32_t* set_start, int32_t* pivot, int32_t* out_len, kvm_stats* stats, cudaStream_t st);
size_t segment_max_smem();
cudaError_t launch_anchor_runs(const Dims& d, const void* K, float* run_out, float* inv_norm, cudaStream_t st);
cudaError_t launch_set_ratio(const Dims& d, const float* sim, float* ratio, cudaStream_t st);
size_t merge_scratch_floats(const Dims& d);
cudaError_t launch_token_sets(const Dims& d, const int32_t* set_start, const int32_t* out_len, int32_t* set_id,
                              cudaStream_t st);
cudaError_t launch_merge(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                         const int32_t* pivot, const int32_t* set_id, const int32_t* out_len, void* K_out,
                         void* V_out, int32_t* out_size, float* scratch, float* set_coef, float* token_d2,
                         kvm_stats* stats, cudaStream_t st);
// Rows that are one input state each (pivot-only weights, eviction): a gather.
cudaError_t launch_gather(const Dims& d, const void* K, const void* V, const int32_t* set_start,
                          const int32_t* pivot, const int32_t* out_len, void* K_out, void* V_out, int32_t* out_size,
                          cudaStream_t st);

// Decode-step attention over a ragged cache and the full-vs-compressed output difference.
int attend_splits(int rows);
size_t attend_scratch_floats(const Dims& d);
cudaError_t launch_attend(const Dims& d, const void* q, const void* K, const void* V, int rows, const int32_t* len,
                          float* out, float* part, cudaStream_t st);
cudaError_t launch_perturbation(const Dims& d, const float* O, const float* Os, float* err, float* ref,
                                cudaStream_t st);

}  // namespace kvm
