"""B200-native KVMerger prefill-time KV-cache compression: CUDA library + thin binding.

`binding` wraps the C ABI of include/kvm.h (libkvm.so, built in-tree by `build`);
`synth_inputs` holds the seeded synthetic workloads.
"""
from . import synth_inputs  # noqa: F401
from .binding import (  # noqa: F401
    KVM_BF16, KVM_F32, KVM_PIVOT_KEY, KVM_PIVOT_LAST, KVM_PIVOT_MAX_SCORE, KVM_SETS_ADJACENT, KVM_SETS_ANCHOR,
    KVM_SETS_CONSERVED_ONLY, KVM_WEIGHT_AVERAGE, KVM_WEIGHT_GAUSSIAN, KVM_WEIGHT_PIVOT_ONLY, KVM_WEIGHT_SET_SIGMA, Compressed, Compressor, KvmError, KvmParams, KvmStats, kvm_compress, kvm_compress_host, kvm_compress_with_lse,
    kvm_host_staging_bytes, kvm_layer_ratio, kvm_row_lse, compress_layers, kvm_attend, kvm_prefill_attend, kvm_output_perturbation, kvm_merge_compact, kvm_score, kvm_score_static, kvm_segment, kvm_sizes, kvm_version,
    kvm_workspace_bytes, make_params, new_stats, read_stats, status_string,
)
