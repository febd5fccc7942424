"""Thin ctypes binding of libkvm.so: argument marshalling only.

Function names and argument order follow include/kvm.h.  Tensors are torch CUDA
tensors (device memory and the current stream come from torch); every step of
the compression path runs inside the library's kernels.  There is no CPU path:
loading fails loudly when the shared library is missing.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvm.so")

KVM_BF16, KVM_F32 = 0, 1
KVM_OK = 0
KVM_PIVOT_MAX_SCORE, KVM_PIVOT_LAST, KVM_PIVOT_KEY = 0, 1, 2
KVM_WEIGHT_GAUSSIAN, KVM_WEIGHT_AVERAGE, KVM_WEIGHT_PIVOT_ONLY, KVM_WEIGHT_SET_SIGMA = 0, 1, 2, 3
KVM_SETS_ADJACENT, KVM_SETS_CONSERVED_ONLY, KVM_SETS_ANCHOR = 0, 1, 2
EXPORTS = (
    "kvm_sizes", "kvm_workspace_bytes", "kvm_score", "kvm_row_lse", "kvm_segment", "kvm_merge_compact", "kvm_compress",
    "kvm_compress_with_lse", "kvm_compress_layers",
    "kvm_host_staging_bytes", "kvm_compress_host", "kvm_score_static", "kvm_layer_ratio", "kvm_attend",
    "kvm_output_perturbation", "kvm_prefill_attend", "kvm_status_string",
    "kvm_version",
)
KVM_STATIC_SCORE_ROWS = 1 << 20


class KvmParams(ctypes.Structure):
    """Mirror of `kvm_params`."""
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("seq", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("budget", ctypes.c_float), ("recent_ratio", ctypes.c_float), ("heavy_ratio", ctypes.c_float),
        ("sim_threshold", ctypes.c_float), ("sigma", ctypes.c_float), ("softmax_scale", ctypes.c_float),
        ("causal", ctypes.c_int32), ("scale_v_by_set_size", ctypes.c_int32), ("enforce_budget", ctypes.c_int32),
        ("pivot_rule", ctypes.c_int32), ("weight_rule", ctypes.c_int32), ("set_rule", ctypes.c_int32),
        ("pivot_key", ctypes.c_void_p),
    ]


class KvmStats(ctypes.Structure):
    """Mirror of `kvm_stats` (24 + 8 bytes)."""
    _fields_ = [
        ("status", ctypes.c_int32), ("units_budget_rule", ctypes.c_int32), ("near_threshold", ctypes.c_int32),
        ("min_out_len", ctypes.c_int32), ("max_out_len", ctypes.c_int32), ("_pad", ctypes.c_int32),
        ("sum_out_len", ctypes.c_int64),
    ]


class KvmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libkvm.so (built by paper_2407_08454_b200.build).  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: run `python -m paper_2407_08454_b200.build` (needs nvcc). "
                "There is no fallback path.")
        L = ctypes.CDLL(LIB_PATH)
        L.kvm_status_string.restype = ctypes.c_char_p
        L.kvm_status_string.argtypes = [ctypes.c_int]
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().kvm_status_string(int(status)).decode()


def make_params(batch: int, n_q_heads: int, n_kv_heads: int, seq: int, head_dim: int, dtype,
                budget: float = 0.5, recent_ratio: float = -1.0, heavy_ratio: float = -1.0,
                sim_threshold: float = 0.75, sigma: float = 5.0, softmax_scale: float = 0.0, causal: int = 1,
                scale_v_by_set_size: int = 1, enforce_budget: int = 1, pivot_rule: int = 0, weight_rule: int = 0,
                set_rule: int = 0, pivot_key: Optional[torch.Tensor] = None) -> KvmParams:
    """`pivot_key` ([batch, n_kv_heads, seq] fp32 CUDA tensor) must stay alive while the parameters are in use."""
    if isinstance(dtype, torch.dtype):
        dtype = {torch.bfloat16: KVM_BF16, torch.float32: KVM_F32}[dtype]
    key_ptr = None
    if pivot_key is not None:
        assert pivot_key.is_cuda and pivot_key.dtype == torch.float32 and pivot_key.is_contiguous()
        assert tuple(pivot_key.shape) == (batch, n_kv_heads, seq)
        key_ptr = pivot_key.data_ptr()
    return KvmParams(batch, n_q_heads, n_kv_heads, seq, head_dim, int(dtype), budget, recent_ratio, heavy_ratio,
                     sim_threshold, sigma, softmax_scale, causal, scale_v_by_set_size, enforce_budget,
                     pivot_rule, weight_rule, set_rule, key_ptr)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_contiguous(), "tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int, where: str) -> None:
    if rc != KVM_OK:
        raise KvmError(rc, where)


def kvm_version() -> int:
    return int(lib().kvm_version())


def kvm_sizes(p: KvmParams):
    cap, nr, nh = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().kvm_sizes(ctypes.byref(p), ctypes.byref(cap), ctypes.byref(nr), ctypes.byref(nh)), "kvm_sizes")
    return cap.value, nr.value, nh.value


def kvm_workspace_bytes(p: KvmParams) -> int:
    n = ctypes.c_size_t()
    _check(lib().kvm_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "kvm_workspace_bytes")
    return n.value


def kvm_host_staging_bytes(p: KvmParams) -> int:
    n = ctypes.c_size_t()
    _check(lib().kvm_host_staging_bytes(ctypes.byref(p), ctypes.byref(n)), "kvm_host_staging_bytes")
    return n.value


def kvm_score(p: KvmParams, Q, K, lse_in, scores, ws, stream=None) -> None:
    _check(lib().kvm_score(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(lse_in), _ptr(scores), _ptr(ws),
                           ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_score")


def kvm_row_lse(p: KvmParams, Q, K, lse_out, ws, stream=None) -> None:
    _check(lib().kvm_row_lse(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(lse_out), _ptr(ws),
                             ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_row_lse")


def kvm_score_static(p: KvmParams, Q, K, scores, stream=None) -> None:
    """kvm_score on the library's built-in scratch: for callers that cannot allocate a workspace.
    batch * n_q_heads * seq must not exceed KVM_STATIC_SCORE_ROWS (fp32) or an eighth of it (bf16); calls on one
    device must not overlap."""
    _check(lib().kvm_score_static(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(scores), _stream(stream)),
           "kvm_score_static")


def kvm_segment(p: KvmParams, K, scores, set_id, set_start, pivot, out_len, sim_out, stats, ws, stream=None) -> None:
    _check(lib().kvm_segment(ctypes.byref(p), _ptr(K), _ptr(scores), _ptr(set_id), _ptr(set_start), _ptr(pivot),
                             _ptr(out_len), _ptr(sim_out), _ptr(stats), _ptr(ws),
                             ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_segment")


def kvm_layer_ratio(p: KvmParams, K, ratio, sim_out, ws, stream=None) -> None:
    _check(lib().kvm_layer_ratio(ctypes.byref(p), _ptr(K), _ptr(ratio), _ptr(sim_out), _ptr(ws),
                                 ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_layer_ratio")


def kvm_attend(p: KvmParams, q, K, V, rows: int, length, out, ws, stream=None) -> None:
    _check(lib().kvm_attend(ctypes.byref(p), _ptr(q), _ptr(K), _ptr(V), ctypes.c_int32(rows), _ptr(length), _ptr(out),
                            _ptr(ws), ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_attend")


def kvm_prefill_attend(p: KvmParams, Q, K, V, O, lse, stats=None, stream=None) -> None:
    """Causal attention over the whole prompt: O [B,Hq,S,D] bf16 and the rows' natural-log log-sum-exp [B,Hq,S]."""
    _check(lib().kvm_prefill_attend(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse), _ptr(stats),
                                    _stream(stream)), "kvm_prefill_attend")


def kvm_output_perturbation(p: KvmParams, q, K, V, K_c, V_c, len_c, out_full, out_comp, err, ref, ws,
                            stream=None) -> None:
    _check(lib().kvm_output_perturbation(ctypes.byref(p), _ptr(q), _ptr(K), _ptr(V), _ptr(K_c), _ptr(V_c),
                                         _ptr(len_c), _ptr(out_full), _ptr(out_comp), _ptr(err), _ptr(ref), _ptr(ws),
                                         ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "kvm_output_perturbation")


def kvm_merge_compact(p: KvmParams, K, V, set_start, pivot, out_len, K_out, V_out, out_size, ws, stream=None) -> None:
    _check(lib().kvm_merge_compact(ctypes.byref(p), _ptr(K), _ptr(V), _ptr(set_start), _ptr(pivot), _ptr(out_len),
                                   _ptr(K_out), _ptr(V_out), _ptr(out_size), _ptr(ws),
                                   ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "kvm_merge_compact")


def kvm_compress(p: KvmParams, Q, K, V, K_out, V_out, out_len, out_pos, scores_out, stats, ws, stream=None) -> None:
    _check(lib().kvm_compress(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(K_out), _ptr(V_out), _ptr(out_len),
                              _ptr(out_pos), _ptr(scores_out), _ptr(stats), _ptr(ws),
                              ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "kvm_compress")


def kvm_compress_with_lse(p: KvmParams, Q, K, V, lse_in, K_out, V_out, out_len, out_pos, scores_out, stats, ws,
                          stream=None) -> None:
    _check(lib().kvm_compress_with_lse(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lse_in), _ptr(K_out),
                                       _ptr(V_out), _ptr(out_len), _ptr(out_pos), _ptr(scores_out), _ptr(stats),
                                       _ptr(ws), ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "kvm_compress_with_lse")


def kvm_compress_host(p: KvmParams, Q, K, V, K_out, V_out, out_len, out_pos, dev, stream=None) -> None:
    """Q..out_pos are HOST tensors (pin them for asynchronous copies); `dev` is a device byte buffer."""
    _check(lib().kvm_compress_host(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(K_out), _ptr(V_out),
                                   _ptr(out_len), _ptr(out_pos), _ptr(dev),
                                   ctypes.c_size_t(dev.numel() * dev.element_size()), _stream(stream)),
           "kvm_compress_host")


# ----------------------------------------------------------------------------- convenience
def new_stats(device) -> torch.Tensor:
    """Zeroed device buffer laid out as `kvm_stats`."""
    return torch.zeros(ctypes.sizeof(KvmStats), dtype=torch.uint8, device=device)


def read_stats(buf: torch.Tensor) -> KvmStats:
    return KvmStats.from_buffer_copy(bytes(buf.cpu().numpy().tobytes()))


@dataclass
class Compressed:
    K_out: torch.Tensor
    V_out: torch.Tensor
    out_len: torch.Tensor
    out_pos: torch.Tensor
    scores: Optional[torch.Tensor]
    cap: int


class Compressor:
    """Owns the workspace and output buffers for one problem shape and calls kvm_compress."""

    def __init__(self, p: KvmParams, device="cuda", want_scores: bool = False):
        self.p = p
        self.cap, self.n_recent, self.n_heavy = kvm_sizes(p)
        U = p.batch * p.n_kv_heads
        dt = torch.bfloat16 if p.dtype == KVM_BF16 else torch.float32
        self.ws = torch.empty(kvm_workspace_bytes(p), dtype=torch.uint8, device=device)
        self.K_out = torch.zeros(p.batch, p.n_kv_heads, self.cap, p.head_dim, dtype=dt, device=device)
        self.V_out = torch.zeros_like(self.K_out)
        self.out_len = torch.zeros(U, dtype=torch.int32, device=device).view(p.batch, p.n_kv_heads)
        self.out_pos = torch.zeros(p.batch, p.n_kv_heads, self.cap, dtype=torch.int32, device=device)
        self.scores = (torch.empty(p.batch, p.n_kv_heads, p.seq, dtype=torch.float32, device=device)
                       if want_scores else None)

    def __call__(self, Q, K, V, stats=None, stream=None) -> Compressed:
        kvm_compress(self.p, Q, K, V, self.K_out, self.V_out, self.out_len, self.out_pos, self.scores, stats,
                     self.ws, stream)
        return Compressed(self.K_out, self.V_out, self.out_len, self.out_pos, self.scores, self.cap)


def compress_layers(p: KvmParams, layers, sim_thresholds=None, device="cuda", stream=None):
    """Compress a stack of layers, each an (Q, K, V) triple of CUDA tensors of the shape `p` describes, with one
    similarity threshold per layer (Section 3.2: thresholds chosen layer by layer), through kvm_compress_layers.
    Returns, per layer, a `Compressed` holding the outputs, and the layer's compression ratio mean(out_len) / S."""
    n = len(layers)
    comps = [Compressor(p, device=device) for _ in range(n)]
    ptrs = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    for Q, K, V in layers:
        assert Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()
    eps = None
    if sim_thresholds is not None:
        assert len(sim_thresholds) == n
        eps = (ctypes.c_float * n)(*[float(e) for e in sim_thresholds])
    ws = comps[0].ws
    _check(lib().kvm_compress_layers(ctypes.byref(p), ctypes.c_int32(n), eps, ptrs([l[0] for l in layers]),
                                     ptrs([l[1] for l in layers]), ptrs([l[2] for l in layers]),
                                     ptrs([c.K_out for c in comps]), ptrs([c.V_out for c in comps]),
                                     ptrs([c.out_len for c in comps]), ptrs([c.out_pos for c in comps]),
                                     ctypes.c_void_p(0), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(stream)),
           "kvm_compress_layers")
    out = [Compressed(c.K_out, c.V_out, c.out_len, c.out_pos, None, c.cap) for c in comps]
    ratios = [float(c.out_len.float().mean() / p.seq) for c in comps]
    return out, ratios
