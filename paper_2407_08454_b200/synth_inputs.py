"""Seeded synthetic Q/K/V generators for KV-cache compression workloads.

This module only draws random tensors.  It contains none of the compression
method's arithmetic (no softmax, no similarity, no merging) so that it can feed
both the CUDA library and the CPU checker without coupling them.

The shapes and the statistical structure follow what the KVMerger paper reports
about real prefill caches (Section 3.1): key states of neighbouring tokens are
strongly similar, value states are not.  Keys and queries are therefore AR(1)
processes over the token axis, independent per channel, multiplied by a
per-channel log-normal scale (optionally with a few large "outlier" channels);
values are iid standard normal.

Every (layer, tensor, batch entry, head) has its own Philox stream, so any
subset of units can be generated on its own and is identical to the same units
of a full generation.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Iterable, Optional, Sequence

import numpy as np
import torch
from numpy.random import Generator, Philox
from scipy.signal import lfilter

# tensor ids for the stream key
_T_Q, _T_K, _T_V, _T_SCALE_Q, _T_SCALE_K, _T_OUTLIER, _T_RHO, _T_SWITCH = range(8)


@dataclass(frozen=True)
class WorkloadConfig:
    """One synthetic workload (a model-shaped stack of attention layers)."""

    name: str
    layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq: int
    dtype: str  # "bf16" | "f32"
    budget: float
    seed: int
    rho: float = 0.95
    rho_range: Optional[Sequence[float]] = None  # per-layer rho ~ U[lo, hi]
    n_outlier_channels: int = 0
    outlier_gain: float = 10.0
    regime_switch_p: float = 0.0  # keys restart from N(0,1) with this probability per token
    logit_std: float = 4.0  # target std of q.k/sqrt(D); <= 0 leaves Q unscaled

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def scaled(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, WorkloadConfig] = {
    # Tiny fp32 case the CPU checker finishes in well under a second.
    "C0": WorkloadConfig("C0-tiny", 1, 1, 4, 4, 64, 512, "f32", 0.50, seed=0),
    # One Llama2-7B-shaped layer, 4k tokens.
    "C1": WorkloadConfig("C1-llama2-7b-layer", 1, 1, 32, 32, 128, 4096, "bf16", 0.50, seed=1,
                         n_outlier_channels=2),
    # Llama2-7B-shaped full cache, batch 4, per-layer rho.
    "C2": WorkloadConfig("C2-llama2-7b-full", 32, 4, 32, 32, 128, 4096, "bf16", 0.35, seed=2,
                         rho_range=(0.85, 0.98), n_outlier_channels=2),
    # Mistral-7B-shaped GQA, 32k tokens.
    "C3": WorkloadConfig("C3-mistral-7b-gqa", 32, 1, 32, 8, 128, 32768, "bf16", 0.50, seed=3),
    # Llama2-13B-shaped, keys with regime switches (many short runs).
    "C4": WorkloadConfig("C4-llama2-13b", 40, 8, 40, 40, 128, 4096, "bf16", 0.35, seed=4,
                         n_outlier_channels=2, regime_switch_p=1.0 / 64.0),
}


def _rng(seed: int, layer: int, tensor: int, b: int = 0, head: int = 0) -> Generator:
    k0 = (int(seed) << 32) | (int(layer) & 0xFFFFFFFF)
    k1 = (int(tensor) << 48) | ((int(b) & 0xFFFFFF) << 24) | (int(head) & 0xFFFFFF)
    return Generator(Philox(key=[k0, k1]))


def layer_rho(cfg: WorkloadConfig, layer: int) -> float:
    if cfg.rho_range is None:
        return cfg.rho
    lo, hi = cfg.rho_range
    return float(_rng(cfg.seed, layer, _T_RHO).uniform(lo, hi))


def _ar1(eps: np.ndarray, rho: float) -> np.ndarray:
    """x_0 = eps_0, x_t = rho x_{t-1} + sqrt(1-rho^2) eps_t along axis 0."""
    u = eps * math.sqrt(max(0.0, 1.0 - rho * rho))
    u[0] = eps[0]
    return lfilter([1.0], [1.0, -rho], u, axis=0)


def _ar1_with_restarts(eps: np.ndarray, rho: float, restart: np.ndarray) -> np.ndarray:
    """AR(1) whose state is redrawn from N(0,1) (all channels) where restart[t]."""
    S = eps.shape[0]
    starts = [0] + [int(t) for t in np.nonzero(restart)[0] if t > 0] + [S]
    out = np.empty_like(eps)
    for a, b in zip(starts[:-1], starts[1:]):
        if b > a:
            out[a:b] = _ar1(eps[a:b].copy(), rho)
    return out


def channel_scales(cfg: WorkloadConfig, layer: int, kv_head: int, q_head: Optional[int]) -> np.ndarray:
    """Per-channel multiplier: exp(0.5 z), times the outlier gain on the KV head's outlier channels."""
    if q_head is None:
        z = _rng(cfg.seed, layer, _T_SCALE_K, 0, kv_head).standard_normal(cfg.head_dim)
    else:
        z = _rng(cfg.seed, layer, _T_SCALE_Q, 0, q_head).standard_normal(cfg.head_dim)
    s = np.exp(0.5 * z)
    if cfg.n_outlier_channels > 0:
        ch = _rng(cfg.seed, layer, _T_OUTLIER, 0, kv_head).permutation(cfg.head_dim)[: cfg.n_outlier_channels]
        s[ch] *= cfg.outlier_gain
    return s


def _to_storage(x: np.ndarray, cfg: WorkloadConfig) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(cfg.torch_dtype)  # round-to-nearest-even for bf16


def make_layer(cfg: WorkloadConfig, layer: int = 0, batch_entries: Optional[Iterable[int]] = None,
               kv_heads: Optional[Iterable[int]] = None) -> Dict[str, torch.Tensor]:
    """Generate Q, K, V of one layer on the CPU in the storage dtype.

    Returns tensors shaped [len(batch_entries), heads, seq, head_dim]; when
    `kv_heads` is given only those KV heads (and their query groups, in order)
    are produced.
    """
    bs = list(range(cfg.batch)) if batch_entries is None else list(batch_entries)
    hs = list(range(cfg.n_kv_heads)) if kv_heads is None else list(kv_heads)
    G, S, D = cfg.group, cfg.seq, cfg.head_dim
    rho = layer_rho(cfg, layer)
    c = 1.0 / math.sqrt(D)
    Q = np.empty((len(bs), len(hs) * G, S, D), dtype=np.float32)
    K = np.empty((len(bs), len(hs), S, D), dtype=np.float32)
    V = np.empty((len(bs), len(hs), S, D), dtype=np.float32)
    for hi, h in enumerate(hs):
        sk = channel_scales(cfg, layer, h, None)
        for bi, b in enumerate(bs):
            eps = _rng(cfg.seed, layer, _T_K, b, h).standard_normal((S, D))
            if cfg.regime_switch_p > 0.0:
                restart = _rng(cfg.seed, layer, _T_SWITCH, b, h).random(S) < cfg.regime_switch_p
                x = _ar1_with_restarts(eps, rho, restart)
            else:
                x = _ar1(eps, rho)
            K[bi, hi] = x * sk
            V[bi, hi] = _rng(cfg.seed, layer, _T_V, b, h).standard_normal((S, D))
        for g in range(G):
            qh = h * G + g
            sq = channel_scales(cfg, layer, h, qh)
            gamma = 1.0
            if cfg.logit_std > 0.0:
                # q and k are independent with unit-variance marginals per channel,
                # so var(q.k/sqrt(D)) = sum_ch (sq*sk)^2 / D.
                gamma = cfg.logit_std / (c * math.sqrt(float(np.sum((sq * sk) ** 2))))
            for bi, b in enumerate(bs):
                eps = _rng(cfg.seed, layer, _T_Q, b, qh).standard_normal((S, D))
                Q[bi, hi * G + g] = _ar1(eps, rho) * (sq * gamma)
    return {"Q": _to_storage(Q, cfg), "K": _to_storage(K, cfg), "V": _to_storage(V, cfg)}


def config_by_name(name: str) -> WorkloadConfig:
    return CONFIGS[name]
