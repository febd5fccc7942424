"""TEST INFRASTRUCTURE -- ctypes loader for the fp64 CPU checker in kvmo.cpp.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It never touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvmo.cpp")
_LIB = os.path.join(_HERE, "libkvmo.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile kvmo.cpp into libkvmo.so next to it (g++ with OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c++17", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.kvmo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().kvmo_num_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(x) -> np.ndarray:
    """Storage-dtype tensor/array -> contiguous fp32 numpy array (exact for bf16 and fp32)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def sizes(S: int, budget: float, recent: float, heavy: float):
    C, nr, nh = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    lib().kvmo_sizes(ctypes.c_int32(S), ctypes.c_double(budget), ctypes.c_double(recent), ctypes.c_double(heavy),
                     ctypes.byref(C), ctypes.byref(nr), ctypes.byref(nh))
    return C.value, nr.value, nh.value


def scores(Q, K, scale: Optional[float] = None, want_lse: bool = False):
    Q, K = _f32(Q), _f32(K)
    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    a = np.empty((B, Hkv, S), dtype=np.float64)
    lse = np.empty((B, Hq, S), dtype=np.float64) if want_lse else None
    lib().kvmo_scores(ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(S),
                      ctypes.c_int32(D), ctypes.c_double(scale), _p(Q), _p(K), _p(a), _p(lse))
    return (a, lse) if want_lse else a


def keep(scores_: np.ndarray, n_r: int, n_h: int) -> np.ndarray:
    a = np.ascontiguousarray(scores_, dtype=np.float64)
    S = a.shape[-1]
    U = a.size // S
    out = np.empty(a.shape, dtype=np.uint8)
    lib().kvmo_keep(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(n_r), ctypes.c_int32(n_h), _p(a), _p(out))
    return out


def similarity(K) -> np.ndarray:
    K = _f32(K)
    S, D = K.shape[-2:]
    U = K.size // (S * D)
    out = np.empty(K.shape[:-1], dtype=np.float64)
    lib().kvmo_similarity(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(D), _p(K), _p(out))
    return out


def boundaries(sim: np.ndarray, keep_: np.ndarray, C: int, eps: float, enforce_budget: bool = True):
    sim = np.ascontiguousarray(sim, dtype=np.float64)
    keep_ = np.ascontiguousarray(keep_, dtype=np.uint8)
    S = sim.shape[-1]
    U = sim.size // S
    b = np.empty(sim.shape, dtype=np.uint8)
    fired = np.empty(sim.shape[:-1], dtype=np.int32)
    lib().kvmo_boundaries(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(C), ctypes.c_double(eps),
                          ctypes.c_int32(1 if enforce_budget else 0), _p(sim), _p(keep_), _p(b), _p(fired))
    return b, fired


def layer_ratio(sim: np.ndarray, eps: float) -> np.ndarray:
    sim = np.ascontiguousarray(sim, dtype=np.float64)
    S = sim.shape[-1]
    U = sim.size // S
    out = np.empty(sim.shape[:-1], dtype=np.float64)
    lib().kvmo_layer_ratio(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_double(eps), _p(sim), _p(out))
    return out


def boundaries_anchor(K, keep_: np.ndarray, eps: float, want_run: bool = False, run_in=None):
    """Anchor reading of the set identification (Section 3.2): flags [.., S], and the run length of every token.
    With `run_in` the walk uses those run lengths instead of evaluating cosines."""
    K = _f32(K)
    keep_ = np.ascontiguousarray(keep_, dtype=np.uint8)
    S, D = K.shape[-2:]
    U = K.size // (S * D)
    b = np.empty(K.shape[:-1], dtype=np.uint8)
    run = np.empty(K.shape[:-1], dtype=np.int32) if want_run else None
    lib().kvmo_boundaries_anchor(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(D), ctypes.c_double(eps),
                                 _p(K), _p(keep_), _p(b), _p(run),
                                 _p(None if run_in is None else np.ascontiguousarray(run_in, dtype=np.int32)))
    return (b, run) if want_run else b


def sets(b: np.ndarray, cap: int):
    b = np.ascontiguousarray(b, dtype=np.uint8)
    S = b.shape[-1]
    U = b.size // S
    lead = b.shape[:-1]
    set_id = np.empty(b.shape, dtype=np.int32)
    set_start = np.full(lead + (cap + 1,), -1, dtype=np.int32)
    out_len = np.empty(lead, dtype=np.int32)
    lib().kvmo_sets(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(cap), _p(b), _p(set_id), _p(set_start),
                    _p(out_len))
    return set_id, set_start, out_len


def pivots(scores_: np.ndarray, set_start: np.ndarray, out_len: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(scores_, dtype=np.float64)
    set_start = np.ascontiguousarray(set_start, dtype=np.int32)
    out_len = np.ascontiguousarray(out_len, dtype=np.int32)
    S = a.shape[-1]
    U = a.size // S
    cap = set_start.shape[-1] - 1
    pv = np.full(a.shape[:-1] + (cap,), -1, dtype=np.int32)
    lib().kvmo_pivots(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(cap), _p(a), _p(set_start), _p(out_len),
                      _p(pv))
    return pv


def pivots_last(set_start: np.ndarray, out_len: np.ndarray) -> np.ndarray:
    set_start = np.ascontiguousarray(set_start, dtype=np.int32)
    out_len = np.ascontiguousarray(out_len, dtype=np.int32)
    cap = set_start.shape[-1] - 1
    U = out_len.size
    pv = np.full(out_len.shape + (cap,), -1, dtype=np.int32)
    lib().kvmo_pivots_last(ctypes.c_int64(U), ctypes.c_int32(cap), _p(set_start), _p(out_len), _p(pv))
    return pv


def evict(keep_: np.ndarray, K, V, cap: int):
    K, V = _f32(K), _f32(V)
    keep_ = np.ascontiguousarray(keep_, dtype=np.uint8)
    S, D = K.shape[-2:]
    U = K.size // (S * D)
    lead = K.shape[:-2]
    out_len = np.empty(lead, np.int32)
    out_pos = np.full(lead + (cap,), -1, np.int32)
    Ko = np.full(lead + (cap, D), np.nan, dtype=np.float64)
    Vo = np.full(lead + (cap, D), np.nan, dtype=np.float64)
    lib().kvmo_evict(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(D), ctypes.c_int32(cap), _p(keep_),
                     _p(K), _p(V), _p(out_len), _p(out_pos), _p(Ko), _p(Vo))
    return out_len, out_pos, Ko, Vo


PIVOT_MAX_SCORE, PIVOT_LAST, PIVOT_KEY = 0, 1, 2
WEIGHT_GAUSSIAN, WEIGHT_AVERAGE, WEIGHT_PIVOT_ONLY, WEIGHT_SET_SIGMA = 0, 1, 2, 3
SETS_ADJACENT, SETS_CONSERVED_ONLY, SETS_ANCHOR = 0, 1, 2


def merge(K, V, set_start, pivot, out_len, sigma: float, scale_v: bool = True, want_weights: bool = False,
          weight_rule: int = 0):
    K, V = _f32(K), _f32(V)
    set_start = np.ascontiguousarray(set_start, dtype=np.int32)
    pivot = np.ascontiguousarray(pivot, dtype=np.int32)
    out_len = np.ascontiguousarray(out_len, dtype=np.int32)
    S, D = K.shape[-2:]
    U = K.size // (S * D)
    cap = set_start.shape[-1] - 1
    lead = K.shape[:-2]
    Ko = np.full(lead + (cap, D), np.nan, dtype=np.float64)
    Vo = np.full(lead + (cap, D), np.nan, dtype=np.float64)
    w = np.full(lead + (S,), np.nan, dtype=np.float64) if want_weights else None
    lib().kvmo_merge(ctypes.c_int64(U), ctypes.c_int32(S), ctypes.c_int32(D), ctypes.c_int32(cap),
                     ctypes.c_double(sigma), ctypes.c_int32(1 if scale_v else 0), ctypes.c_int32(weight_rule),
                     _p(K), _p(V), _p(set_start),
                     _p(pivot), _p(out_len), _p(Ko), _p(Vo), _p(w))
    return (Ko, Vo, w) if want_weights else (Ko, Vo)


def attend(q, K, V, length=None, scale: Optional[float] = None) -> np.ndarray:
    """One decode step (Eq. 1): q [B,Hq,D], K/V [B,Hkv,rows,D], length [B,Hkv] or None -> O [B,Hq,D] fp64."""
    q, K, V = _f32(q), _f32(K), _f32(V)
    B, Hq, D = q.shape
    Hkv, rows = K.shape[1], K.shape[2]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if length is not None:
        length = np.ascontiguousarray(length, dtype=np.int32)
        assert length.size == B * Hkv
    out = np.empty((B, Hq, D), dtype=np.float64)
    lib().kvmo_attend(ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(rows),
                      ctypes.c_int32(D), ctypes.c_double(scale), _p(q), _p(K), _p(V), _p(length), _p(out))
    return out


def prefill_attend(Q, K, V, scale: Optional[float] = None):
    """Causal attention over the whole prompt (Eq. 1 for every position): Q [B,Hq,S,D], K/V [B,Hkv,S,D] ->
    O [B,Hq,S,D] fp64 and the rows' natural-log log-sum-exp [B,Hq,S]."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    out = np.empty((B, Hq, S, D), dtype=np.float64)
    lse = np.empty((B, Hq, S), dtype=np.float64)
    lib().kvmo_prefill_attend(ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(S),
                              ctypes.c_int32(D), ctypes.c_double(scale), _p(Q), _p(K), _p(V), _p(out), _p(lse))
    return out, lse


def perturbation(O: np.ndarray, O_star: np.ndarray):
    """Definition 2.1's |O_t - O_t*| per head (Euclidean norm) and |O_t|."""
    O = np.ascontiguousarray(O, dtype=np.float64)
    O_star = np.ascontiguousarray(O_star, dtype=np.float64)
    D = O.shape[-1]
    n = O.size // D
    err = np.empty(O.shape[:-1], dtype=np.float64)
    ref = np.empty(O.shape[:-1], dtype=np.float64)
    lib().kvmo_perturbation(ctypes.c_int64(n), ctypes.c_int32(D), _p(O), _p(O_star), _p(err), _p(ref))
    return err, ref


@dataclass
class Compressed:
    scores: np.ndarray
    keep: np.ndarray
    sim: np.ndarray
    b: np.ndarray
    set_id: np.ndarray
    set_start: np.ndarray
    out_len: np.ndarray
    pivot: np.ndarray
    K_out: np.ndarray
    V_out: np.ndarray
    cap: int
    n_r: int
    n_h: int


def compress(Q, K, V, budget: float, recent: float, heavy: float, eps: float = 0.75, sigma: float = 5.0,
             scale: Optional[float] = None, scale_v: bool = True, enforce_budget: bool = True,
             pivot_rule: int = 0, weight_rule: int = 0, set_rule: int = 0, pivot_key=None) -> Compressed:
    """All steps for one layer through the single C entry point kvmo_compress."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    C, n_r, n_h = sizes(S, budget, recent, heavy)
    cap = C if enforce_budget else S
    lead = (B, Hkv)
    if pivot_key is not None:
        pivot_key = np.ascontiguousarray(pivot_key, dtype=np.float64)
        assert pivot_key.shape == lead + (S,)
    assert (pivot_rule == PIVOT_KEY) == (pivot_key is not None)
    r = Compressed(
        scores=np.empty(lead + (S,), np.float64), keep=np.empty(lead + (S,), np.uint8),
        sim=np.empty(lead + (S,), np.float64), b=np.empty(lead + (S,), np.uint8),
        set_id=np.empty(lead + (S,), np.int32), set_start=np.full(lead + (cap + 1,), -1, np.int32),
        out_len=np.empty(lead, np.int32), pivot=np.full(lead + (cap,), -1, np.int32),
        K_out=np.full(lead + (cap, D), np.nan, np.float64), V_out=np.full(lead + (cap, D), np.nan, np.float64),
        cap=cap, n_r=n_r, n_h=n_h)
    lib().kvmo_compress(ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(S),
                        ctypes.c_int32(D), ctypes.c_double(scale), ctypes.c_int32(cap), ctypes.c_int32(n_r),
                        ctypes.c_int32(n_h), ctypes.c_double(eps), ctypes.c_double(sigma),
                        ctypes.c_int32(1 if scale_v else 0), ctypes.c_int32(1 if enforce_budget else 0),
                        ctypes.c_int32(pivot_rule), ctypes.c_int32(weight_rule), ctypes.c_int32(set_rule),
                        _p(pivot_key), _p(Q), _p(K), _p(V), _p(r.scores), _p(r.keep), _p(r.sim), _p(r.b), _p(r.set_id),
                        _p(r.set_start), _p(r.out_len), _p(r.pivot), _p(r.K_out), _p(r.V_out))
    return r
