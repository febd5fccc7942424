"""Shared machinery of the GPU parity tests: run the CUDA library through its C
ABI, run the fp64 CPU checker on the same inputs, and compare.

Bars (written here once, used by every parity test):
  * aggregated scores:  |gpu - ref| <= 1e-3 |ref| + 1e-6
  * merged K/V:         max_elem |gpu - ref| / max(|ref|, rowmax|ref| * 2^-6) <= 4e-3
  * set boundaries, pivots, output offsets: bit-exact.  Where floating point
    decides an integer both sides must decide on the same numbers, so the
    checker is run a second time on the library's own fp32 scores and
    similarities ("forced" chain) and the integers must match exactly on every
    unit.  Against the pure fp64 chain a unit may differ only if it contains a
    near-tie (similarity within 1e-3 of the effective threshold, or two scores
    within 1e-4 relative at the top-k cut or at a pivot); such units are
    counted and reported.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np
import torch

import paper_2407_08454_b200 as kvm
from oracle import kvmo

SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-6
KV_TOL = 4e-3
SIM_ATOL = 4e-6
NEAR_SIM, NEAR_SCORE = 1e-3, 1e-4


def f32(x: float) -> float:
    """The library's parameters are C floats: give the checker the same number."""
    return float(np.float32(x))


def preset(budget: float):
    return (0.17, 0.12) if f32(budget) >= f32(0.425) else (0.08, 0.02)


@dataclass
class Case:
    Q: torch.Tensor
    K: torch.Tensor
    V: torch.Tensor
    budget: float = 0.5
    recent: Optional[float] = None
    heavy: Optional[float] = None
    eps: float = 0.75
    sigma: float = 5.0
    scale: Optional[float] = None
    scale_v: bool = True
    enforce: bool = True
    pivot_rule: int = 0
    weight_rule: int = 0
    set_rule: int = 0
    pivot_key: Optional[torch.Tensor] = None      # [B,Hkv,S] fp32 (CPU) when pivot_rule is "key"

    def __post_init__(self):
        r, h = preset(self.budget)
        if self.recent is None:
            self.recent = r
        if self.heavy is None:
            self.heavy = h

    def params(self) -> kvm.KvmParams:
        B, Hq, S, D = self.Q.shape
        if self.pivot_key is not None and getattr(self, "_key_dev", None) is None:
            self._key_dev = self.pivot_key.float().contiguous().cuda()      # kept alive with the case
        return kvm.make_params(B, Hq, self.K.shape[1], S, D, self.Q.dtype, budget=self.budget,
                               recent_ratio=self.recent, heavy_ratio=self.heavy, sim_threshold=self.eps,
                               sigma=self.sigma, softmax_scale=self.scale or 0.0,
                               scale_v_by_set_size=int(self.scale_v), enforce_budget=int(self.enforce),
                               pivot_rule=self.pivot_rule, weight_rule=self.weight_rule, set_rule=self.set_rule,
                               pivot_key=getattr(self, "_key_dev", None))

    def oracle_scale(self) -> float:
        D = self.Q.shape[-1]
        return f32(self.scale) if self.scale else f32(1.0 / np.sqrt(np.float32(D)))


@dataclass
class GpuOut:
    scores: np.ndarray
    sim: np.ndarray
    set_id: np.ndarray
    set_start: np.ndarray
    pivot: np.ndarray
    out_len: np.ndarray
    K_out: np.ndarray
    V_out: np.ndarray
    out_size: np.ndarray
    c_out_len: np.ndarray
    c_out_pos: np.ndarray
    c_K_out: np.ndarray
    c_V_out: np.ndarray
    c_scores: np.ndarray
    stats: kvm.KvmStats
    cap: int


def run_gpu(case: Case, device="cuda") -> GpuOut:
    """Call every entry point once: the three steps one by one, then kvm_compress."""
    p = case.params()
    cap, n_r, n_h = kvm.kvm_sizes(p)
    B, Hq, S, D = case.Q.shape
    Hkv = case.K.shape[1]
    Q, K, V = (t.to(device).contiguous() for t in (case.Q, case.K, case.V))
    ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device=device)
    i32 = dict(dtype=torch.int32, device=device)
    scores = torch.full((B, Hkv, S), float("nan"), device=device)
    kvm.kvm_score(p, Q, K, None, scores, ws)
    sim = torch.full((B, Hkv, S), float("nan"), device=device)
    set_id = torch.full((B, Hkv, S), -7, **i32)
    set_start = torch.full((B, Hkv, cap + 1), -7, **i32)
    pivot = torch.full((B, Hkv, cap), -7, **i32)
    out_len = torch.full((B, Hkv), -7, **i32)
    stats = kvm.new_stats(device)
    kvm.kvm_segment(p, K, scores, set_id, set_start, pivot, out_len, sim, stats, ws)
    K_out = torch.full((B, Hkv, cap, D), 768.0, dtype=Q.dtype, device=device)
    V_out = torch.full_like(K_out, 768.0)
    out_size = torch.full((B, Hkv, cap), -7, **i32)
    kvm.kvm_merge_compact(p, K, V, set_start, pivot, out_len, K_out, V_out, out_size, ws)
    c_K = torch.full_like(K_out, 768.0)
    c_V = torch.full_like(K_out, 768.0)
    c_len = torch.full((B, Hkv), -7, **i32)
    c_pos = torch.full((B, Hkv, cap), -7, **i32)
    c_scores = torch.full((B, Hkv, S), float("nan"), device=device)
    kvm.kvm_compress(p, Q, K, V, c_K, c_V, c_len, c_pos, c_scores, None, ws)
    torch.cuda.synchronize()
    n = lambda t: t.float().cpu().numpy() if t.is_floating_point() else t.cpu().numpy()
    return GpuOut(n(scores), n(sim), n(set_id), n(set_start), n(pivot), n(out_len), n(K_out), n(V_out), n(out_size),
                  n(c_len), n(c_pos), n(c_K), n(c_V), n(c_scores), kvm.read_stats(stats), cap)


def score_excess(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max |gpu-ref| / (rtol |ref| + atol); parity holds when <= 1."""
    return float(np.max(np.abs(gpu.astype(np.float64) - ref) / (SCORE_RTOL * np.abs(ref) + SCORE_ATOL)))


def kv_error(gpu: np.ndarray, ref: np.ndarray) -> float:
    """Element-wise relative error with a per-row floor of rowmax * 2^-6."""
    ref = ref.astype(np.float64)
    floor = np.max(np.abs(ref), axis=-1, keepdims=True) * 2.0 ** -6
    den = np.maximum(np.abs(ref), floor)
    den[den == 0] = 1.0
    return float(np.max(np.abs(gpu.astype(np.float64) - ref) / den))


def _chain(case: Case, scores: np.ndarray, sim: np.ndarray, cap: int, n_r: int, n_h: int,
           key: Optional[np.ndarray] = None):
    keep = kvmo.keep(scores, n_r, n_h)
    b, fired = kvmo.boundaries(sim, keep, cap, f32(case.eps), case.enforce)
    set_id, set_start, out_len = kvmo.sets(b, cap)
    if case.pivot_rule == kvm.KVM_PIVOT_LAST:
        pivot = kvmo.pivots_last(set_start, out_len)
    else:
        pivot = kvmo.pivots(key if case.pivot_rule == kvm.KVM_PIVOT_KEY else scores, set_start, out_len)
    return dict(keep=keep, b=b, fired=fired, set_id=set_id, set_start=set_start, out_len=out_len, pivot=pivot)


def _near_tie_unit(case: Case, a: np.ndarray, c: np.ndarray, ch: Dict[str, np.ndarray], u, cap, n_r, n_h) -> bool:
    S = a.shape[-1]
    R = max(0, S - n_r)
    if 0 < n_h < R:
        srt = np.sort(a[:R])[::-1]
        if srt[n_h - 1] - srt[n_h] < NEAR_SCORE * srt[n_h - 1]:
            return True
    keep = ch["keep"][u]
    hard = keep.astype(bool).copy()
    hard[1:] |= keep[:-1].astype(bool)
    hard[0] = True
    eps_eff = f32(case.eps)
    if ch["fired"][u]:
        soft = np.sort(c[(~hard) & ~(c > eps_eff)])
        m = cap - int(hard.sum())
        if 0 < m < len(soft) and soft[m] - soft[m - 1] < NEAR_SIM:
            return True
        eps_eff = soft[m - 1] if m > 0 else -np.inf
    if np.any(np.abs(c[~hard] - f32(case.eps)) < NEAR_SIM):
        return True
    st, n = ch["set_start"][u], ch["out_len"][u]
    for s in range(n if case.pivot_rule == kvm.KVM_PIVOT_MAX_SCORE else 0):
        lo, hi = st[s], st[s + 1]
        if hi - lo >= 2:
            top = np.sort(a[lo:hi])[-2:]
            if top[1] - top[0] < NEAR_SCORE * top[1]:
                return True
    return False


@dataclass
class Report:
    score_excess: float = 0.0
    sim_err: float = 0.0
    k_err: float = 0.0
    v_err: float = 0.0
    units: int = 0
    units_differ_from_fp64_chain: int = 0
    units_near_tie: int = 0
    notes: list = field(default_factory=list)


def check_case(case: Case, g: Optional[GpuOut] = None, units: Optional[list] = None) -> Report:
    """Full parity check.  `units` (flat indices into [B*Hkv]) restricts the checker to a sample."""
    if g is None:
        g = run_gpu(case)
    B, Hq, S, D = case.Q.shape
    Hkv = case.K.shape[1]
    G = Hq // Hkv
    U = B * Hkv
    sel = list(range(U)) if units is None else list(units)
    p = case.params()
    cap, n_r, n_h = kvm.kvm_sizes(p)
    assert (cap, n_r, n_h) == _oracle_sizes(case, S)
    rep = Report(units=len(sel))

    def unit_view(x, tail):  # [B,Hkv,*tail] -> [U,*tail][sel]
        return x.reshape((U,) + tail)[sel]

    # inputs of the sampled units, as the checker wants them
    Qs = case.Q.reshape(U, G, S, D)[sel].reshape(len(sel), G, S, D)
    Ks = case.K.reshape(U, 1, S, D)[sel]
    Vs = case.V.reshape(U, 1, S, D)[sel]
    ref_scores = kvmo.scores(Qs, Ks, scale=case.oracle_scale())[:, 0]            # [n,S]
    ref_sim = kvmo.similarity(Ks[:, 0])                                         # [n,S]

    g_scores, g_sim = unit_view(g.scores, (S,)), unit_view(g.sim, (S,))
    rep.score_excess = score_excess(g_scores, ref_scores)
    assert rep.score_excess <= 1.0, f"scores off: {rep.score_excess:.3f} x tolerance"
    assert np.array_equal(unit_view(g.c_scores, (S,)), g_scores), "kvm_compress scores differ from kvm_score"
    rep.sim_err = float(np.max(np.abs(g_sim - ref_sim)))
    assert rep.sim_err <= SIM_ATOL, f"similarity off by {rep.sim_err}"

    # integers: forced chain (checker fed the library's own fp32 scores and similarities)
    key = None
    if case.pivot_key is not None:
        key = case.pivot_key.float().numpy().reshape(U, S)[sel].astype(np.float64)
    forced = _chain(case, g_scores.astype(np.float64), g_sim.astype(np.float64), cap, n_r, n_h, key)
    pure = _chain(case, ref_scores, ref_sim, cap, n_r, n_h, key)
    g_len = unit_view(g.out_len, ())
    g_st, g_pv, g_id = unit_view(g.set_start, (cap + 1,)), unit_view(g.pivot, (cap,)), unit_view(g.set_id, (S,))
    g_sz = unit_view(g.out_size, (cap,))
    assert np.array_equal(g_len, forced["out_len"]), "out_len differs from the forced chain"
    assert np.array_equal(g_id, forced["set_id"]), "set_id differs from the forced chain"
    for i in range(len(sel)):
        n = g_len[i]
        assert 1 <= n <= cap
        assert np.array_equal(g_st[i, : n + 1], forced["set_start"][i, : n + 1]), f"set_start, unit {sel[i]}"
        assert np.array_equal(g_pv[i, :n], forced["pivot"][i, :n]), f"pivot, unit {sel[i]}"
        assert np.array_equal(g_sz[i, :n], np.diff(g_st[i, : n + 1])), f"out_size, unit {sel[i]}"
        assert (g_st[i, n + 1:] == -7).all() and (g_pv[i, n:] == -7).all(), "wrote past out_len"
        same = (pure["out_len"][i] == n and np.array_equal(pure["set_start"][i, : n + 1], g_st[i, : n + 1])
                and np.array_equal(pure["pivot"][i, :n], g_pv[i, :n]))
        if not same:
            rep.units_differ_from_fp64_chain += 1
            assert _near_tie_unit(case, ref_scores[i], ref_sim[i], {k: v for k, v in pure.items()}, i, cap, n_r,
                                  n_h), f"unit {sel[i]} differs from the fp64 chain without a near-tie"
            rep.units_near_tie += 1
    # the device-side report of kvm_segment (all units only: it is a sum over the launch)
    if units is None and case.set_rule == kvm.KVM_SETS_ADJACENT:
        st_ = g.stats
        assert st_.status == 0
        assert (st_.min_out_len, st_.max_out_len, st_.sum_out_len) == (g_len.min(), g_len.max(), g_len.sum())
        assert st_.units_budget_rule == int(np.count_nonzero(forced["fired"]))
        near = np.abs(g_sim[:, 1:].astype(np.float32) - np.float32(case.eps)) < np.float32(1e-3)
        assert st_.near_threshold == int(near.sum())

    # kvm_compress must agree with the step-by-step calls bit for bit
    assert np.array_equal(unit_view(g.c_out_len, ()), g_len)
    c_pos, c_K, c_V = unit_view(g.c_out_pos, (cap,)), unit_view(g.c_K_out, (cap, D)), unit_view(g.c_V_out, (cap, D))
    g_K, g_V = unit_view(g.K_out, (cap, D)), unit_view(g.V_out, (cap, D))
    for i in range(len(sel)):
        n = g_len[i]
        assert np.array_equal(c_pos[i, :n], g_pv[i, :n])
        assert np.array_equal(c_K[i, :n], g_K[i, :n]) and np.array_equal(c_V[i, :n], g_V[i, :n])

    # merged states: checker with the library's integer decisions forced in
    rK, rV = kvmo.merge(Ks[:, 0], Vs[:, 0], g_st, np.where(g_pv < 0, 0, g_pv), g_len, f32(case.sigma), case.scale_v,
                        weight_rule=case.weight_rule)
    K32, V32 = Ks[:, 0].float().numpy(), Vs[:, 0].float().numpy()
    for i in range(len(sel)):
        n = g_len[i]
        rep.k_err = max(rep.k_err, kv_error(g_K[i, :n], rK[i, :n]))
        rep.v_err = max(rep.v_err, kv_error(g_V[i, :n], rV[i, :n]))
        assert (g_K[i, n:] == 768.0).all() and (g_V[i, n:] == 768.0).all(), "rows past out_len were written"
        single = np.nonzero(np.diff(g_st[i, : n + 1]) == 1)[0]
        assert np.array_equal(g_K[i, single], K32[i, g_st[i, single]]), "singleton rows must be bit-identical"
        assert np.array_equal(g_V[i, single], V32[i, g_st[i, single]])
        if case.weight_rule == kvm.KVM_WEIGHT_PIVOT_ONLY:      # the pivot's own rows, whatever the set size
            assert np.array_equal(g_K[i, :n], K32[i, g_pv[i, :n]])
            if not case.scale_v:
                assert np.array_equal(g_V[i, :n], V32[i, g_pv[i, :n]])
    assert rep.k_err <= KV_TOL, f"K_out error {rep.k_err}"
    assert rep.v_err <= KV_TOL, f"V_out error {rep.v_err}"
    return rep


def _oracle_sizes(case: Case, S: int):
    C, n_r, n_h = kvmo.sizes(S, f32(case.budget), f32(case.recent), f32(case.heavy))
    return (C if case.enforce else S), n_r, n_h


def check_invariants_all_units(case: Case, g: GpuOut) -> None:
    """Properties that hold at any size, checked on every unit."""
    B, Hq, S, D = case.Q.shape
    Hkv = case.K.shape[1]
    U = B * Hkv
    cap = g.cap
    lens = g.c_out_len.reshape(U)
    pos = g.c_out_pos.reshape(U, cap)
    assert (lens >= 1).all() and (lens <= cap).all()
    np.testing.assert_allclose(g.c_scores.reshape(U, S).sum(-1), S, rtol=2e-4)   # rows of the attention map sum to 1
    K32 = case.K.float().numpy().reshape(U, S, D)
    cK = g.c_K_out.reshape(U, cap, D)
    st = g.set_start.reshape(U, cap + 1)
    for u in range(U):
        n = lens[u]
        assert (np.diff(pos[u, :n]) > 0).all(), "out_pos must be strictly increasing"
        assert st[u, 0] == 0 and st[u, n] == S and (np.diff(st[u, : n + 1]) > 0).all()
        assert ((pos[u, :n] >= st[u, :n]) & (pos[u, :n] < st[u, 1: n + 1])).all(), "pivot outside its set"
        single = np.nonzero(np.diff(st[u, : n + 1]) == 1)[0]
        assert np.array_equal(cK[u, single], K32[u, st[u, single]])


def check_evict_case(case: Case, g: Optional[GpuOut] = None) -> Report:
    """Parity of the eviction mode (only the conserved tokens stay).  The floating-point part is the
    scores; given them every output is an integer or a copied row, so everything else is bit-exact
    against the checker fed the library's own scores."""
    assert case.set_rule == kvm.KVM_SETS_CONSERVED_ONLY
    if g is None:
        g = run_gpu(case)
    B, Hq, S, D = case.Q.shape
    Hkv = case.K.shape[1]
    G, U = Hq // Hkv, B * Hkv
    cap, n_r, n_h = kvm.kvm_sizes(case.params())
    assert (cap, n_r, n_h) == _oracle_sizes(case, S)
    rep = Report(units=U)
    Qs = case.Q.reshape(U, G, S, D)
    Ks, Vs = case.K.reshape(U, S, D), case.V.reshape(U, S, D)
    ref_scores = kvmo.scores(Qs, Ks[:, None], scale=case.oracle_scale())[:, 0]
    g_scores = g.scores.reshape(U, S)
    rep.score_excess = score_excess(g_scores, ref_scores)
    assert rep.score_excess <= 1.0
    keep_forced = kvmo.keep(g_scores.astype(np.float64), n_r, n_h)
    keep_pure = kvmo.keep(ref_scores, n_r, n_h)
    r_len, r_pos, rK, rV = kvmo.evict(keep_forced, Ks, Vs, cap)
    g_len, g_pv = g.out_len.reshape(U), g.pivot.reshape(U, cap)
    g_st, g_id = g.set_start.reshape(U, cap + 1), g.set_id.reshape(U, S)
    assert np.array_equal(g_len, r_len) and (g_len == min(S, n_r) + min(n_h, max(0, S - n_r))).all()
    for name, step, comp in (("K", g.K_out, g.c_K_out), ("V", g.V_out, g.c_V_out)):
        ref = rK if name == "K" else rV
        step, comp = step.reshape(U, cap, D), comp.reshape(U, cap, D)
        for u in range(U):
            n = g_len[u]
            assert np.array_equal(step[u, :n].astype(np.float64), ref[u, :n]), f"{name}_out rows, unit {u}"
            assert np.array_equal(comp[u, :n], step[u, :n])
            assert (step[u, n:] == 768.0).all() and (comp[u, n:] == 768.0).all()
    for u in range(U):
        n = g_len[u]
        assert np.array_equal(g_pv[u, :n], r_pos[u, :n]) and (g_pv[u, n:] == -7).all()
        assert np.array_equal(g_st[u, :n], r_pos[u, :n]) and g_st[u, n] == S
        kf = keep_forced[u].astype(np.int64)
        want_id = np.where(kf != 0, np.cumsum(kf) - 1, -1)
        assert np.array_equal(g_id[u], want_id)
        assert np.array_equal(g.out_size.reshape(U, cap)[u, :n], np.ones(n, np.int32))
        assert np.array_equal(g.c_out_pos.reshape(U, cap)[u, :n], r_pos[u, :n])
        if not np.array_equal(keep_forced[u], keep_pure[u]):
            rep.units_differ_from_fp64_chain += 1
            R = max(0, S - n_r)
            srt = np.sort(ref_scores[u, :R])[::-1]
            assert srt[n_h - 1] - srt[n_h] < NEAR_SCORE * srt[n_h - 1], f"unit {u}: kept set differs without a near-tie"
            rep.units_near_tie += 1
    assert np.array_equal(g.c_out_len.reshape(U), g_len)
    return rep
