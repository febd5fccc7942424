"""Pins for the CPU checker's attention-score and conserved-set steps (Eq. 1,
Algorithm 2's aggregated score, Eq. 6, the GQA mean of Section 5.2, and the
top-k / recent rule of Sections 4.1-4.2).  Everything here compares the checker
with closed forms, invariants or library routines, never with itself."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import kvmo

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _dense_scores(Q, K, scale):
    """Textbook route: full S x S logits, library softmax on the causal part."""
    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hkv, S))
    lse = np.zeros((B, Hq, S))
    mask = np.tril(np.ones((S, S), dtype=bool))
    for b in range(B):
        for h in range(Hq):
            logits = scale * (Q[b, h].astype(np.float64) @ K[b, h // G].astype(np.float64).T)
            logits = np.where(mask, logits, -np.inf)
            A = softmax(logits, axis=1)
            out[b, h // G] += A.sum(axis=0) / G
            lse[b, h] = logsumexp(logits, axis=1)
    return out, lse


def test_uniform_rows_match_harmonic_golden():
    # Q = 0 makes every causal row uniform: a_j = H_S - H_j.
    rows = [l.split() for l in open(os.path.join(GOLDEN, "harmonic_scores_S12.txt")) if not l.startswith("#")]
    S = len(rows)
    Q = np.zeros((1, 1, S, 8), np.float32)
    K = _rand((1, 1, S, 8), 1)
    a = kvmo.scores(Q, K)
    want = np.array([float(Fraction(r[1])) for r in rows])
    np.testing.assert_allclose(a[0, 0], want, rtol=1e-14)
    # identical keys (any Q) give the same map
    K2 = np.repeat(_rand((1, 1, 1, 8), 2), S, axis=2)
    np.testing.assert_allclose(kvmo.scores(_rand((1, 1, S, 8), 3), K2)[0, 0], want, rtol=1e-12)


def test_single_token_and_row_sum_invariant():
    assert kvmo.scores(_rand((1, 1, 1, 4), 0), _rand((1, 1, 1, 4), 1))[0, 0, 0] == 1.0
    Q, K = _rand((2, 6, 37, 16), 4), _rand((2, 3, 37, 16), 5)
    a = kvmo.scores(Q, K, scale=0.7)
    np.testing.assert_allclose(a.sum(-1), 37.0, rtol=1e-12)  # rows of A sum to 1
    assert (a[..., 0] >= 1.0 - 1e-12).all()  # key 0 gets all of row 0
    assert (a > 0).all()


def test_matches_dense_library_softmax_with_gqa_and_scale():
    Q, K = _rand((2, 4, 23, 8), 6) * 2.0, _rand((2, 2, 23, 8), 7)
    for scale in (1.0 / math.sqrt(8), 0.3):
        a, lse = kvmo.scores(Q, K, scale=scale, want_lse=True)
        wa, wl = _dense_scores(Q, K, scale)
        np.testing.assert_allclose(a, wa, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(lse, wl, rtol=1e-12, atol=1e-12)


def test_sharp_diagonal_attention_gives_unit_scores():
    # orthogonal one-hot keys, q_i = beta k_i: A -> I, so every a_j -> 1
    S = 9
    K = np.eye(S, dtype=np.float32)[None, None]
    a = kvmo.scores(60.0 * K, K, scale=1.0)
    np.testing.assert_allclose(a[0, 0], 1.0, atol=1e-20 + S * math.exp(-60.0))


def test_identical_query_heads_equal_single_head():
    q, K = _rand((1, 1, 19, 8), 8), _rand((1, 1, 19, 8), 9)
    a1 = kvmo.scores(q, K)
    a4 = kvmo.scores(np.repeat(q, 4, axis=1), K)
    np.testing.assert_allclose(a4, a1, rtol=1e-13)


def test_two_token_closed_form_is_causal_and_not_transposed():
    # S = 2: a_0 = 1 + 1/(1+e^{s11-s10}), a_1 = 1/(1+e^{s10-s11}); s uses q_1 only.
    Q = np.array([[[[1.0, 0.0], [0.5, 2.0]]]], np.float32)
    K = np.array([[[[3.0, 1.0], [-1.0, 0.25]]]], np.float32)
    s10 = 0.5 * 3.0 + 2.0 * 1.0
    s11 = 0.5 * -1.0 + 2.0 * 0.25
    a = kvmo.scores(Q, K, scale=1.0)[0, 0]
    assert a[0] == pytest.approx(1.0 + 1.0 / (1.0 + math.exp(s11 - s10)), rel=1e-14)
    assert a[1] == pytest.approx(1.0 / (1.0 + math.exp(s10 - s11)), rel=1e-14)


def test_sizes_follow_the_paper_presets():
    # Section 5.1: 50% -> recent 0.17, heavy 0.12; 35% -> 0.08, 0.02 (fractions of S)
    assert kvmo.sizes(4096, 0.50, 0.17, 0.12) == (2048, 696, 491)
    assert kvmo.sizes(4096, 0.35, 0.08, 0.02) == (1433, 327, 81)
    assert kvmo.sizes(512, 0.50, 0.17, 0.12) == (256, 87, 61)
    assert kvmo.sizes(32768, 0.50, 0.17, 0.12) == (16384, 5570, 3932)


def test_keep_is_recent_window_plus_sorted_top_k():
    rng = np.random.default_rng(11)
    for S, n_r, n_h in [(40, 7, 5), (16, 0, 3), (16, 4, 0), (9, 9, 2), (12, 3, 20)]:
        a = rng.random((3, S))
        a[0, 2] = a[0, 5] = a[0, 1] = 0.99  # ties: lower index wins
        kp = kvmo.keep(a, n_r, n_h)
        R = max(0, S - n_r)
        for u in range(3):
            order = np.argsort(-a[u, :R], kind="stable")[: min(n_h, R)]
            want = np.zeros(S, np.uint8)
            want[R:] = 1
            want[order] = 1
            np.testing.assert_array_equal(kp[u], want)
            assert kp[u].sum() == min(S, n_r) + min(n_h, R)


def test_keep_tie_break_prefers_lower_index():
    a = np.array([[0.5, 0.9, 0.9, 0.9, 0.1, 0.2]])
    np.testing.assert_array_equal(kvmo.keep(a, 1, 2)[0], [0, 1, 1, 0, 0, 1])
