"""Pins for the CPU checker's Gaussian-kernel weighted merge (Eq. 4, Eq. 5,
Definition 4.2, Algorithm 2) and for the end-to-end chain.  Closed forms,
limits and invariants only."""
import math

import numpy as np
import pytest

from oracle import kvmo
from paper_2407_08454_b200 import synth_inputs as si


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _one_set(n, pivot, cap=None):
    cap = cap or 1
    st = np.full((1, cap + 1), -1, np.int32)
    st[0, 0], st[0, 1] = 0, n
    return st, np.array([[pivot] + [-1] * (cap - 1)], np.int32), np.array([1], np.int32)


def test_two_token_closed_form():
    # w_p = 1/(1+g), w_i = g/(1+g), g = exp(-|dk|^2 / (2 sigma^2))
    K = np.array([[[1.0, 2.0, 0.0], [2.0, 0.0, 1.0]]], np.float32)
    V = np.array([[[4.0, -1.0, 0.5], [0.0, 3.0, 2.0]]], np.float32)
    sigma = 1.7
    g = math.exp(-(1.0 + 4.0 + 1.0) / (2 * sigma * sigma))
    for p in (0, 1):
        st, pv, ol = _one_set(2, p)
        Ko, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma, scale_v=True, want_weights=True)
        wp, wi = 1 / (1 + g), g / (1 + g)
        K, V = K.astype(np.float64), V.astype(np.float64)
        want_w = [wp, wi] if p == 0 else [wi, wp]
        np.testing.assert_allclose(w[0], want_w, rtol=1e-14)
        np.testing.assert_allclose(Ko[0, 0], want_w[0] * K[0, 0] + want_w[1] * K[0, 1], rtol=1e-14)
        # values: same weights, times |S_v| = 2; keys are NOT scaled
        np.testing.assert_allclose(Vo[0, 0], 2 * (want_w[0] * V[0, 0] + want_w[1] * V[0, 1]), rtol=1e-14)
        Ko2, Vo2 = kvmo.merge(K, V, st, pv, ol, sigma, scale_v=False)
        np.testing.assert_allclose(Vo2[0, 0], Vo[0, 0] / 2, rtol=1e-14)
        np.testing.assert_allclose(Ko2, Ko, rtol=0)


def test_weights_positive_normalised_and_pivot_largest():
    K, V = _rand((1, 13, 6), 1), _rand((1, 13, 6), 2)
    st, pv, ol = _one_set(13, 4)
    Ko, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma=2.0, want_weights=True)
    assert (w > 0).all() and w.sum() == pytest.approx(1.0, rel=1e-14)
    assert np.argmax(w[0]) == 4
    # merged key is a convex combination of the set's keys
    assert (Ko[0, 0] >= K[0].min(0) - 1e-12).all() and (Ko[0, 0] <= K[0].max(0) + 1e-12).all()
    # weights are the normalised Gaussian of the distance to the pivot: ratios fix them
    d2 = ((K[0].astype(np.float64) - K[0, 4].astype(np.float64)) ** 2).sum(-1)
    np.testing.assert_allclose(np.log(w[0] / w[0, 4]), -d2 / 8.0, rtol=1e-12, atol=1e-12)


def test_singletons_pass_through_exactly():
    K, V = _rand((1, 5, 4), 3), _rand((1, 5, 4), 4)
    st = np.arange(6, dtype=np.int32)[None]
    pv = np.arange(5, dtype=np.int32)[None]
    Ko, Vo = kvmo.merge(K, V, st, pv, np.array([5], np.int32), sigma=5.0)
    np.testing.assert_array_equal(Ko[0], K[0].astype(np.float64))
    np.testing.assert_array_equal(Vo[0], V[0].astype(np.float64))


def test_identical_keys_and_identical_values():
    k = _rand((1, 1, 5), 5)
    K = np.repeat(k, 7, axis=1)
    V = _rand((1, 7, 5), 6)
    st, pv, ol = _one_set(7, 3)
    Ko, Vo = kvmo.merge(K, V, st, pv, ol, sigma=0.5)
    np.testing.assert_allclose(Ko[0, 0], k[0, 0].astype(np.float64), rtol=1e-15)               # merges to that key
    np.testing.assert_allclose(Vo[0, 0], 7 * V[0].astype(np.float64).mean(0), rtol=1e-13)
    Vsame = np.repeat(_rand((1, 1, 5), 7), 7, axis=1)
    Ko, Vo = kvmo.merge(_rand((1, 7, 5), 8), Vsame, st, pv, ol, sigma=3.0)
    np.testing.assert_allclose(Vo[0, 0], 7 * Vsame[0, 0].astype(np.float64), rtol=1e-13)        # V weights times |S_v|


def test_sigma_limits():
    K, V = _rand((1, 6, 4), 9), _rand((1, 6, 4), 10)
    st, pv, ol = _one_set(6, 2)
    Ko, Vo = kvmo.merge(K, V, st, pv, ol, sigma=1e9, scale_v=False)         # uniform average
    np.testing.assert_allclose(Ko[0, 0], K[0].astype(np.float64).mean(0), rtol=1e-12)
    np.testing.assert_allclose(Vo[0, 0], V[0].astype(np.float64).mean(0), rtol=1e-12)
    Ko, Vo = kvmo.merge(K, V, st, pv, ol, sigma=1e-3, scale_v=False)        # pivot alone
    np.testing.assert_allclose(Ko[0, 0], K[0, 2].astype(np.float64), rtol=1e-12)
    np.testing.assert_allclose(Vo[0, 0], V[0, 2].astype(np.float64), rtol=1e-12)


def test_compress_chain_on_tiny_config():
    cfg = si.CONFIGS["C0"]
    d = si.make_layer(cfg)
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12, eps=0.75, sigma=5.0)
    S, C = cfg.seq, r.cap
    assert (C, r.n_r, r.n_h) == (256, 87, 61)
    K64, V64 = d["K"].double().numpy(), d["V"].double().numpy()
    for u in range(cfg.n_kv_heads):
        n = r.out_len[0, u]
        assert 1 <= n <= C                                                   # within budget
        assert r.keep[0, u].sum() == r.n_r + r.n_h
        pv = r.pivot[0, u, :n]
        assert (np.diff(pv) > 0).all()
        kept = np.nonzero(r.keep[0, u])[0]
        rows = r.set_id[0, u, kept]
        np.testing.assert_array_equal(r.pivot[0, u, rows], kept)             # conserved tokens are their own pivot
        np.testing.assert_array_equal(r.K_out[0, u, rows], K64[0, u, kept])  # and are stored unchanged
        np.testing.assert_array_equal(r.V_out[0, u, rows], V64[0, u, kept])
    # the chain equals its steps called one by one
    a = kvmo.scores(d["Q"], d["K"])
    np.testing.assert_array_equal(a, r.scores)
    kp = kvmo.keep(a, r.n_r, r.n_h)
    b, _ = kvmo.boundaries(kvmo.similarity(d["K"]), kp, C, 0.75)
    np.testing.assert_array_equal(b, r.b)
    # threshold above 1 and no budget: the output is the input cache
    r2 = kvmo.compress(d["Q"], d["K"], d["V"], 1.0, 0.0, 0.0, eps=1.5, enforce_budget=False)
    assert (r2.out_len == S).all()
    np.testing.assert_array_equal(r2.K_out, K64)
    np.testing.assert_array_equal(r2.V_out, V64)


def test_generator_is_seeded_and_sliceable():
    cfg = si.CONFIGS["C1"].scaled(seq=64, n_q_heads=4, n_kv_heads=2)
    full = si.make_layer(cfg, layer=3)
    again = si.make_layer(cfg, layer=3)
    part = si.make_layer(cfg, layer=3, kv_heads=[1])
    for t in ("Q", "K", "V"):
        assert (full[t] == again[t]).all()
    assert (part["K"][:, 0] == full["K"][:, 1]).all()
    assert (part["Q"][:, 0:2] == full["Q"][:, 2:4]).all()
    other = si.make_layer(cfg, layer=4)
    assert not (other["K"] == full["K"]).all()
