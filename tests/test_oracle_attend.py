"""Pins for the CPU checker's decode-step attention (Eq. 1) and the output
perturbation of Definition 2.1: library softmax, closed forms, and the
properties the compression path must have (no merging -> no perturbation)."""
import math

import numpy as np
import pytest
from scipy.special import softmax

from oracle import kvmo
from paper_2407_08454_b200 import synth_inputs as si


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def test_attend_matches_library_softmax_with_gqa_lengths_and_scale():
    B, Hq, Hkv, rows, D = 2, 6, 3, 17, 8
    q, K, V = _rand((B, Hq, D), 0), _rand((B, Hkv, rows, D), 1), _rand((B, Hkv, rows, D), 2)
    length = np.array([[17, 5, 1], [9, 17, 3]], np.int32)
    for scale in (None, 0.37):
        out = kvmo.attend(q, K, V, length, scale)
        sc = scale if scale is not None else 1 / math.sqrt(D)
        for b in range(B):
            for h in range(Hq):
                g = h // 2                                  # query heads 2g, 2g+1 share KV head g
                n = length[b, g]
                a = softmax(sc * (K[b, g, :n].astype(np.float64) @ q[b, h].astype(np.float64)))
                np.testing.assert_allclose(out[b, h], a @ V[b, g, :n].astype(np.float64), rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(kvmo.attend(q, K, V, None), kvmo.attend(q, K, V, np.full((B, Hkv), rows)))


def test_attend_closed_forms():
    D = 4
    q = _rand((1, 1, D), 3)
    K, V = _rand((1, 1, 6, D), 4), _rand((1, 1, 6, D), 5)
    # one row: the output is that value row; no rows: zero
    np.testing.assert_array_equal(kvmo.attend(q, K, V, [1])[0, 0], V[0, 0, 0].astype(np.float64))
    assert (kvmo.attend(q, K, V, [0]) == 0).all()
    # identical keys: uniform attention -> mean of the values
    Ks = np.repeat(K[:, :, :1], 6, axis=2)
    np.testing.assert_allclose(kvmo.attend(q, Ks, V)[0, 0], V[0, 0].astype(np.float64).mean(0), rtol=1e-13)
    # two rows: logistic weights, and the key (not the value) decides them
    k2 = np.array([[[[1.0, 0, 0, 0], [0, 2.0, 0, 0]]]], np.float32)
    v2 = np.array([[[[1.0, 0, 0, 0], [0, 0, 0, 5.0]]]], np.float32)
    qq = np.array([[[3.0, 1.0, 0, 0]]], np.float32)
    w1 = 1 / (1 + math.exp(3.0 - 2.0))                      # scale = 1: s0 = 3, s1 = 2
    np.testing.assert_allclose(kvmo.attend(qq, k2, v2, scale=1.0)[0, 0], [1 - w1, 0, 0, 5 * w1], rtol=1e-14)
    # a sharply matching key returns its value
    big = kvmo.attend(40 * K[:, :, 2], K, V, scale=1.0)
    np.testing.assert_allclose(big[0, 0], V[0, 0, 2], atol=1e-6)
    # adding a constant vector to all keys shifts every logit equally: no change
    np.testing.assert_allclose(kvmo.attend(q, K + 0.5 * np.ones(D, np.float32), V), kvmo.attend(q, K, V), rtol=1e-5)


def test_perturbation_is_the_euclidean_norm():
    O, P = _rand((3, 2, 5), 6).astype(np.float64), _rand((3, 2, 5), 7).astype(np.float64)
    err, ref = kvmo.perturbation(O, P)
    np.testing.assert_allclose(err, np.linalg.norm(O - P, axis=-1), rtol=1e-14)
    np.testing.assert_allclose(ref, np.linalg.norm(O, axis=-1), rtol=1e-14)
    assert (kvmo.perturbation(O, O)[0] == 0).all()


def test_no_merging_means_no_perturbation_and_merging_perturbs():
    cfg = si.CONFIGS["C0"]
    d = si.make_layer(cfg)
    qt = d["Q"][:, :, -1]                                    # the most recent query as the decode-step query
    full = kvmo.attend(qt, d["K"], d["V"])
    r = kvmo.compress(d["Q"], d["K"], d["V"], 1.0, 0.0, 0.0, eps=1.5, enforce_budget=False)
    same = kvmo.attend(qt, r.K_out, r.V_out, r.out_len)
    assert (kvmo.perturbation(full, same)[0] == 0).all()
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.5, 0.17, 0.12, scale_v=False)
    err, ref = kvmo.perturbation(full, kvmo.attend(qt, r.K_out, r.V_out, r.out_len))
    assert (err > 0).all() and (err < 2 * ref).all()
    # a cache in which every merged state has one member merged with an exact copy of itself: unchanged keys,
    # doubled softmax mass is NOT restored by the value scaling alone, so the exact invariant is the unscaled one
    K2 = np.repeat(d["K"].numpy()[:, :, :32], 2, axis=2)     # tokens 0,0,1,1,...
    V2 = np.repeat(d["V"].numpy()[:, :, :32], 2, axis=2)
    st = np.tile(np.arange(0, 65, 2, dtype=np.int32), (1, 4, 1))
    pv = st[..., :-1].copy()
    Ko, Vo = kvmo.merge(K2, V2, st, pv, np.full((1, 4), 32, np.int32), sigma=5.0, scale_v=False)
    np.testing.assert_allclose(kvmo.attend(qt, Ko, Vo), kvmo.attend(qt, K2, V2), rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- causal attention over the whole prompt (Eq. 1)
def test_prefill_attend_matches_library_softmax_row_by_row_with_gqa_and_scale():
    from scipy.special import logsumexp
    B, Hq, Hkv, S, D = 2, 4, 2, 13, 8
    Q, K, V = _rand((B, Hq, S, D), 20), _rand((B, Hkv, S, D), 21), _rand((B, Hkv, S, D), 22)
    for scale in (None, 0.61):
        O, lse = kvmo.prefill_attend(Q, K, V, scale)
        sc = scale if scale is not None else 1 / math.sqrt(D)
        for b in range(B):
            for h in range(Hq):
                g = h // 2
                for i in range(S):
                    logits = sc * (K[b, g, :i + 1].astype(np.float64) @ Q[b, h, i].astype(np.float64))
                    np.testing.assert_allclose(O[b, h, i], softmax(logits) @ V[b, g, :i + 1].astype(np.float64),
                                               rtol=1e-12, atol=1e-14)
                    np.testing.assert_allclose(lse[b, h, i], logsumexp(logits), rtol=1e-13)


def test_prefill_attend_invariants_and_its_links_to_the_other_steps():
    B, Hq, Hkv, S, D = 1, 4, 2, 21, 8
    Q, K, V = _rand((B, Hq, S, D), 23), _rand((B, Hkv, S, D), 24), _rand((B, Hkv, S, D), 25)
    O, lse = kvmo.prefill_attend(Q, K, V)
    # the first position sees only itself: its output is the first value row, its log-sum-exp its own logit
    for h in range(Hq):
        np.testing.assert_array_equal(O[0, h, 0], V[0, h // 2, 0].astype(np.float64))
        np.testing.assert_allclose(lse[0, h, 0], (Q[0, h, 0].astype(np.float64) @ K[0, h // 2, 0]) / math.sqrt(D),
                                   rtol=1e-14)
    # rows of the attention map sum to one: constant values come back unchanged; outputs lie in the values' hull
    ones = np.ones_like(V)
    np.testing.assert_allclose(kvmo.prefill_attend(Q, K, ones)[0], 1.0, rtol=1e-13)
    Vd = V.astype(np.float64)
    for h in range(Hq):
        for i in range(S):
            assert (O[0, h, i] <= Vd[0, h // 2, :i + 1].max(0) + 1e-12).all()
            assert (O[0, h, i] >= Vd[0, h // 2, :i + 1].min(0) - 1e-12).all()
    # the last position is the decode step over the whole cache, and the log-sum-exp is the one the score step uses
    np.testing.assert_allclose(O[:, :, -1], kvmo.attend(Q[:, :, -1], K, V), rtol=1e-12, atol=1e-14)
    _, lse_scores = kvmo.scores(Q, K, want_lse=True)
    np.testing.assert_allclose(lse, lse_scores, rtol=1e-13)
    # a future token never matters: changing the last key and value leaves every earlier row as it was
    K2, V2 = K.copy(), V.copy()
    K2[:, :, -1] += 3.0
    V2[:, :, -1] -= 2.0
    O2, lse2 = kvmo.prefill_attend(Q, K2, V2)
    np.testing.assert_array_equal(O2[:, :, :-1], O[:, :, :-1])
    np.testing.assert_array_equal(lse2[:, :, :-1], lse[:, :, :-1])
    assert not np.allclose(O2[:, :, -1], O[:, :, -1])
