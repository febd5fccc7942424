"""Pins for the CPU checker's variants of the method: the average-weighted
baseline with last-index pivots (Section 4.2), pivots by a caller-supplied key
(the random-pivot ablation of Section 5.3), the pivot-only limit named after
Eq. 5, and eviction of everything but the conserved tokens (Section 2.2).
Library routines, limits of the pinned Gaussian merge, and invariants only."""
import numpy as np
import pytest

from oracle import kvmo
from paper_2407_08454_b200 import synth_inputs as si


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _random_partition(S, U, seed, p=0.3):
    b = (np.random.default_rng(seed).random((U, S)) < p).astype(np.uint8)
    b[:, 0] = 1
    return kvmo.sets(b, cap=S)


def test_last_index_pivot_is_the_set_maximum_index():
    set_id, st, ol = _random_partition(80, 3, 0)
    pv = kvmo.pivots_last(st, ol)
    for u in range(3):
        for s in range(ol[u]):
            members = np.nonzero(set_id[u] == s)[0]
            assert pv[u, s] == members.max()
        assert (pv[u, ol[u]:] == -1).all()
    # same thing as an arg-max whose key grows with the index
    np.testing.assert_array_equal(pv, kvmo.pivots(np.tile(np.arange(80.0), (3, 1)), st, ol))


def test_key_pivot_is_uniform_over_the_set_for_iid_keys():
    # one set of 5 tokens, many independent draws: every member is chosen about equally often
    n, trials = 5, 4000
    b = np.zeros((trials, n), np.uint8)
    b[:, 0] = 1
    _, st, ol = kvmo.sets(b, cap=n)
    key = np.random.default_rng(1).random((trials, n))
    pv = kvmo.pivots(key, st, ol)[:, 0]
    np.testing.assert_array_equal(pv, key.argmax(1))
    counts = np.bincount(pv, minlength=n)
    chi2 = ((counts - trials / n) ** 2 / (trials / n)).sum()
    assert chi2 < 18.5          # 99.9 % point of chi-square with 4 degrees of freedom


def test_average_rule_is_the_library_mean():
    K, V = _rand((2, 50, 6), 2), _rand((2, 50, 6), 3)
    set_id, st, ol = _random_partition(50, 2, 4)
    pv = kvmo.pivots_last(st, ol)
    Ko, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma=5.0, scale_v=False, want_weights=True,
                           weight_rule=kvmo.WEIGHT_AVERAGE)
    Ks, Vs, _ = kvmo.merge(K, V, st, pv, ol, sigma=5.0, scale_v=True, want_weights=True,
                           weight_rule=kvmo.WEIGHT_AVERAGE)
    for u in range(2):
        for s in range(ol[u]):
            m = set_id[u] == s
            np.testing.assert_allclose(Ko[u, s], K[u, m].astype(np.float64).mean(0), rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(Vo[u, s], V[u, m].astype(np.float64).mean(0), rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(Vs[u, s], V[u, m].astype(np.float64).sum(0), rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(w[u, m], 1.0 / m.sum(), rtol=1e-15)
    np.testing.assert_array_equal(Ks[0, :ol[0]], Ko[0, :ol[0]])    # keys never carry the set size
    # and it is the Gaussian rule's sigma -> infinity limit, whatever the pivot
    Kg, Vg = kvmo.merge(K, V, st, kvmo.pivots(_rand((2, 50), 5), st, ol), ol, sigma=1e9, scale_v=False)
    np.testing.assert_allclose(Kg[0, :ol[0]], Ko[0, :ol[0]], rtol=1e-12, atol=1e-14)


def test_pivot_only_rule_copies_the_pivot_rows():
    K, V = _rand((2, 40, 5), 6), _rand((2, 40, 5), 7)
    set_id, st, ol = _random_partition(40, 2, 8)
    pv = kvmo.pivots(_rand((2, 40), 9), st, ol)
    Ko, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma=5.0, scale_v=False, want_weights=True,
                           weight_rule=kvmo.WEIGHT_PIVOT_ONLY)
    for u in range(2):
        n = ol[u]
        np.testing.assert_array_equal(Ko[u, :n], K[u, pv[u, :n]].astype(np.float64))
        np.testing.assert_array_equal(Vo[u, :n], V[u, pv[u, :n]].astype(np.float64))
        assert w[u].sum() == n and set(np.unique(w[u])) <= {0.0, 1.0}
    # the Gaussian rule tends to it as sigma -> 0 (distinct keys)
    Kg, Vg = kvmo.merge(K, V, st, pv, ol, sigma=1e-3, scale_v=False)
    np.testing.assert_allclose(Kg[0, :ol[0]], Ko[0, :ol[0]], rtol=1e-12)
    # with the set-size factor the value row is the pivot's value times the set size
    _, Vs = kvmo.merge(K, V, st, pv, ol, sigma=5.0, scale_v=True, weight_rule=kvmo.WEIGHT_PIVOT_ONLY)
    sizes = np.diff(st[0, :ol[0] + 1])
    np.testing.assert_array_equal(Vs[0, :ol[0]], Vo[0, :ol[0]] * sizes[:, None])


def test_eviction_keeps_exactly_the_conserved_rows_in_order():
    rng = np.random.default_rng(10)
    K, V = _rand((3, 30, 4), 11), _rand((3, 30, 4), 12)
    a = rng.random((3, 30))
    keep = kvmo.keep(a, 6, 5)
    ol, pos, Ko, Vo = kvmo.evict(keep, K, V, cap=11)
    for u in range(3):
        idx = np.nonzero(keep[u])[0]                       # numpy's own gather is the definition
        assert ol[u] == len(idx) == 11
        np.testing.assert_array_equal(pos[u], idx)
        np.testing.assert_array_equal(Ko[u], K[u, idx].astype(np.float64))
        np.testing.assert_array_equal(Vo[u], V[u, idx].astype(np.float64))
        # heavy hitters: every kept non-recent score is at least every dropped score
        old = idx[idx < 24]
        dropped = np.setdiff1d(np.arange(24), old)
        assert a[u, old].min() >= a[u, dropped].max()
    # nothing conserved -> nothing kept; everything conserved -> the cache itself
    ol, pos, Ko, Vo = kvmo.evict(np.zeros((1, 30), np.uint8), K[:1], V[:1], cap=4)
    assert ol[0] == 0 and (pos == -1).all() and np.isnan(Ko).all()
    ol, pos, Ko, Vo = kvmo.evict(np.ones((1, 30), np.uint8), K[:1], V[:1], cap=30)
    np.testing.assert_array_equal(Ko[0], K[0].astype(np.float64))


def test_compress_variants_equal_their_steps():
    cfg = si.CONFIGS["C0"]
    d = si.make_layer(cfg)
    base = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12)
    S, U = cfg.seq, cfg.n_kv_heads
    key = np.random.default_rng(13).random((1, U, S))
    # average-weighted baseline: same sets as the method, last-index pivots, plain means
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12, scale_v=False,
                      pivot_rule=kvmo.PIVOT_LAST, weight_rule=kvmo.WEIGHT_AVERAGE)
    np.testing.assert_array_equal(r.set_start, base.set_start)
    np.testing.assert_array_equal(r.pivot, kvmo.pivots_last(base.set_start, base.out_len))
    Ko, Vo = kvmo.merge(d["K"], d["V"], base.set_start, r.pivot, base.out_len, 5.0, scale_v=False,
                        weight_rule=kvmo.WEIGHT_AVERAGE)
    np.testing.assert_array_equal(r.K_out, Ko)
    # keyed pivots: sets unchanged, conserved tokens still their own pivot, pivots differ somewhere
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12, pivot_rule=kvmo.PIVOT_KEY, pivot_key=key)
    np.testing.assert_array_equal(r.set_start, base.set_start)
    np.testing.assert_array_equal(r.pivot, kvmo.pivots(key, base.set_start, base.out_len))
    assert (r.pivot != base.pivot).any()
    for u in range(U):
        kept = np.nonzero(base.keep[0, u])[0]
        np.testing.assert_array_equal(r.pivot[0, u, base.set_id[0, u, kept]], kept)
    # eviction with the heavy share filling the budget: exactly cap rows, all of them input rows
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.50 - 0.17, set_rule=kvmo.SETS_CONSERVED_ONLY)
    K64 = d["K"].double().numpy()
    for u in range(U):
        n = r.out_len[0, u]
        assert n == r.n_r + r.n_h and n <= r.cap
        idx = np.nonzero(r.keep[0, u])[0]
        np.testing.assert_array_equal(r.pivot[0, u, :n], idx)
        np.testing.assert_array_equal(r.K_out[0, u, :n], K64[0, u, idx])
        assert (r.set_id[0, u, idx] == np.arange(n)).all() and (np.delete(r.set_id[0, u], idx) == -1).all()


def test_layer_ratio_walk_equals_flag_count_and_limits():
    # the backward walk of Section 3.2 and the forward boundary flags of Algorithm 1 count the same groups
    rng = np.random.default_rng(14)
    sim = rng.uniform(0.4, 1.0, (5, 300))
    sim[:, 0] = 0
    none = np.zeros((5, 300), np.uint8)
    for eps in (0.5, 0.75, 0.9):
        b, _ = kvmo.boundaries(sim, none, C=300, eps=eps, enforce_budget=False)
        np.testing.assert_array_equal(kvmo.layer_ratio(sim, eps), b.sum(-1) / 300.0)
    r = [kvmo.layer_ratio(sim, e).mean() for e in np.linspace(0.3, 1.0, 15)]
    assert all(x <= y for x, y in zip(r, r[1:]))                         # lower threshold -> fewer groups
    ident = np.repeat(_rand((1, 1, 8), 15), 40, axis=1)
    assert kvmo.layer_ratio(kvmo.similarity(ident), 0.75)[0] == 1 / 40  # one group
    assert kvmo.layer_ratio(kvmo.similarity(np.eye(8, dtype=np.float32)[None]), 0.75)[0] == 1.0
    # brute force on a hand-made row: similar pairs (1,2), (2,3) and (5,6) -> groups {0},{1,2,3},{4},{5,6}
    row = np.array([[0.0, 0.1, 0.9, 0.8, 0.2, 0.3, 0.99]])
    assert kvmo.layer_ratio(row, 0.75)[0] == 4 / 7


def test_layer_ratio_of_wide_ar1_keys_is_a_step_in_rho():
    # for many channels the cosine of AR(1) neighbours concentrates at rho: all in one group below it, none above
    rng = np.random.default_rng(16)
    S, D, rho = 64, 8192, 0.9
    x = np.empty((S, D))
    x[0] = rng.standard_normal(D)
    for t in range(1, S):
        x[t] = rho * x[t - 1] + np.sqrt(1 - rho * rho) * rng.standard_normal(D)
    sim = kvmo.similarity(x[None].astype(np.float32))
    assert np.abs(sim[0, 1:] - rho).max() < 0.02
    assert kvmo.layer_ratio(sim, rho - 0.05)[0] == 1 / S
    assert kvmo.layer_ratio(sim, rho + 0.05)[0] == 1.0


# ---------------------------------------------------------------- anchor reading of the set identification
def _cos(a, b):
    a, b = a.astype(np.float64), b.astype(np.float64)
    na, nb = np.linalg.norm(a), np.linalg.norm(b)
    return float(a @ b / (na * nb)) if na > 0 and nb > 0 else 0.0


def test_anchor_grouping_is_the_unique_partition_with_its_defining_properties():
    # Walking from the last token, the result is fixed by: every member is similar to its group's LAST token;
    # the token before a group is not (or is conserved, or does not exist); conserved tokens stand alone.
    rng = np.random.default_rng(20)
    for trial in range(20):
        S, D = int(rng.integers(3, 40)), 3
        x = np.cumsum(rng.standard_normal((1, S, D)) * 0.35, axis=1).astype(np.float32) + 1.0   # slowly turning keys
        keep = (rng.random((1, S)) < 0.15).astype(np.uint8)
        eps = float(rng.uniform(0.5, 0.95))
        b, run = kvmo.boundaries_anchor(x, keep, eps, want_run=True)
        assert b[0, 0] == 1
        starts = np.nonzero(b[0])[0]
        ends = np.append(starts[1:], S) - 1
        for lo, hi in zip(starts, ends):
            if keep[0, lo:hi + 1].any():
                assert lo == hi
                continue
            assert all(_cos(x[0, hi], x[0, j]) > eps for j in range(lo, hi))
            assert lo == 0 or keep[0, lo - 1] or not (_cos(x[0, hi], x[0, lo - 1]) > eps)
        np.testing.assert_array_equal(kvmo.boundaries_anchor(x, keep, eps, run_in=run), b)   # integer-only walk
        for i in range(S):                      # run lengths: brute force over every anchor candidate
            r = 0
            while i - 1 - r >= 0 and _cos(x[0, i], x[0, i - 1 - r]) > eps:
                r += 1
            assert run[0, i] == r


def test_anchor_and_neighbour_readings_differ_exactly_where_they_should():
    def unit(deg):
        t = np.deg2rad(np.array(deg, dtype=np.float64))
        return np.stack([np.cos(t), np.sin(t)], -1)[None].astype(np.float32)
    none = np.zeros((1, 3), np.uint8)
    # keys turning by 25 degrees per token: neighbours are similar (cos 25 = 0.906) so Algorithm 1's neighbour
    # reading chains all three, but token 0 is 50 degrees from the last token (cos 50 = 0.643 < 0.75)
    K = unit([0, 25, 50])
    np.testing.assert_array_equal(kvmo.boundaries_anchor(K, none, 0.75)[0], [1, 1, 0])
    b_adj, _ = kvmo.boundaries(kvmo.similarity(K), none, C=3, eps=0.75)
    np.testing.assert_array_equal(b_adj[0], [1, 0, 0])
    # when every state within a neighbour-run is also similar to the run's last state, the readings agree
    K = unit([0, 5, 10, 80, 85, 170])
    none = np.zeros((1, 6), np.uint8)
    b_adj, _ = kvmo.boundaries(kvmo.similarity(K), none, C=6, eps=0.75)
    np.testing.assert_array_equal(kvmo.boundaries_anchor(K, none, 0.75)[0], b_adj[0])
    np.testing.assert_array_equal(b_adj[0], [1, 0, 0, 1, 0, 1])
    # limits: identical keys -> one group; orthogonal keys -> singletons; a conserved token splits the run
    ident = np.repeat(_rand((1, 1, 8), 21), 9, axis=1)
    assert kvmo.boundaries_anchor(ident, np.zeros((1, 9), np.uint8), 0.75).sum() == 1
    assert kvmo.boundaries_anchor(np.eye(8, dtype=np.float32)[None], np.zeros((1, 8), np.uint8), 0.75).sum() == 8
    keep = np.zeros((1, 9), np.uint8)
    keep[0, 4] = 1
    np.testing.assert_array_equal(kvmo.boundaries_anchor(ident, keep, 0.75)[0], [1, 0, 0, 0, 1, 1, 0, 0, 0])
    # the number of groups never falls when the threshold rises
    K = np.cumsum(_rand((1, 200, 4), 22) * 0.3, axis=1) + 1.0
    n = [kvmo.boundaries_anchor(K, np.zeros((1, 200), np.uint8), e).sum() for e in np.linspace(0.0, 0.99, 12)]
    assert n[0] <= n[-1] and n[-1] > n[0]


def test_compress_with_anchor_sets_equals_its_steps():
    cfg = si.CONFIGS["C0"]
    d = si.make_layer(cfg)
    r = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12, enforce_budget=False, set_rule=kvmo.SETS_ANCHOR)
    b = kvmo.boundaries_anchor(d["K"], r.keep, 0.75)
    np.testing.assert_array_equal(b, r.b)
    set_id, st, ol = kvmo.sets(b, cap=cfg.seq)
    np.testing.assert_array_equal(ol, r.out_len)
    np.testing.assert_array_equal(kvmo.pivots(r.scores, st, ol), r.pivot)
    base = kvmo.compress(d["Q"], d["K"], d["V"], 0.50, 0.17, 0.12, enforce_budget=False)
    assert (r.out_len >= base.out_len).all()        # similarity to the anchor is the stricter requirement here


# ---------------------------------------------------------------- bandwidth per merging set (a reading of Eq. 4)
def test_set_sigma_rule_is_the_fixed_rule_at_the_set_own_bandwidth():
    K, V = _rand((1, 60, 6), 30), _rand((1, 60, 6), 31)
    set_id, st, ol = _random_partition(60, 1, 32)
    pv = kvmo.pivots(_rand((1, 60), 33), st, ol)
    Ko, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma=123.0, scale_v=False, want_weights=True,
                           weight_rule=kvmo.WEIGHT_SET_SIGMA)          # sigma is ignored
    K64 = K.astype(np.float64)
    for s in range(ol[0]):
        lo, hi, p = st[0, s], st[0, s + 1], pv[0, s]
        d2 = ((K64[0, lo:hi] - K64[0, p]) ** 2).sum(-1)
        if hi - lo == 1:
            np.testing.assert_array_equal(Ko[0, s], K64[0, lo])
            continue
        sigma_s = np.sqrt(d2.mean() / 2.0)
        one = (np.array([[0, hi - lo]], np.int32), np.array([[p - lo]], np.int32), np.array([1], np.int32))
        Kf, Vf, wf = kvmo.merge(K[:, lo:hi], V[:, lo:hi], *one, sigma=sigma_s, scale_v=False, want_weights=True)
        np.testing.assert_allclose(Ko[0, s], Kf[0, 0], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(w[0, lo:hi], wf[0], rtol=1e-12)
        np.testing.assert_allclose(np.log(w[0, lo:hi] / w[0, p]), -d2 / d2.mean(), rtol=1e-10, atol=1e-12)


def test_set_sigma_rule_closed_forms_and_scale_invariance():
    # two tokens: mean squared distance = d^2 / 2, so the other token's kernel value is exp(-2) whatever d is
    for d in (0.1, 3.0, 50.0):
        K = np.array([[[0.0, 0.0], [d, 0.0]]], np.float32)
        V = np.array([[[1.0, 0.0], [0.0, 1.0]]], np.float32)
        st, pv, ol = np.array([[0, 2]], np.int32), np.array([[0]], np.int32), np.array([1], np.int32)
        _, Vo, w = kvmo.merge(K, V, st, pv, ol, sigma=5.0, scale_v=False, want_weights=True,
                              weight_rule=kvmo.WEIGHT_SET_SIGMA)
        g = np.exp(-2.0)
        np.testing.assert_allclose(w[0], [1 / (1 + g), g / (1 + g)], rtol=1e-14)
    # identical keys: every kernel value is 1 -> uniform weights
    K = np.repeat(_rand((1, 1, 4), 34), 5, axis=1)
    st, pv, ol = np.array([[0, 5]], np.int32), np.array([[2]], np.int32), np.array([1], np.int32)
    _, _, w = kvmo.merge(K, _rand((1, 5, 4), 35), st, pv, ol, 5.0, want_weights=True, weight_rule=kvmo.WEIGHT_SET_SIGMA)
    np.testing.assert_allclose(w[0], 0.2, rtol=1e-15)
    # rescaling all keys leaves the weights unchanged (the fixed-sigma rule does not have this property)
    K, V = _rand((1, 9, 4), 36), _rand((1, 9, 4), 37)
    st, pv, ol = np.array([[0, 9]], np.int32), np.array([[4]], np.int32), np.array([1], np.int32)
    w1 = kvmo.merge(K, V, st, pv, ol, 5.0, want_weights=True, weight_rule=kvmo.WEIGHT_SET_SIGMA)[2]
    w2 = kvmo.merge(4 * K, V, st, pv, ol, 5.0, want_weights=True, weight_rule=kvmo.WEIGHT_SET_SIGMA)[2]
    np.testing.assert_allclose(w2, w1, rtol=1e-12)
    f1 = kvmo.merge(K, V, st, pv, ol, 5.0, want_weights=True)[2]
    f2 = kvmo.merge(4 * K, V, st, pv, ol, 5.0, want_weights=True)[2]
    assert np.abs(f2 - f1).max() > 1e-3
