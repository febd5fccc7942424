"""Pins for the CPU checker's similarity, merging-set, and pivot steps (Eq. 2,
Algorithm 1 / Definition 4.1, Eq. 6).  Brute force, invariants and library
routines only."""
import itertools

import numpy as np
import pytest
from scipy.spatial.distance import cosine as scipy_cosine_distance

from oracle import kvmo


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


# ---------------------------------------------------------------- similarity
def test_similarity_matches_library_cosine_and_index_convention():
    K = _rand((2, 11, 6), 0)
    sim = kvmo.similarity(K)
    assert (sim[:, 0] == 0).all()
    for u in range(2):
        for j in range(1, 11):  # sim_j pairs token j with its LEFT neighbour
            want = 1.0 - scipy_cosine_distance(K[u, j - 1].astype(np.float64), K[u, j].astype(np.float64))
            assert sim[u, j] == pytest.approx(want, abs=1e-14)


def test_similarity_special_cases():
    K = np.zeros((1, 6, 4), np.float32)
    K[0, 0] = [1, 0, 0, 0]
    K[0, 1] = [3, 0, 0, 0]      # parallel -> 1
    K[0, 2] = [0, 2, 0, 0]      # orthogonal -> 0
    K[0, 3] = [0, -5, 0, 0]     # opposite -> -1
    K[0, 4] = [0, 0, 0, 0]      # zero norm -> 0 by convention
    K[0, 5] = [1, 1, 0, 0]
    np.testing.assert_allclose(kvmo.similarity(K)[0], [0, 1, 0, -1, 0, 0], atol=1e-15)
    # invariant to positive per-token rescaling
    K = _rand((1, 9, 5), 1)
    s = np.random.default_rng(2).random((1, 9, 1)).astype(np.float32) * 4 + 0.5
    np.testing.assert_allclose(kvmo.similarity(K * s), kvmo.similarity(K), atol=1e-6)


# ---------------------------------------------------------------- merging sets
def _partition_from_flags(b):
    starts = [j for j in range(len(b)) if b[j]]
    return tuple(starts)


def _brute_force_partition(sim, keep, eps):
    """Enumerate every consecutive partition (2^(S-1) of them) and return those in
    which (a) every pair inside a set has similarity > eps and touches no
    conserved token, and (b) every cut between two sets is forced: the pair
    across it is not mergeable.  Algorithm 1's result must be the only one."""
    S = len(sim)
    ok = []
    for cuts in itertools.product([0, 1], repeat=S - 1):
        b = (1,) + cuts
        good = True
        for j in range(1, S):
            mergeable = (sim[j] > eps) and not keep[j] and not keep[j - 1]
            if b[j] == 0 and not mergeable:
                good = False
            if b[j] == 1 and mergeable:
                good = False
        if good:
            ok.append(_partition_from_flags(b))
    return ok


def test_sets_equal_unique_brute_force_partition():
    rng = np.random.default_rng(3)
    for trial in range(30):
        S = int(rng.integers(2, 11))
        sim = rng.uniform(-1, 1, S)
        sim[0] = 0
        keep = (rng.random(S) < 0.25).astype(np.uint8)
        eps = float(rng.uniform(-0.5, 0.8))
        b, fired = kvmo.boundaries(sim[None], keep[None], C=S, eps=eps)
        assert fired[0] == 0
        ok = _brute_force_partition(sim, keep, eps)
        assert len(ok) == 1
        assert _partition_from_flags(b[0]) == ok[0]


def test_partition_invariants_and_set_arrays():
    rng = np.random.default_rng(4)
    S, U = 200, 3
    sim = rng.uniform(0.3, 1, (U, S))
    keep = (rng.random((U, S)) < 0.1).astype(np.uint8)
    b, _ = kvmo.boundaries(sim, keep, C=S, eps=0.75)
    set_id, set_start, out_len = kvmo.sets(b, cap=S)
    for u in range(U):
        n = out_len[u]
        assert n == b[u].sum() and b[u, 0] == 1
        st = set_start[u, : n + 1]
        assert st[0] == 0 and st[n] == S and (np.diff(st) > 0).all()       # consecutive, disjoint, cover
        for s in range(n):
            assert (set_id[u, st[s]:st[s + 1]] == s).all()
            if keep[u, st[s]:st[s + 1]].any():                               # conserved tokens are singletons
                assert st[s + 1] - st[s] == 1
            assert (sim[u, st[s] + 1:st[s + 1]] > 0.75).all()                # interior pairs exceed eps


def test_threshold_limits_and_monotonicity():
    K = _rand((1, 64, 8), 5)
    sim = kvmo.similarity(K)
    none = np.zeros((1, 64), np.uint8)
    b, _ = kvmo.boundaries(sim, none, C=64, eps=1.0)
    assert b.sum() == 64                      # eps >= 1: nothing merges (strict '>')
    b, _ = kvmo.boundaries(np.ones((1, 64)), none, C=64, eps=1.0)
    assert b.sum() == 64                      # even identical keys: 1 > 1 is false
    b, _ = kvmo.boundaries(sim, none, C=64, eps=-1.5)
    assert b.sum() == 1                       # eps < -1, nothing conserved: one set
    counts = [kvmo.boundaries(sim, none, C=64, eps=e)[0].sum() for e in np.linspace(-1, 1, 41)]
    assert all(x <= y for x, y in zip(counts, counts[1:]))   # #sets non-decreasing in eps
    ident = np.repeat(_rand((1, 1, 8), 6), 10, axis=1)
    assert kvmo.boundaries(kvmo.similarity(ident), np.zeros((1, 10), np.uint8), 10, 0.75)[0].sum() == 1
    orth = np.eye(8, dtype=np.float32)[None]
    assert kvmo.boundaries(kvmo.similarity(orth), np.zeros((1, 8), np.uint8), 8, 0.75)[0].sum() == 8


def test_single_similar_pair_removes_the_right_boundary():
    sim = np.array([[0.0, 0.1, 0.1, 0.9, 0.1, 0.1]])
    b, _ = kvmo.boundaries(sim, np.zeros((1, 6), np.uint8), 6, 0.75)
    np.testing.assert_array_equal(b[0], [1, 1, 1, 0, 1, 1])       # tokens 2 and 3 group
    keep = np.array([[0, 0, 1, 0, 0, 0]], np.uint8)               # token 2 conserved: no grouping
    b, _ = kvmo.boundaries(sim, keep, 6, 0.75)
    np.testing.assert_array_equal(b[0], [1, 1, 1, 1, 1, 1])
    sim = np.array([[0.0, 0.9, 0.9, 0.9, 0.9, 0.9]])
    b, _ = kvmo.boundaries(sim, keep, 6, 0.75)                    # conserved token splits the run
    np.testing.assert_array_equal(b[0], [1, 0, 1, 1, 0, 0])


def test_budget_rule_brute_force_and_threshold_equivalence():
    rng = np.random.default_rng(7)
    fired_any = 0
    for trial in range(40):
        S = int(rng.integers(4, 11))
        sim = rng.uniform(-1, 1, S)
        sim[0] = 0
        keep = (rng.random(S) < 0.15).astype(np.uint8)
        eps = 0.6
        b0, _ = kvmo.boundaries(sim[None], keep[None], C=S, eps=eps)
        hard = np.array([bool((j == 0) or keep[j] or keep[j - 1]) for j in range(S)])
        n_hard, n0 = int(hard.sum()), int(b0.sum())
        if n0 <= n_hard:
            continue
        C = int(rng.integers(n_hard, n0))          # strictly below the unconstrained count
        b, fired = kvmo.boundaries(sim[None], keep[None], C=C, eps=eps)
        assert fired[0] == 1 and b.sum() == C      # exactly the capacity when the rule fires
        fired_any += 1
        assert (b[0][hard] == 1).all()             # hard boundaries survive
        assert ((b[0] == 1) <= (b0[0] == 1)).all() # nothing new is cut
        # brute force: among all ways to keep C - n_hard of the soft cuts, the rule
        # keeps the ones with the smallest similarities
        soft = [j for j in range(S) if b0[0, j] and not hard[j]]
        m = C - n_hard
        best = min(itertools.combinations(soft, m), key=lambda c: sum(sim[list(c)]))
        assert sorted(j for j in soft if b[0, j]) == sorted(best)
        # same as lowering the threshold for this unit to the m-th smallest soft similarity
        if m > 0:
            eps_low = sorted(sim[soft])[m - 1]
            b_low, _ = kvmo.boundaries(sim[None], keep[None], C=S, eps=eps_low)
            np.testing.assert_array_equal(b_low, b)
    assert fired_any >= 10


def test_budget_rule_off_or_not_needed():
    sim = np.array([[0.0, 0.1, 0.2, 0.3, 0.4, 0.5]])
    none = np.zeros((1, 6), np.uint8)
    b, fired = kvmo.boundaries(sim, none, C=3, eps=0.75, enforce_budget=False)
    assert b.sum() == 6 and fired[0] == 0
    b, fired = kvmo.boundaries(sim, none, C=6, eps=0.75)
    assert b.sum() == 6 and fired[0] == 0
    b, fired = kvmo.boundaries(sim, none, C=3, eps=0.75)
    np.testing.assert_array_equal(b[0], [1, 1, 1, 0, 0, 0])
    assert fired[0] == 1
    b, _ = kvmo.boundaries(np.array([[0.0, 0.2, 0.2, 0.2, 0.2, 0.2]]), none, C=3, eps=0.75)
    np.testing.assert_array_equal(b[0], [1, 1, 1, 0, 0, 0])     # ties -> lower index kept


# ---------------------------------------------------------------- pivots
def test_pivot_is_exhaustive_argmax_lowest_index_on_ties():
    rng = np.random.default_rng(8)
    S = 60
    a = rng.random((2, S))
    a[0, 10] = a[0, 12] = 2.0
    b = (rng.random((2, S)) < 0.3).astype(np.uint8)
    b[:, 0] = 1
    b[0, 9:14] = [1, 0, 0, 0, 0]
    set_id, set_start, out_len = kvmo.sets(b, cap=S)
    pv = kvmo.pivots(a, set_start, out_len)
    for u in range(2):
        for s in range(out_len[u]):
            lo, hi = set_start[u, s], set_start[u, s + 1]
            assert lo <= pv[u, s] < hi
            assert pv[u, s] == lo + int(np.argmax(a[u, lo:hi]))   # numpy argmax: first maximum
        assert (np.diff(pv[u, :out_len[u]]) > 0).all()
    assert pv[0, set_id[0, 10]] == 10
    pv2 = kvmo.pivots(np.exp(3 * a) + 1, set_start, out_len)       # strictly increasing transform
    np.testing.assert_array_equal(pv2, pv)
