"""GPU parity of the method's variants: average-weighted merging with last-index
pivots (Section 4.2), keyed (random) pivots (Section 5.3), pivot-only weights
(the sigma -> 0 limit after Eq. 5) and eviction (Section 2.2), through the C ABI
against the fp64 CPU checker.  Bars are defined in parity.py."""
import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import synth_inputs as si
from parity import Case, check_case, check_evict_case, run_gpu

pytestmark = pytest.mark.gpu

SHAPES = [
    ("C0", dict()),                                                            # fp32, D = 64
    ("C1", dict(seq=777, n_q_heads=4, n_kv_heads=2, batch=2, seed=21)),         # bf16, GQA, ragged
    ("C1", dict(seq=2048, n_q_heads=4, n_kv_heads=4, budget=0.35, seed=22)),    # long sets cross tiles
]


def _case(name, kw, **rules):
    cfg = si.CONFIGS[name].scaled(**kw) if kw else si.CONFIGS[name]
    d = si.make_layer(cfg)
    return Case(d["Q"], d["K"], d["V"], budget=cfg.budget, **rules)


def _key_for(case, seed):
    B, _, S, _ = case.Q.shape
    g = torch.Generator().manual_seed(seed)
    return torch.rand((B, case.K.shape[1], S), generator=g, dtype=torch.float32)


@pytest.mark.parametrize("name,kw", SHAPES)
def test_average_weighted_last_index_baseline(name, kw):
    for scale_v in (False, True):
        rep = check_case(_case(name, kw, pivot_rule=kvm.KVM_PIVOT_LAST, weight_rule=kvm.KVM_WEIGHT_AVERAGE,
                               scale_v=scale_v))
        print(name, kw, scale_v, rep)


@pytest.mark.parametrize("name,kw", SHAPES)
def test_keyed_pivots_random_ablation(name, kw):
    case = _case(name, kw, pivot_rule=kvm.KVM_PIVOT_KEY)
    case.pivot_key = _key_for(case, 5)
    g = run_gpu(case)
    rep = check_case(case, g)
    base = run_gpu(_case(name, kw))
    assert np.array_equal(g.set_start, base.set_start)          # the sets do not depend on the pivot rule
    assert (g.pivot != base.pivot).any()
    print(name, kw, rep)


@pytest.mark.parametrize("name,kw", SHAPES[:2])
def test_pivot_only_weights(name, kw):
    for scale_v in (False, True):
        rep = check_case(_case(name, kw, weight_rule=kvm.KVM_WEIGHT_PIVOT_ONLY, scale_v=scale_v))
        print(name, kw, scale_v, rep)


@pytest.mark.parametrize("name,kw", SHAPES)
def test_eviction_keeps_the_conserved_tokens(name, kw):
    cfg = si.CONFIGS[name].scaled(**kw) if kw else si.CONFIGS[name]
    recent = 0.17 if cfg.budget >= 0.425 else 0.08
    case = _case(name, kw, set_rule=kvm.KVM_SETS_CONSERVED_ONLY, recent=recent, heavy=cfg.budget - recent)
    rep = check_evict_case(case)
    print(name, kw, rep)


def test_layer_ratio_and_per_layer_thresholds():
    # per-layer token correlation differs (as across a model's layers): the ratio statistic follows it, and a
    # threshold per layer steers it (Section 3.2)
    cfg = si.CONFIGS["C2"].scaled(seq=1024, n_q_heads=4, n_kv_heads=4, batch=1, layers=4)
    from oracle import kvmo
    p = kvm.make_params(1, 4, 4, 1024, 128, torch.bfloat16, budget=cfg.budget)
    ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    layers, ratios = [], []
    for layer in range(4):
        d = si.make_layer(cfg, layer)
        K = d["K"].cuda()
        layers.append((d["Q"].cuda(), K, d["V"].cuda()))
        ratio = torch.full((4,), -1.0, device="cuda")
        sim = torch.empty(1, 4, 1024, device="cuda")
        kvm.kvm_layer_ratio(p, K, ratio, sim, ws)
        ref_sim = kvmo.similarity(d["K"][0])
        assert np.abs(sim[0].cpu().numpy() - ref_sim).max() <= 4e-6
        want = kvmo.layer_ratio(sim[0].double().cpu().numpy(), float(np.float32(0.75)))     # same fp32 similarities
        np.testing.assert_allclose(ratio.cpu().numpy(), want, rtol=1e-6)
        ratios.append(float(ratio.mean()))
        assert 1.0 / 1024 <= ratios[-1] <= 1.0
    # per-layer thresholds through the whole path: a lower threshold never gives more rows
    outs_hi, r_hi = kvm.compress_layers(p, layers, [0.9] * 4)
    outs_lo, r_lo = kvm.compress_layers(p, layers, [0.6, 0.65, 0.7, 0.75])
    assert all(lo <= hi for lo, hi in zip(r_lo, r_hi))
    for (Q, K, V), o, eps in zip(layers, outs_lo, [0.6, 0.65, 0.7, 0.75]):
        g = run_gpu(Case(Q.cpu(), K.cpu(), V.cpu(), budget=cfg.budget, eps=eps))
        assert np.array_equal(o.out_len.cpu().numpy(), g.c_out_len)
    print("layer ratios", ratios, "compressed", r_lo, r_hi)


@pytest.mark.parametrize("name,kw", SHAPES + [("C1", dict(seq=4096, n_q_heads=2, n_kv_heads=2, seed=23)),
                                              ("C4", dict(seq=1500, n_q_heads=4, n_kv_heads=4, batch=1, seed=24))])
def test_anchor_reading_of_the_set_identification(name, kw):
    """Section 3.2's wording: similarity to the group's last state.  The run lengths are the only numbers floating
    point decides: they must equal the checker's except where a pair lies within 1e-3 of the threshold, and given
    the library's own run lengths and scores every integer output must equal the checker's integer-only walk."""
    from oracle import kvmo
    from parity import f32, kv_error, KV_TOL
    case = _case(name, kw, set_rule=kvm.KVM_SETS_ANCHOR, enforce=False)
    g = run_gpu(case)
    B, Hq, S, D = case.Q.shape
    U = B * case.K.shape[1]
    cap, n_r, n_h = kvm.kvm_sizes(case.params())
    assert cap == S
    K = case.K.reshape(U, S, D)
    eps = f32(case.eps)
    g_run = g.sim.reshape(U, S)
    assert (g_run == np.round(g_run)).all()
    g_run = g_run.astype(np.int32)
    keep = kvmo.keep(g.scores.reshape(U, S).astype(np.float64), n_r, n_h)
    _, ref_run = kvmo.boundaries_anchor(K, keep, eps, want_run=True)
    K64 = K.double().numpy()
    differ = np.argwhere(g_run != ref_run)
    for u, i in differ:                         # each disagreement needs a pair at the threshold
        lo = max(0, i - max(g_run[u, i], ref_run[u, i]) - 1)
        a = K64[u, i]
        c = (K64[u, lo:i] @ a) / (np.linalg.norm(K64[u, lo:i], axis=1) * np.linalg.norm(a) + 1e-300)
        assert np.abs(c - eps).min() < 1e-3, (u, i, g_run[u, i], ref_run[u, i])
    assert len(differ) <= 0.01 * U * S
    b = kvmo.boundaries_anchor(K, keep, eps, run_in=g_run)
    set_id, st, ol = kvmo.sets(b, cap)
    pv = kvmo.pivots(g.scores.reshape(U, S).astype(np.float64), st, ol)
    assert np.array_equal(g.out_len.reshape(U), ol) and np.array_equal(g.set_id.reshape(U, S), set_id)
    g_st, g_pv = g.set_start.reshape(U, cap + 1), g.pivot.reshape(U, cap)
    rK, rV = kvmo.merge(K, case.V.reshape(U, S, D), st, pv, ol, f32(case.sigma), True)
    for u in range(U):
        n = ol[u]
        assert np.array_equal(g_st[u, :n + 1], st[u, :n + 1]) and np.array_equal(g_pv[u, :n], pv[u, :n])
        assert kv_error(g.K_out.reshape(U, cap, D)[u, :n], rK[u, :n]) <= KV_TOL
        assert kv_error(g.V_out.reshape(U, cap, D)[u, :n], rV[u, :n]) <= KV_TOL
        assert np.array_equal(g.c_out_pos.reshape(U, cap)[u, :n], pv[u, :n])
        assert np.array_equal(g.c_K_out.reshape(U, cap, D)[u, :n], g.K_out.reshape(U, cap, D)[u, :n])
    assert np.array_equal(g.c_out_len.reshape(U), ol)
    print(name, kw, "sets", ol.tolist()[:4], "run disagreements", len(differ))


def test_anchor_reading_limits():
    with pytest.raises(kvm.KvmError) as e:      # needs the full capacity and a sequence that fits shared memory
        kvm.kvm_sizes(kvm.make_params(1, 2, 2, 512, 64, torch.float32, set_rule=kvm.KVM_SETS_ANCHOR))
    assert e.value.status == -7
    with pytest.raises(kvm.KvmError) as e:
        kvm.kvm_sizes(kvm.make_params(1, 2, 2, 40961, 64, torch.float32, set_rule=kvm.KVM_SETS_ANCHOR,
                                      enforce_budget=0))
    assert e.value.status == -7
    # the longest accepted sequence runs (one unit), with the invariants of a partition
    S = 40960
    cfg = si.CONFIGS["C1"].scaled(seq=S, head_dim=64, n_q_heads=1, n_kv_heads=1, seed=25)
    d = si.make_layer(cfg)
    p = kvm.make_params(1, 1, 1, S, 64, torch.bfloat16, set_rule=kvm.KVM_SETS_ANCHOR, enforce_budget=0)
    r = kvm.Compressor(p)(d["Q"].cuda(), d["K"].cuda(), d["V"].cuda())
    n = int(r.out_len[0, 0])
    pos = r.out_pos[0, 0, :n].cpu().numpy()
    assert 1 <= n <= S and (np.diff(pos) > 0).all() and pos[-1] <= S - 1


@pytest.mark.parametrize("name,kw", SHAPES)
def test_bandwidth_per_merging_set(name, kw):
    # one non-circular reading of Eq. 4 (parity unpinned by the paper): 2 sigma^2 = the set's mean squared
    # distance to its pivot; the sets and pivots are those of the method
    for scale_v in (False, True):
        case = _case(name, kw, weight_rule=kvm.KVM_WEIGHT_SET_SIGMA, scale_v=scale_v, sigma=0.0)
        g = run_gpu(case)
        rep = check_case(case, g)
        print(name, kw, scale_v, rep)
    base = run_gpu(_case(name, kw))
    assert np.array_equal(g.set_start, base.set_start) and np.array_equal(g.pivot, base.pivot)
    assert not np.array_equal(g.K_out, base.K_out)
