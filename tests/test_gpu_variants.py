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
