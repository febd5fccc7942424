"""Causal attention over the whole prompt (Eq. 1 for every position) on the GPU against the CPU checker, and the
compression path fed by the row log-sum-exp that this attention returns.

Bars.  lse: |gpu - ref| <= 2e-4 (fp32 sums of fp32 exponentials; the score bar of 1e-3 relative leaves room for
it).  O: the probabilities enter the second product rounded to bf16 (relative 2^-9 each, as in every tensor-core
attention kernel) and O is rounded to bf16 once at the store (2^-9 of |O|), so element-wise
|gpu - ref| <= 1e-2 |ref| + 2^-8 max|V| of the unit; the measured error is a small fraction of that.
"""
import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import synth_inputs as si

pytestmark = pytest.mark.gpu

LSE_ATOL = 2e-4


def _run(cfg, d):
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype,
                        budget=cfg.budget)
    Q, K, V = d["Q"].cuda(), d["K"].cuda(), d["V"].cuda()
    O = torch.full_like(Q, 7.0)
    lse = torch.full(Q.shape[:3], -3.0, dtype=torch.float32, device="cuda")
    stats = kvm.new_stats("cuda")
    kvm.kvm_prefill_attend(p, Q, K, V, O, lse, stats)
    torch.cuda.synchronize()
    assert kvm.read_stats(stats).status == 0
    return p, Q, K, V, O, lse


def _check(O, lse, refO, ref_lse, V, G):
    g_lse = lse.cpu().numpy().astype(np.float64)
    assert np.abs(g_lse - ref_lse).max() <= LSE_ATOL
    gO = O.float().cpu().numpy().astype(np.float64)
    vmax = np.abs(V.float().numpy()).max(axis=(2, 3))                      # per (batch entry, KV head)
    tol = 1e-2 * np.abs(refO) + 2.0 ** -8 * np.repeat(vmax, G, axis=1)[:, :, None, None]
    excess = np.abs(gO - refO) / tol
    assert excess.max() <= 1.0, excess.max()
    return float(excess.max())


@pytest.mark.parametrize("S,D,Hq,Hkv,B", [(640, 128, 4, 2, 1), (300, 64, 2, 2, 2), (1024, 128, 8, 2, 1), (129, 128, 1, 1, 1),
                                          (77, 64, 4, 1, 1),
                                          (1100, 64, 40, 8, 1)])      # 360 work items: several per CTA, ragged last tile
def test_prefill_attention_matches_the_checker_elementwise(S, D, Hq, Hkv, B):
    from oracle import kvmo
    cfg = si.CONFIGS["C1"].scaled(seq=S, head_dim=D, n_q_heads=Hq, n_kv_heads=Hkv, batch=B, seed=31)
    d = si.make_layer(cfg)
    _, _, _, _, O, lse = _run(cfg, d)
    refO, ref_lse = kvmo.prefill_attend(d["Q"], d["K"], d["V"])
    _check(O, lse, refO, ref_lse, d["V"], Hq // Hkv)


def test_prefill_attention_with_unscaled_logits_and_a_custom_scale():
    """Nearly one-hot rows (logits of standard deviation in the tens) move the reference maximum often."""
    from oracle import kvmo
    cfg = si.CONFIGS["C1"].scaled(seq=512, n_q_heads=2, n_kv_heads=2, seed=32, logit_std=-1.0)
    d = si.make_layer(cfg)
    p = kvm.make_params(1, 2, 2, 512, 128, torch.bfloat16, softmax_scale=0.05)
    Q, K, V = d["Q"].cuda(), d["K"].cuda(), d["V"].cuda()
    O, lse = torch.empty_like(Q), torch.empty(1, 2, 512, device="cuda")
    kvm.kvm_prefill_attend(p, Q, K, V, O, lse)
    torch.cuda.synchronize()
    refO, ref_lse = kvmo.prefill_attend(d["Q"], d["K"], d["V"], 0.05)
    g_lse = lse.cpu().numpy().astype(np.float64)
    assert np.abs(g_lse - ref_lse).max() <= 1e-5 * np.abs(ref_lse).max() + LSE_ATOL    # logits of magnitude 100s
    gO = O.float().cpu().numpy().astype(np.float64)
    assert (np.abs(gO - refO) <= 1e-2 * np.abs(refO) + 2.0 ** -8 * np.abs(d["V"].float().numpy()).max()).all()


def test_compression_fed_by_the_attention_kernels_lse_matches_the_checker():
    """The production order: prefill attention -> its lse -> kvm_compress_with_lse (no row pass)."""
    from oracle import kvmo
    from parity import Case, _chain, f32, kv_error, score_excess, KV_TOL
    S = 1000
    cfg = si.CONFIGS["C1"].scaled(seq=S, n_q_heads=4, n_kv_heads=2, seed=33)
    d = si.make_layer(cfg)
    p, Q, K, V, O, lse = _run(cfg, d)
    case = Case(d["Q"], d["K"], d["V"], budget=0.5)
    comp = kvm.Compressor(p, want_scores=True)
    kvm.kvm_compress_with_lse(p, Q, K, V, lse, comp.K_out, comp.V_out, comp.out_len, comp.out_pos, comp.scores, None,
                              comp.ws)
    torch.cuda.synchronize()
    ref = kvmo.scores(d["Q"], d["K"])
    g_scores = comp.scores.cpu().numpy().reshape(2, S)
    assert score_excess(g_scores, ref.reshape(2, S)) <= 1.0
    sim = torch.empty(1, 2, S, device="cuda")
    ratio = torch.empty(2, device="cuda")
    kvm.kvm_layer_ratio(p, K, ratio, sim, comp.ws)
    cap, n_r, n_h = kvm.kvm_sizes(p)
    ch = _chain(case, g_scores.astype(np.float64), sim.cpu().numpy().reshape(2, S).astype(np.float64), cap, n_r, n_h)
    g_len = comp.out_len.cpu().numpy().reshape(2)
    assert np.array_equal(g_len, ch["out_len"])
    g_pos = comp.out_pos.cpu().numpy().reshape(2, cap)
    rK, rV = kvmo.merge(d["K"][0], d["V"][0], ch["set_start"], ch["pivot"], ch["out_len"], f32(5.0), True)
    for u in range(2):
        n = g_len[u]
        assert np.array_equal(g_pos[u, :n], ch["pivot"][u, :n])
        assert kv_error(comp.K_out[0, u, :n].float().cpu().numpy(), rK[u, :n]) <= KV_TOL
        assert kv_error(comp.V_out[0, u, :n].float().cpu().numpy(), rV[u, :n]) <= KV_TOL
    # the same scores as the library's own two-pass path, to the score bar
    own = torch.empty_like(comp.scores)
    kvm.kvm_score(p, Q, K, None, own, comp.ws)
    torch.cuda.synchronize()
    assert score_excess(g_scores, own.cpu().numpy().reshape(2, S).astype(np.float64)) <= 1.0


def test_prefill_attention_full_c1_layer_sampled_heads_and_twice_identical():
    """The benchmark's shape and launch configuration: every head through the library, two heads against the
    checker in full, two runs bit-identical, untouched memory around the outputs."""
    from oracle import kvmo
    cfg = si.CONFIGS["C1"]
    d = si.make_layer(cfg)
    p, Q, K, V, O, lse = _run(cfg, d)
    O2, lse2 = torch.empty_like(O), torch.empty_like(lse)
    kvm.kvm_prefill_attend(p, Q, K, V, O2, lse2)
    torch.cuda.synchronize()
    assert torch.equal(O, O2) and torch.equal(lse, lse2)
    assert torch.isfinite(O.float()).all() and torch.isfinite(lse).all()
    for h in (0, 31):
        refO, ref_lse = kvmo.prefill_attend(d["Q"][:, h:h + 1], d["K"][:, h:h + 1], d["V"][:, h:h + 1])
        _check(O[:, h:h + 1], lse[:, h:h + 1], refO, ref_lse, d["V"][:, h:h + 1], 1)


def test_prefill_attention_rejects_what_it_does_not_support():
    p = kvm.make_params(1, 2, 2, 256, 64, torch.float32)
    x = torch.zeros(1, 2, 256, 64, device="cuda")
    with pytest.raises(kvm.KvmError) as e:
        kvm.kvm_prefill_attend(p, x, x, x, x, torch.zeros(1, 2, 256, device="cuda"))
    assert e.value.status == -7          # KVM_E_UNSUPPORTED
