"""GPU parity of the decode-step attention (Eq. 1) and of the output perturbation
of Definition 2.1, through the C ABI against the fp64 CPU checker.

Bars: attention output  |gpu - ref| <= 1e-4 * max_d |ref| + 1e-6  per head (fp32 accumulation over at most
a few thousand bf16/fp32 rows); norms  |gpu - ref| <= 1e-4 * |O_t| + 1e-6."""
import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from oracle import kvmo
from paper_2407_08454_b200 import synth_inputs as si

pytestmark = pytest.mark.gpu

O_RTOL, O_ATOL = 1e-4, 1e-6


def _close(gpu, ref):
    bound = O_RTOL * np.abs(ref).max(axis=-1, keepdims=True) + O_ATOL
    assert (np.abs(gpu.astype(np.float64) - ref) <= bound).all(), float(np.max(np.abs(gpu - ref) / bound))


@pytest.mark.parametrize("B,Hq,Hkv,rows,D,dtype", [
    (2, 4, 4, 300, 64, torch.float32),
    (1, 8, 2, 1000, 128, torch.bfloat16),      # group of 4, several chunks, ragged tail
    (2, 6, 3, 129, 128, torch.bfloat16),
    (1, 2, 1, 4096, 64, torch.bfloat16),
])
def test_attend_matches_the_checker_on_ragged_caches(B, Hq, Hkv, rows, D, dtype):
    g = torch.Generator().manual_seed(rows + D)
    q = (torch.randn(B, Hq, D, generator=g) * 2).to(dtype)
    K = torch.randn(B, Hkv, rows, D, generator=g).to(dtype)
    V = torch.randn(B, Hkv, rows, D, generator=g).to(dtype)
    length = torch.randint(1, rows + 1, (B, Hkv), generator=g, dtype=torch.int32)
    length.view(-1)[0] = rows
    if length.numel() > 1:
        length.view(-1)[1] = 1
    if length.numel() > 2:
        length.view(-1)[2] = 0                  # an empty unit gives zeros
    p = kvm.make_params(B, Hq, Hkv, rows, D, dtype)
    ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    qd, Kd, Vd = q.cuda(), K.cuda(), V.cuda()
    for ln in (length, None):
        out = torch.full((B, Hq, D), float("nan"), device="cuda")
        kvm.kvm_attend(p, qd, Kd, Vd, rows, None if ln is None else ln.cuda(), out, ws)
        ref = kvmo.attend(q, K, V, None if ln is None else ln.numpy())
        _close(out.cpu().numpy(), ref)
    # a shorter row count than the parameter's seq is accepted; a longer one is not
    half = rows // 2
    out = torch.empty((B, Hq, D), device="cuda")
    kvm.kvm_attend(p, qd, Kd[:, :, :half].contiguous(), Vd[:, :, :half].contiguous(), half, None, out, ws)
    _close(out.cpu().numpy(), kvmo.attend(q, K[:, :, :half], V[:, :, :half]))
    with pytest.raises(kvm.KvmError):
        kvm.kvm_attend(p, qd, Kd, Vd, rows + 1, None, out, ws)


def _perturb(cfg, **rules):
    d = si.make_layer(cfg)
    Q, K, V = d["Q"].cuda(), d["K"].cuda(), d["V"].cuda()
    B, Hq, S, D = Q.shape
    p = kvm.make_params(B, Hq, K.shape[1], S, D, Q.dtype, budget=cfg.budget, **rules)
    c = kvm.Compressor(p)
    r = c(Q, K, V)
    qt = Q[:, :, -1].contiguous()                # the most recent query stands in for the decode-step query
    of = torch.empty(B, Hq, D, device="cuda")
    oc = torch.empty_like(of)
    err = torch.empty(B, Hq, device="cuda")
    ref = torch.empty_like(err)
    kvm.kvm_output_perturbation(p, qt, K, V, r.K_out, r.V_out, r.out_len, of, oc, err, ref, c.ws)
    torch.cuda.synchronize()
    # checker on the same caches (the compressed one as the library stored it)
    rf = kvmo.attend(qt.cpu(), d["K"], d["V"])
    rc = kvmo.attend(qt.cpu(), r.K_out.cpu(), r.V_out.cpu(), r.out_len.cpu().numpy())
    _close(of.cpu().numpy(), rf)
    _close(oc.cpu().numpy(), rc)
    e_ref, n_ref = kvmo.perturbation(rf, rc)
    assert (np.abs(err.cpu().numpy() - e_ref) <= O_RTOL * n_ref + O_ATOL).all()
    assert (np.abs(ref.cpu().numpy() - n_ref) <= O_RTOL * n_ref + O_ATOL).all()
    return float((err / ref).mean()), float((err / ref).max())


def test_output_perturbation_of_the_method_and_its_variants():
    cfgs = [si.CONFIGS["C0"], si.CONFIGS["C1"].scaled(seq=2048, n_q_heads=8, n_kv_heads=4, seed=31)]
    for cfg in cfgs:
        rows = {
            "gaussian merge, |S| scaling": dict(),
            "gaussian merge, plain mean": dict(scale_v_by_set_size=0),
            "average weights, last pivot": dict(pivot_rule=kvm.KVM_PIVOT_LAST, weight_rule=kvm.KVM_WEIGHT_AVERAGE,
                                                scale_v_by_set_size=0),
            "pivot only": dict(weight_rule=kvm.KVM_WEIGHT_PIVOT_ONLY, scale_v_by_set_size=0),
            "eviction": dict(set_rule=kvm.KVM_SETS_CONSERVED_ONLY, recent_ratio=0.17,
                             heavy_ratio=cfg.budget - 0.17),
        }
        for name, rules in rows.items():
            mean, worst = _perturb(cfg, **rules)
            print(f"{cfg.name} S={cfg.seq} {name}: mean |dO|/|O| = {mean:.4f}, max = {worst:.4f}")


def test_no_merging_gives_zero_perturbation():
    cfg = si.CONFIGS["C1"].scaled(seq=640, n_q_heads=4, n_kv_heads=2, seed=32)
    mean, worst = _perturb(cfg, sim_threshold=1.5, enforce_budget=0, recent_ratio=0.0, heavy_ratio=0.0)
    assert mean == 0.0 and worst == 0.0
