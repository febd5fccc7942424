"""The give-up path of the bounded device waits (failure detection without a fault).

Every wait on an mbarrier in the tensor-core score kernel has a limit; when one runs out the kernel stops
touching tensor memory, writes NaN for the work items it could not finish, reports KVM_E_DEVICE_TIMEOUT through
kvm_stats, frees its tensor memory and returns.  Nothing in the shipped library can make a wait run out, so
this test uses a second build of the same sources (never loaded by the package) in which the limit is two
milliseconds of SM clocks and the TMA producer leaves out its fourth stage: the barrier of that stage is never
armed, the MMA warp's wait for it gives up, and the kernel must come back by itself.  No trap, no unbounded
loop, no bad address is involved.  The eviction rule is used so that what runs after the score step (the
conserved tokens are gathered by index) does not depend on the values of the scores.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import build
from paper_2407_08454_b200 import synth_inputs as si

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct():
    from oracle import kvmo
    from parity import SCORE_ATOL, SCORE_RTOL, f32
    lib = ctypes.CDLL(build.build_waittest())
    cfg = si.CONFIGS["C1"].scaled(seq=1024, n_q_heads=4, n_kv_heads=4, seed=77)     # 8 tiles: the longest items have 4 stages
    d = si.make_layer(cfg)
    Q, K, V = d["Q"].cuda(), d["K"].cuda(), d["V"].cuda()
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype,
                        budget=0.5, set_rule=kvm.KVM_SETS_CONSERVED_ONLY)
    cap, _, _ = kvm.kvm_sizes(p)
    ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    Ko = torch.zeros(cfg.batch, cfg.n_kv_heads, cap, cfg.head_dim, dtype=Q.dtype, device="cuda")
    Vo = torch.zeros_like(Ko)
    out_len = torch.zeros(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    out_pos = torch.zeros(cfg.batch, cfg.n_kv_heads, cap, dtype=torch.int32, device="cuda")
    scores = torch.zeros(cfg.batch, cfg.n_kv_heads, cfg.seq, device="cuda")
    stats = kvm.new_stats("cuda")
    vp = ctypes.c_void_p
    rc = lib.kvm_compress(ctypes.byref(p), vp(Q.data_ptr()), vp(K.data_ptr()), vp(V.data_ptr()), vp(Ko.data_ptr()),
                          vp(Vo.data_ptr()), vp(out_len.data_ptr()), vp(out_pos.data_ptr()), vp(scores.data_ptr()),
                          vp(stats.data_ptr()), vp(ws.data_ptr()), ctypes.c_size_t(ws.numel()),
                          vp(torch.cuda.current_stream().cuda_stream))
    assert rc == 0                                  # nothing is known on the host when the call returns
    torch.cuda.synchronize()                        # the kernels came back by themselves
    assert kvm.read_stats(stats).status == -9       # KVM_E_DEVICE_TIMEOUT
    assert torch.isnan(scores).any()                # what could not be finished is marked, not made up
    # the context is intact: the shipped library computes the same layer correctly right afterwards
    good = torch.empty_like(scores)
    kvm.kvm_score(p, Q, K, None, good, ws)
    torch.cuda.synchronize()
    ref = kvmo.scores(d["Q"].double().numpy(), d["K"].double().numpy(), f32(1.0 / np.sqrt(np.float32(cfg.head_dim))))
    g = good.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(g - ref) <= SCORE_RTOL * np.abs(ref) + SCORE_ATOL)


def test_the_prefill_attention_kernel_also_comes_back_and_reports():
    """Same build, the attention kernel: its producer leaves out the fourth V tile of every work item that has one,
    the MMA thread's wait for it runs out, the kernel returns, the status is set, the rows that were in hand are NaN
    and the work items that never needed that tile are complete."""
    from oracle import kvmo
    lib = ctypes.CDLL(build.build_waittest())
    cfg = si.CONFIGS["C1"].scaled(seq=1024, n_q_heads=4, n_kv_heads=4, seed=78)     # 8 query tiles per head, one per CTA
    d = si.make_layer(cfg)
    Q, K, V = d["Q"].cuda(), d["K"].cuda(), d["V"].cuda()
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype)
    O = torch.zeros_like(Q)
    lse = torch.zeros(1, 4, 1024, device="cuda")
    stats = kvm.new_stats("cuda")
    vp = ctypes.c_void_p
    rc = lib.kvm_prefill_attend(ctypes.byref(p), vp(Q.data_ptr()), vp(K.data_ptr()), vp(V.data_ptr()), vp(O.data_ptr()),
                                vp(lse.data_ptr()), vp(stats.data_ptr()), vp(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    torch.cuda.synchronize()                        # the kernel came back by itself
    assert kvm.read_stats(stats).status == -9       # KVM_E_DEVICE_TIMEOUT
    bad = torch.isnan(lse)
    assert bad[:, :, 3 * 128:].all()                # query tiles 3..7 need a fourth V tile: marked, not made up
    assert not bad[:, :, :3 * 128].any()            # tiles 0..2 never needed it
    refO, ref_lse = kvmo.prefill_attend(d["Q"][:, :, :384], d["K"][:, :, :384], d["V"][:, :, :384])
    assert np.abs(lse[:, :, :384].cpu().numpy() - ref_lse).max() <= 2e-4
    # the context is intact: the shipped library computes the same layer correctly right afterwards
    kvm.kvm_prefill_attend(p, Q, K, V, O, lse)
    torch.cuda.synchronize()
    refO, ref_lse = kvmo.prefill_attend(d["Q"], d["K"], d["V"])
    assert torch.isfinite(lse).all() and np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-4
