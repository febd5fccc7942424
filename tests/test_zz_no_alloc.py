"""kvm_score_static: the score step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: the process
gave all of its device memory to another allocator at start-up, or an allocation
(which can stall the device) is not allowed on the calling path, and no spare
buffer is at hand to lend as the workspace kvm_score asks for.  For them the
library carries a fixed scratch array inside its own image.  This file checks,
through the C ABI, that the variant gives the same scores as kvm_score, twice in
a row (the second call finds the first call's leftovers in the shared array),
and that problems too large for the array are refused with their own status.

It is collected last on purpose, so a failure here cannot hide another test's result.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import binding, build
from paper_2407_08454_b200 import synth_inputs as si


def test_problems_beyond_the_built_in_scratch_are_refused():
    build.build()
    # 2 * 32 * 32768 rows = 2 Mi > KVM_STATIC_SCORE_ROWS; refused on the host, before any GPU work
    p = kvm.make_params(2, 32, 8, 32768, 128, kvm.KVM_BF16)
    ok = ctypes.c_void_p(4096)
    rc = binding.lib().kvm_score_static(ctypes.byref(p), ok, ok, ok, ctypes.c_void_p(0))
    assert rc == -10
    assert "kvm_score_static" in kvm.status_string(rc)
    assert binding.KVM_STATIC_SCORE_ROWS == 1 << 20


@pytest.mark.gpu
def test_static_scratch_variant_matches_kvm_score_on_two_calls_in_a_row():
    from parity import SCORE_ATOL, SCORE_RTOL
    shapes = [si.CONFIGS["C1"].scaled(seq=1000, n_q_heads=8, n_kv_heads=2, seed=21),     # first call: larger
              si.CONFIGS["C0"].scaled(seq=300, seed=22)]                                  # second: smaller, fp32
    for cfg in shapes:
        d = si.make_layer(cfg)
        Q, K = d["Q"].cuda(), d["K"].cuda()
        p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype)
        ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        want = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seq, device="cuda")
        kvm.kvm_score(p, Q, K, None, want, ws)
        for call in range(2):
            got = torch.full_like(want, float("nan"))
            kvm.kvm_score_static(p, Q, K, got)
            torch.cuda.synchronize()
            w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
            assert np.all(np.abs(g - w) <= SCORE_RTOL * np.abs(w) + SCORE_ATOL), (cfg.name, call)
