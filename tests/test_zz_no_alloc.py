"""kvm_score_static: the score step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: the process
gave all of its device memory to another allocator at start-up, or an allocation
(which can stall the device) is not allowed on the calling path, and no spare
buffer is at hand to lend as the workspace kvm_score asks for.  For them the
library carries a fixed scratch array inside its own image.  This file checks,
through the C ABI, that the variant gives exactly the scores of kvm_score (the
two run the same kernels), several times in a row (later calls find the earlier
calls' leftovers in the shared array), that those scores also meet the bar
against the CPU checker, that the call leaves the amount of free device memory
as it found it, that the largest bf16 problem the array can hold is accepted,
and that problems too large for it are refused with their own status.

It is collected last on purpose, so a failure here cannot hide another test's result.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import binding
from paper_2407_08454_b200 import synth_inputs as si


@pytest.fixture(scope="module")
def lib(kvm_lib):
    return kvm_lib


def test_problems_beyond_the_built_in_scratch_are_refused(lib):
    ok = ctypes.c_void_p(4096)
    # 2 * 32 * 32768 rows = 2 Mi > KVM_STATIC_SCORE_ROWS; refused on the host, before any GPU work
    p = kvm.make_params(2, 32, 8, 32768, 128, kvm.KVM_BF16)
    rc = lib.kvm_score_static(ctypes.byref(p), ok, ok, ok, ctypes.c_void_p(0))
    assert rc == -10
    assert "kvm_score_static" in kvm.status_string(rc)
    assert binding.KVM_STATIC_SCORE_ROWS == 1 << 20
    # bf16 leaves 32 bytes per row: one row past 2^17 is refused, fp32 with the same row count is not a size error
    p = kvm.make_params(1, 4, 4, (1 << 15) + 1, 128, kvm.KVM_BF16)
    assert lib.kvm_score_static(ctypes.byref(p), ok, ok, ok, ctypes.c_void_p(0)) == -10


@pytest.mark.gpu
def test_static_scratch_variant_matches_kvm_score_on_two_calls_in_a_row():
    from oracle import kvmo
    from parity import SCORE_ATOL, SCORE_RTOL, f32
    shapes = [si.CONFIGS["C1"].scaled(seq=1000, n_q_heads=8, n_kv_heads=2, seed=21),     # first call: larger
              si.CONFIGS["C0"].scaled(seq=300, seed=22)]                                  # second: smaller, fp32
    for cfg in shapes:
        d = si.make_layer(cfg)
        Q, K = d["Q"].cuda(), d["K"].cuda()
        p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype)
        ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        want = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seq, device="cuda")
        kvm.kvm_score(p, Q, K, None, want, ws)
        ref = kvmo.scores(d["Q"].double().numpy(), d["K"].double().numpy(),
                          f32(1.0 / np.sqrt(np.float32(cfg.head_dim))))
        for call in range(3):
            got = torch.full_like(want, float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            kvm.kvm_score_static(p, Q, K, got)
            torch.cuda.synchronize()
            # The first call on a device is the documented one-time set-up (the CUDA runtime may only then place
            # the library's built-in array in device memory); after it a call must leave free memory untouched.
            if call > 0:
                assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
            assert torch.equal(got, want), (cfg.name, call)          # same kernels, same inputs: same bits
            g = got.cpu().numpy().astype(np.float64)
            assert np.all(np.abs(g - ref) <= SCORE_RTOL * np.abs(ref) + SCORE_ATOL), (cfg.name, call)


@pytest.mark.gpu
def test_the_largest_bf16_problem_the_array_holds_is_accepted():
    # 1 x 32 heads x 4096 tokens = 2^17 rows of 32 bytes: exactly the array
    cfg = si.CONFIGS["C1"]
    assert cfg.batch * cfg.n_q_heads * cfg.seq == binding.KVM_STATIC_SCORE_ROWS // 8
    d = si.make_layer(cfg)
    Q, K = d["Q"].cuda(), d["K"].cuda()
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype)
    ws = torch.empty(kvm.kvm_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    want = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seq, device="cuda")
    kvm.kvm_score(p, Q, K, None, want, ws)
    got = torch.full_like(want, float("nan"))
    kvm.kvm_score_static(p, Q, K, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
