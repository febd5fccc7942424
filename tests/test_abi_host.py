"""Host-side checks of the C ABI: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching a GPU."""
import ctypes
import os
import re

import pytest

import paper_2407_08454_b200 as kvm
from paper_2407_08454_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib(kvm_lib):
    return kvm_lib


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "kvm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kvm_[a-z_0-9]+)\s*\(", header))
    assert {"kvm_score", "kvm_segment", "kvm_merge_compact", "kvm_compress"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS) | (declared - set(binding.EXPORTS))
    assert set(binding.EXPORTS) <= declared
    assert kvm.kvm_version() == 101
    assert ctypes.sizeof(kvm.KvmParams) == 80 and kvm.KvmParams.pivot_key.offset == 72


def test_sizes_and_presets(lib):
    p = kvm.make_params(1, 32, 32, 4096, 128, kvm.KVM_BF16, budget=0.5)
    assert kvm.kvm_sizes(p) == (2048, 696, 491)
    p = kvm.make_params(4, 32, 32, 4096, 128, kvm.KVM_BF16, budget=0.35)
    assert kvm.kvm_sizes(p) == (1433, 327, 81)
    p = kvm.make_params(1, 32, 8, 32768, 128, kvm.KVM_BF16, budget=0.5)
    assert kvm.kvm_sizes(p) == (16384, 5570, 3932)
    p = kvm.make_params(1, 4, 4, 512, 64, kvm.KVM_F32, budget=0.5, enforce_budget=0)
    assert kvm.kvm_sizes(p) == (512, 87, 61)
    assert kvm.kvm_workspace_bytes(p) > 0
    assert kvm.kvm_host_staging_bytes(p) > kvm.kvm_workspace_bytes(p)


@pytest.mark.parametrize("kw,status", [
    (dict(dtype=7), -3),
    (dict(head_dim=96), -2),
    (dict(n_q_heads=6, n_kv_heads=4), -2),
    (dict(seq=0), -2),
    (dict(seq=70000), -2),
    (dict(budget=0.0), -4),
    (dict(budget=1.5), -4),
    (dict(sigma=0.0), -4),
    (dict(budget=0.2, recent_ratio=0.17, heavy_ratio=0.12), -4),   # conserved tokens alone exceed the capacity
    (dict(causal=0), -7),
])
def test_bad_parameters_are_rejected_on_the_host(lib, kw, status):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=4, seq=512, head_dim=64, dtype=kvm.KVM_F32)
    base.update(kw)
    p = kvm.make_params(**base)
    n = ctypes.c_size_t()
    assert lib.kvm_workspace_bytes(ctypes.byref(p), ctypes.byref(n)) == status
    assert kvm.status_string(status) != "unknown status"


def test_variant_parameter_checks(lib):
    p = kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_F32, pivot_rule=kvm.KVM_PIVOT_KEY)     # key missing
    with pytest.raises(kvm.KvmError) as e:
        kvm.kvm_sizes(p)
    assert e.value.status == -1
    for bad in (dict(pivot_rule=3), dict(weight_rule=4), dict(set_rule=3)):
        with pytest.raises(kvm.KvmError) as e:
            kvm.kvm_sizes(kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_F32, **bad))
        assert e.value.status == -4
    # eviction: the kept tokens must fit the capacity
    with pytest.raises(kvm.KvmError) as e:
        kvm.kvm_sizes(kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_F32, budget=0.5, recent_ratio=0.3, heavy_ratio=0.3,
                                      set_rule=kvm.KVM_SETS_CONSERVED_ONLY))
    assert e.value.status == -4
    # ... while the same shares are fine when they fill it exactly, which Algorithm 1's forced cuts would not allow
    assert kvm.kvm_sizes(kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_F32, budget=0.5, recent_ratio=0.25,
                                         heavy_ratio=0.25, set_rule=kvm.KVM_SETS_CONSERVED_ONLY))[0] == 128
    # average weights ignore sigma
    assert kvm.kvm_sizes(kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_F32, sigma=0.0,
                                         weight_rule=kvm.KVM_WEIGHT_AVERAGE))[0] == 128


def test_null_alignment_and_workspace_errors(lib):
    p = kvm.make_params(1, 4, 4, 512, 64, kvm.KVM_F32)
    vp = ctypes.c_void_p
    ok = vp(4096)          # never dereferenced: the checks below fail first
    assert lib.kvm_compress(ctypes.byref(p), vp(0), ok, ok, ok, ok, ok, ok, vp(0), vp(0), ok, ctypes.c_size_t(1 << 30), vp(0)) == -1
    assert lib.kvm_compress(ctypes.byref(p), vp(4100), ok, ok, ok, ok, ok, ok, vp(0), vp(0), ok, ctypes.c_size_t(1 << 30), vp(0)) == -5
    assert lib.kvm_compress(ctypes.byref(p), ok, ok, ok, ok, ok, ok, ok, vp(0), vp(0), vp(0), ctypes.c_size_t(0), vp(0)) == -6
    assert lib.kvm_compress(ctypes.byref(p), ok, ok, ok, ok, ok, ok, ok, vp(0), vp(0), ok, ctypes.c_size_t(16), vp(0)) == -6
    assert lib.kvm_score(None, ok, ok, vp(0), ok, ok, ctypes.c_size_t(1 << 30), vp(0)) == -1


def test_layer_stack_entry_point_checks_every_layer_before_it_enqueues(lib):
    p = kvm.make_params(1, 2, 2, 256, 64, kvm.KVM_BF16)
    vp = ctypes.c_void_p
    ok2 = (vp * 2)(4096, 4096)
    bad2 = (vp * 2)(4096, 0)                       # the second layer's pointer is missing
    off2 = (vp * 2)(4096, 4100)                    # ... or not 16-byte aligned
    ws, n = vp(4096), ctypes.c_size_t(1 << 30)
    call = lambda nl, eps, Q: lib.kvm_compress_layers(ctypes.byref(p), ctypes.c_int32(nl), eps, Q, ok2, ok2, ok2, ok2,
                                                      ok2, ok2, vp(0), ws, n, vp(0))
    assert call(0, None, ok2) == -2                # KVM_E_SHAPE
    assert call(2, None, bad2) == -1               # KVM_E_NULL
    assert call(2, None, off2) == -5               # KVM_E_ALIGN
    assert call(2, (ctypes.c_float * 2)(0.75, float("nan")), ok2) == -4      # KVM_E_PARAM
    assert lib.kvm_compress_layers(ctypes.byref(p), ctypes.c_int32(2), None, ok2, ok2, ok2, ok2, ok2, ok2, ok2, vp(0),
                                   ws, ctypes.c_size_t(16), vp(0)) == -6     # KVM_E_WORKSPACE


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libkvm.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()


def test_header_is_plain_c_and_links_from_c(lib, tmp_path):
    """include/kvm.h must be usable from C: compile a small C99 program against it, link it with the
    library, and run the host-only entry points (no device is touched)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "abi.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "kvm.h"
int main(void) {
    kvm_params p;
    memset(&p, 0, sizeof p);
    p.batch = 1; p.n_q_heads = 32; p.n_kv_heads = 8; p.seq = 32768; p.head_dim = 128; p.dtype = KVM_BF16;
    p.budget = 0.5f; p.recent_ratio = -1.f; p.heavy_ratio = -1.f; p.sim_threshold = 0.75f; p.sigma = 5.f;
    p.causal = 1; p.scale_v_by_set_size = 1; p.enforce_budget = 1;
    int32_t cap, nr, nh; size_t ws, host;
    if (kvm_sizes(&p, &cap, &nr, &nh) != KVM_OK) return 1;
    if (kvm_workspace_bytes(&p, &ws) != KVM_OK || kvm_host_staging_bytes(&p, &host) != KVM_OK) return 2;
    p.head_dim = 96;
    if (kvm_sizes(&p, &cap, &nr, &nh) != KVM_E_SHAPE) return 3;
    printf("%d %d %d %zu %zu %d %s\n", (int)cap, (int)nr, (int)nh, ws, host, kvm_version(), kvm_status_string(KVM_E_SHAPE));
    return 0;
}
''')
    exe = tmp_path / "abi"
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-l:libkvm.so", "-Wl,-rpath," + libdir])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    cap, nr, nh, ws, host, ver = out.stdout.split()[:6]
    assert (int(cap), int(nr), int(nh)) == (16384, 5570, 3932)
    assert int(ws) == kvm.kvm_workspace_bytes(kvm.make_params(1, 32, 8, 32768, 128, kvm.KVM_BF16))
    assert int(host) > int(ws) and int(ver) == kvm.kvm_version()
    assert "shape" in out.stdout
