"""Host-side checks that need no GPU: the C-ABI library loads and exports every symbol that
include/buzz.h declares, and the workload generators are seeded and shaped as documented."""
import ctypes
import os
import re

import torch

import workloads
from paper_2410_23079_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    with open(os.path.join(ROOT, "include", "buzz.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(buzz_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2410_23079_b200 import build
    lib = ctypes.CDLL(build.build())
    declared = _declared_symbols()
    assert len(declared) >= 14
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in buzz.h but not exported"
    assert sorted(binding.exported_symbols()) == declared


def test_error_strings_without_a_gpu():
    lib = binding.load_library()
    assert lib.buzz_error_string(0) == b"ok"
    for code in range(-6, 0):
        assert lib.buzz_error_string(code) not in (b"ok", b"unknown error")


def test_workspace_sizes_and_validation_without_a_gpu():
    lib = binding.load_library()
    sh = binding._Shape(32, 8, 32, 32, 128, binding.BUZZ_BF16, 32768, 0)
    sb, cb = ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.buzz_workspace_bytes(ctypes.byref(sh), 1843, ctypes.byref(sb), ctypes.byref(cb)) == 0
    inst = 32 * 8 * 32
    assert sb.value >= inst * 1843 * (2 * 128 * 2 + 8) + 3 * 4 * inst
    assert cb.value >= (32 + 32) * 32768 * 4
    bad = binding._Shape(32, 8, 32, 5, 128, binding.BUZZ_BF16, 32768, 0)
    assert lib.buzz_workspace_bytes(ctypes.byref(bad), 1843, ctypes.byref(sb), ctypes.byref(cb)) == -1
    h = ctypes.c_void_p()
    assert lib.buzz_create(ctypes.byref(h), 4, 512, 8, 1, 1843, ctypes.byref(sh), None, 0, None, 0) == -1


def test_generators_are_seeded_and_shaped():
    w = workloads.scaled(workloads.get("C5"), layers=1, batch=3, q_heads=4, kv_heads=2,
                         prompt_min=50, prompt_max=90, decode_steps=4)
    lens = workloads.prompt_lengths(w)
    assert lens == workloads.prompt_lengths(w) and all(50 <= n <= 90 for n in lens)
    a = workloads.prefill_inputs(w, 0)
    b = workloads.prefill_inputs(w, 0)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    q, k, v, cu = a
    assert q.shape == (sum(lens), 4, 128) and k.shape == (sum(lens), 2, 128) and q.dtype == torch.bfloat16
    assert cu.tolist() == [0] + list(torch.tensor(lens).cumsum(0).tolist())
    assert not torch.equal(workloads.prefill_inputs(w, 1)[1], k)
    qd, kd, vd = workloads.decode_inputs(w, 0)
    assert qd.shape == (4, 3, 4, 128) and kd.shape == (4, 3, 2, 128)


def test_outlier_rows_are_present():
    w = workloads.scaled(workloads.get("C1"), prompt_min=4000, prompt_max=4000)
    _, k, _, _ = workloads.prefill_inputs(w, 0)
    norms = k.float().norm(dim=-1).flatten()
    frac = (norms > 2.0 * norms.median()).float().mean().item()
    assert 0.03 < frac < 0.07
