"""Random Q/K/V tensors for the workloads; nothing here knows what attention or eviction is.

Layouts: prompt tensors are packed over the batch, Q ``[sum N, Hq, d]`` and K, V
``[sum N, Hkv, d]`` with ``cu_seqlens`` ``[batch + 1]``; decode tensors are ``[steps, batch, H, d]``.
Values are drawn on the requested device from a generator seeded by (workload, layer, tensor), then
rounded to the workload's dtype; those rounded values *are* the inputs (whoever needs them on the
host copies the same bytes).
"""
from __future__ import annotations

import math

import torch

from .configs import Workload

_DT = {"f32": torch.float32, "bf16": torch.bfloat16}
_TAG = {"q": 1, "k": 2, "v": 3, "mask": 4, "w": 5, "phi": 6, "mu": 7, "dq": 11, "dk": 12, "dv": 13,
        "dmask": 14, "len": 21}


def _gen(w: Workload, layer: int, tag: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((w.seed * 1000003 + layer * 7919 + _TAG[tag] * 104729) % (2 ** 63 - 1))
    return g


def prompt_lengths(w: Workload) -> list[int]:
    """Per-sequence prompt lengths (uniform in [prompt_min, prompt_max], fixed by the seed)."""
    if w.prompt_max == w.prompt_min:
        return [w.prompt_min] * w.batch
    g = _gen(w, 0, "len", "cpu")
    return torch.randint(w.prompt_min, w.prompt_max + 1, (w.batch,), generator=g).tolist()


def _randn(shape, g, device):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _outliers(k, p, scale, g, device):
    if p <= 0.0:
        return k
    hit = torch.rand(k.shape[:-1], generator=g, device=device) < p
    return torch.where(hit.unsqueeze(-1), k * scale, k)


def _lowrank_terms(w: Workload, layer: int, pos: torch.Tensor, device):
    """Rank-8 position-dependent component shared by Q and K: sum_r c_r(pos) W_r."""
    W = _randn((w.kv_heads, 8, w.head_dim), _gen(w, layer, "w", device), device)
    phi = torch.rand(8, generator=_gen(w, layer, "phi", device), device=device) * (2 * math.pi)
    r = torch.arange(1, 9, device=device, dtype=torch.float32)
    c = torch.cos(2 * math.pi * pos.to(torch.float32).unsqueeze(-1) * r / 1024.0 + phi) / math.sqrt(8.0)
    return torch.einsum("tr,hrd->thd", c, W)  # [T, Hkv, d]


def _ar1(shape, rho, g, device):
    """Unit-variance AR(1) along dim 0, realised as a 128-tap moving average of white noise."""
    T = shape[0]
    taps = 128
    e = _randn((T + taps - 1,) + tuple(shape[1:]), g, device)
    wts = (rho ** torch.arange(taps - 1, -1, -1, device=device, dtype=torch.float32)) * math.sqrt(1 - rho * rho)
    flat = e.reshape(T + taps - 1, -1).t().unsqueeze(1)           # [C, 1, T+taps-1]
    out = torch.nn.functional.conv1d(flat, wts.view(1, 1, taps))  # [C, 1, T]
    return out.squeeze(1).t().reshape(shape)


def _doc_offsets(w: Workload, layer: int, device):
    return 0.5 * _randn((w.batch, 10, w.kv_heads, w.head_dim), _gen(w, layer, "mu", device), device)


def prefill_inputs(w: Workload, layer: int, device="cpu"):
    """Returns (q, k, v, cu_seqlens) for one layer's prompt."""
    lens = prompt_lengths(w)
    total = sum(lens)
    cu = torch.tensor([0] + list(torch.tensor(lens).cumsum(0).tolist()), dtype=torch.int32, device=device)
    d = w.head_dim
    q = _randn((total, w.q_heads, d), _gen(w, layer, "q", device), device)
    k = _randn((total, w.kv_heads, d), _gen(w, layer, "k", device), device)
    v = _randn((total, w.kv_heads, d), _gen(w, layer, "v", device), device)
    pos = torch.cat([torch.arange(n, device=device) for n in lens])
    if w.keys == "lowrank":
        lr = _lowrank_terms(w, layer, pos, device)
        k = k + lr
        q = q + lr.repeat_interleave(w.group, dim=1)
    elif w.keys == "ar1":
        off = 0
        for n in lens:
            k[off:off + n] += _ar1((n, w.kv_heads, d), 0.9, _gen(w, layer * 131 + off % 127, "mu", device), device)
            off += n
    elif w.keys == "docs":
        mu = _doc_offsets(w, layer, device)
        off = 0
        for b, n in enumerate(lens):
            doc = (torch.arange(n, device=device) * 10) // n
            k[off:off + n] += mu[b][doc]
            off += n
    k = _outliers(k, w.outlier_p, w.outlier_scale, _gen(w, layer, "mask", device), device)
    dt = _DT[w.dtype]
    return q.to(dt), k.to(dt), v.to(dt), cu


def decode_inputs(w: Workload, layer: int, device="cpu", steps: int | None = None):
    """Returns (q, k, v) for `steps` decode steps of one layer, each ``[steps, batch, H, d]``."""
    S = w.decode_steps if steps is None else steps
    d = w.head_dim
    q = _randn((S, w.batch, w.q_heads, d), _gen(w, layer, "dq", device), device)
    k = _randn((S, w.batch, w.kv_heads, d), _gen(w, layer, "dk", device), device)
    v = _randn((S, w.batch, w.kv_heads, d), _gen(w, layer, "dv", device), device)
    if w.keys == "lowrank":
        lens = torch.tensor(prompt_lengths(w), device=device)
        pos = (lens.unsqueeze(0) + torch.arange(S, device=device).unsqueeze(1)).reshape(-1)  # [S*B]
        lr = _lowrank_terms(w, layer, pos, device).reshape(S, w.batch, w.kv_heads, d)
        k = k + lr
        q = q + lr.repeat_interleave(w.group, dim=2)
    elif w.keys == "ar1":
        k = k + _ar1((S, w.batch, w.kv_heads, d), 0.9, _gen(w, layer, "dmask", device), device)
    elif w.keys == "docs":
        mu = _doc_offsets(w, layer, device)
        k = k + mu[:, 9].unsqueeze(0)
    if w.keys != "ar1":
        k = _outliers(k, w.outlier_p, w.outlier_scale, _gen(w, layer, "dmask", device), device)
    dt = _DT[w.dtype]
    return q.to(dt), k.to(dt), v.to(dt)
