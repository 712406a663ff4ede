"""Harder prefill parity cases for the tensor-core path (bf16, d = 128): a whole instance at full
shape, a mid-prompt key block of the longest workload, and planted logits that drive the
attention kernel's speculative softmax through its slow paths."""
from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np
import pytest
import torch

import workloads
from oracle.buzz_oracle import OracleHead
from tests.harness import TOL, assert_close, assert_scores_close, make_buzz, run_lockstep

pytestmark = pytest.mark.gpu


def _np64(t):
    return t.detach().to("cpu", torch.float64).numpy()


def test_c4_one_instance_in_full(cuda_device):
    """One (sequence, KV head) instance of C4 at its full shape -- 8192 tokens, four query heads per
    KV head -- through the oracle's whole prefill: every output row and all 8192 column sums."""
    w = workloads.scaled(workloads.get("C4"), layers=1, batch=2, q_heads=4, kv_heads=1, decode_steps=2)
    stats = run_lockstep(w, [(0, 1, 0)])
    assert stats["prefill_rounds"] >= 1


def test_c3_mid_prompt_key_block(cuda_device):
    """Column sums of a key block in the middle of a 32768-token prompt (keys 4096..4159): every later
    query tile and, in the column-sum kernel, every iteration of that key tile's CTA contributes.
    The oracle replays rows 4096..N-1 as decode steps over their prefixes (Eq. 3 row by row), in
    slices run side by side, and adds up the probabilities those keys receive."""
    w = workloads.scaled(workloads.get("C3"), layers=1, batch=1, q_heads=2, kv_heads=2, decode_steps=1)
    N, d, g = w.prompt_min, w.head_dim, w.group
    bz = make_buzz(w)
    q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
    out = torch.empty_like(q)
    bz.prefill(0, q, k, v, cu, N, out)
    assert bz.status() == 0
    head, lo, hi = 1, 4096, 4160
    gpu = bz.export_prefill_scores(head, N).numpy()
    Q, K, V = _np64(q[:, head * g:(head + 1) * g]).transpose(1, 0, 2), _np64(k[:, head]), _np64(v[:, head])
    got = _np64(out[:, head * g:(head + 1) * g]).transpose(1, 0, 2)
    workers = max(1, min(os.cpu_count() or 1, 16))
    # slices of rows with equal work (row i costs ~ i)
    edges = np.sqrt(np.linspace(lo ** 2, N ** 2, 4 * workers + 1)).astype(int)
    edges[0], edges[-1] = lo, N

    def slice_sum(a, b):
        o = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, 1 << 30)
        o.set_state(0, a, np.arange(a), np.zeros(a), K[:a], V[:a])
        worst = 0.0
        for i in range(a, b):
            ref = o.decode(Q[:, i], K[i], V[i])
            if i % 512 == 0:
                worst = max(worst, float(np.abs(got[:, i] - ref).max()))
        return o.state(with_kv=False)[1][lo:hi], worst

    with ThreadPoolExecutor(max_workers=workers) as ex:
        parts = list(ex.map(lambda ab: slice_sum(*ab), zip(edges[:-1].tolist(), edges[1:].tolist())))
    ref = np.sum([p[0] for p in parts], axis=0)
    assert max(p[1] for p in parts) < 2e-2
    assert_scores_close(gpu[lo:hi], ref, "column sums of keys 4096..4159")
    bz.close()


def _planted(N, d, profile, seed):
    """Q, K, V [N, 1, d] bf16 whose logits are planted: key j has logit2[j] (log2 units, i.e. already
    multiplied by log2(e)/sqrt(d)) against EVERY query, plus small noise from the other dimensions."""
    g = torch.Generator().manual_seed(seed)
    scale_log2 = 1.4426950408889634 / np.sqrt(d)
    q = 0.05 * torch.randn(N, 1, d, generator=g)
    k = 0.05 * torch.randn(N, 1, d, generator=g)
    v = torch.randn(N, 1, d, generator=g)
    q[:, 0, 0] = 16.0                                          # exactly representable in bf16
    k[:, 0, 0] = torch.from_numpy(profile / (16.0 * scale_log2)).to(torch.float32)
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


@pytest.mark.parametrize("name", ["staircase", "cliff", "sawtooth", "descending"])
def test_planted_logits_through_the_speculative_softmax(cuda_device, name):
    """The attention kernel forms P with the row maximum in use and only looks for a new maximum when
    a tile's probabilities add up to more than 2^20. Planted logit profiles force every branch of
    that: a maximum that climbs by more than 2^8 at every 64-key tile (rescale every tile), a single
    jump large enough to overflow the tile sum to infinity, an up-and-down pattern (stale maxima
    that stay valid), and a descending profile (the first tile's maximum serves the whole row).
    Rows in the first half of a query tile have the second key tile of the diagonal fully masked."""
    N, d = 1024 + 77, 128
    j = np.arange(N)
    tile = j // 64
    if name == "staircase":
        prof = 12.0 * tile
    elif name == "cliff":
        prof = np.where(j >= 400, 300.0, 0.0) + 2.0 * (tile % 3)
    elif name == "sawtooth":
        prof = 30.0 * (tile % 2) + 9.0 * ((j // 16) % 2)
    else:
        prof = -10.0 * tile
    prof = prof.astype(np.float64)
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=2, q_heads=1, kv_heads=1, prompt_min=N, prompt_max=N,
                         decode_steps=0, window=64, budget=N + 8)
    bz = make_buzz(w)
    q0, k0, v0 = _planted(N, d, prof, 1)
    q1, k1, v1 = _planted(N, d, prof[::-1].copy() if name != "cliff" else prof, 2)
    q = torch.cat([q0, q1]).cuda(); k = torch.cat([k0, k1]).cuda(); v = torch.cat([v0, v1]).cuda()
    cu = torch.tensor([0, N, 2 * N], dtype=torch.int32, device="cuda:0")
    out = torch.empty_like(q)
    bz.prefill(0, q, k, v, cu, N, out)
    assert bz.status() == 0
    scores = bz.export_prefill_scores(0, 2 * N).numpy()
    assert np.isfinite(_np64(out)).all() and np.isfinite(scores).all()
    for b in range(2):
        sl = slice(b * N, (b + 1) * N)
        o = OracleHead(1, d, w.sink, w.window, w.segment, w.hitters, N + 8)
        O, full, _ = o.prefill(_np64(q[sl, 0])[None], _np64(k[sl, 0]), _np64(v[sl, 0]))
        assert_close(_np64(out[sl, 0]), O[0], what=f"{name} output, sequence {b}", **TOL["bf16"])
        # keys that received next to nothing are compared absolutely: their sums are far below fp32 resolution of a probability
        big = full > 1e-6
        assert_scores_close(scores[sl][big], full[big], f"{name} column sums, sequence {b}")
        assert np.abs(scores[sl][~big] - full[~big]).max(initial=0.0) < 1e-8
    bz.close()


def test_c2_full_shape_second_decode_time_eviction(cuda_device):
    """One full-shape C2 layer driven past its SECOND decode-time eviction (decode step 1984), where
    survivors of the first eviction (old tokens) and tokens that left the window since (new tokens)
    are both present; oracle in lock-step on one instance."""
    w = workloads.scaled(workloads.get("C2"), layers=1, decode_steps=1990)
    stats = run_lockstep(w, [(0, 3, 17)], sampled_rows=[0, 1, 4095], tail_keys=16, check_every=256)
    assert stats["evictions"] == 2
