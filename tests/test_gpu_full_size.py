"""One layer of each benchmark workload at its FULL shape (all sequences and heads, full prompt
lengths, the launch configuration bench.py times), checked against the oracle on sampled
instances: sampled output rows one by one, the column sums of the last keys, mass conservation
of every sampled head's scores, bit-exact retained positions after the prefill-time sampling
rounds, and a few lock-step decode steps."""
import numpy as np
import pytest

import workloads
from tests.harness import run_lockstep

pytestmark = pytest.mark.gpu


def _rows(N):
    return [0, 1, 127, 128, 129, N // 3, N // 2 + 77, N - 130, N - 2]


def test_c3_full_shape_one_layer(cuda_device):
    """32768-token prompts, 4 x 32 heads, two hitters per segment of 16, budget 4096 (two sampling
    rounds at prefill)."""
    w = workloads.scaled(workloads.get("C3"), layers=1, decode_steps=3)
    stats = run_lockstep(w, [(0, 0, 0), (0, 3, 31)], sampled_rows=_rows(32768), tail_keys=48)
    assert stats["max_out_err"] < 5e-2


def test_c4_full_shape_one_layer_gqa(cuda_device):
    """8192-token prompts, 16 sequences, 32 query heads over 8 KV heads, budget 2048."""
    w = workloads.scaled(workloads.get("C4"), layers=1, decode_steps=3)
    run_lockstep(w, [(0, 0, 0), (0, 15, 7), (0, 9, 3)], sampled_rows=_rows(8192), tail_keys=64)


def test_c5_full_shape_one_layer_ragged(cuda_device):
    """32 ragged prompts of 8192..16384 tokens, per-sequence sampling rounds, budget 2048."""
    w = workloads.scaled(workloads.get("C5"), layers=1, decode_steps=3)
    lens = workloads.prompt_lengths(w)
    short, long_ = int(np.argmin(lens)), int(np.argmax(lens))
    run_lockstep(w, [(0, short, 0), (0, long_, 31), (0, 17, 13)], sampled_rows=_rows(min(lens)), tail_keys=64)


def test_c2_full_shape_extended_decode_eviction(cuda_device):
    """C2's first decode-time eviction happens at decode step 879, beyond its configured 512 steps.
    One full-shape layer is driven there (oracle in lock-step on two instances, state compared every
    64 steps and around the eviction)."""
    w = workloads.scaled(workloads.get("C2"), layers=1, decode_steps=885)
    stats = run_lockstep(w, [(0, 0, 0), (0, 7, 31)], sampled_rows=_rows(4096), tail_keys=32, check_every=64)
    assert stats["evictions"] == 2


def test_c2_full_shape_one_layer_logn(cuda_device):
    """One full-shape C2 layer with log_512(n) logit scaling (Section 3.5): sampled rows (the first
    token of a sequence, whose scale is zero, among them), tail column sums, lock-step decode."""
    w = workloads.scaled(workloads.get("C2"), layers=1, decode_steps=3)
    run_lockstep(w, [(0, 0, 0), (0, 5, 19)], sampled_rows=_rows(4096), tail_keys=48, logn=True)
