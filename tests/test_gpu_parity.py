"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import workloads
from oracle.buzz_oracle import OracleHead
from tests.harness import (assert_close, assert_scores_close, compare_state, make_buzz, run_lockstep)

pytestmark = pytest.mark.gpu


def test_c1_full(cuda_device):
    """The tiny fp32 workload in full: 512-token prompt, 256 decode steps, evictions on the way."""
    w = workloads.get("C1")
    stats = run_lockstep(w, [(0, 0, 0)])
    assert stats["prefill_rounds"] == 1 and stats["evictions"] == 3


@pytest.mark.parametrize("layers_call", [False, True])
def test_c2_shape_scaled(cuda_device, layers_call):
    """Llama-2-7B head shape (bf16, d=128, MHA), low-rank + outlier keys; several key tiles and a
    ragged tail; budget small enough that decode-time evictions happen. Run once with one decode
    call per layer and once with the whole stack in one multi-layer call."""
    w = workloads.scaled(workloads.get("C2"), layers=2, batch=3, q_heads=4, kv_heads=4,
                         prompt_min=700, prompt_max=700, decode_steps=150, window=64, budget=180)
    stats = run_lockstep(w, [(0, 0, 0), (0, 2, 3), (1, 1, 2)], check_every=7, layers_call=layers_call)
    assert stats["prefill_rounds"] >= 1 and stats["evictions"] >= 3


def test_c3_shape_scaled(cuda_device):
    """Two hitters per segment of 16, AR(1) keys, prompt much longer than the budget."""
    w = workloads.scaled(workloads.get("C3"), layers=1, batch=2, q_heads=2, kv_heads=2,
                         prompt_min=1500, prompt_max=1500, decode_steps=200, window=96, budget=420)
    stats = run_lockstep(w, [(0, 0, 1), (0, 1, 0)], check_every=9)
    assert stats["evictions"] >= 2


def test_c4_shape_scaled_gqa(cuda_device):
    """Grouped-query attention: 4 query heads per KV head, scores summed over the group."""
    w = workloads.scaled(workloads.get("C4"), layers=2, batch=2, q_heads=8, kv_heads=2,
                         prompt_min=900, prompt_max=900, decode_steps=130, window=64, budget=300)
    stats = run_lockstep(w, [(0, 1, 0), (1, 0, 1)], check_every=5)
    assert stats["evictions"] >= 2


def test_c5_shape_scaled_ragged(cuda_device):
    """Ragged prompts, per-sequence eviction triggers."""
    w = workloads.scaled(workloads.get("C5"), layers=1, batch=4, q_heads=2, kv_heads=2,
                         prompt_min=300, prompt_max=900, decode_steps=180, window=48, budget=200)
    lens = workloads.prompt_lengths(w)
    assert len(set(lens)) > 1
    stats = run_lockstep(w, [(0, b, b % 2) for b in range(4)], check_every=6)
    assert stats["evictions"] >= 4


def test_logn_scaling(cuda_device):
    """log_512(n) logit scaling (Section 3.5) in prefill and decode."""
    w = workloads.scaled(workloads.get("C1"), prompt_min=200, prompt_max=200, decode_steps=40)
    run_lockstep(w, [(0, 0, 0)], logn=True)


@pytest.mark.parametrize("topk", [False, True])
def test_eviction_with_a_middle_region_too_large_to_stage(cuda_device, topk):
    """Middle regions beyond the size whose scores and positions the eviction copies to shared memory
    take the path that selects straight from global memory; same bit-exact bar, both policies."""
    rng = np.random.default_rng(77 + topk)
    sink, window, segment, hitters, d = 4, 32, 16, 2, 64
    T = 6000
    budget = sink + window + T
    w = workloads.scaled(workloads.get("C1"), batch=3, q_heads=1, kv_heads=1, sink=sink, window=window,
                         segment=segment, hitters=hitters, budget=budget, head_dim=d, dtype="bf16")
    bz = make_buzz(w, max_prompt_tokens=64)
    bz.set_policy(topk)
    cases = []
    for b, n_old in enumerate([0, T // 2 + 3, T]):
        pos, score, k, v = _random_state(rng, budget, d, torch.bfloat16, 7)
        bz.import_state(0, b, 0, n_old, int(pos[-1]) + 1, torch.from_numpy(pos), torch.from_numpy(score), k, v)
        orc = OracleHead(1, d, sink, window, segment, hitters, budget)
        orc.set_policy(topk)
        orc.set_state(n_old, int(pos[-1]) + 1, pos, score.astype(np.float64), k.double().numpy(), v.double().numpy())
        cases.append((b, orc))
    bz.evict(0)
    assert bz.status() == 0
    for b, orc in cases:
        assert orc.evict() == 1
        compare_state(bz, orc, 0, b, 0, f"large middle region b{b}", exact_scores=True)
    bz.close()


@pytest.mark.parametrize("name,over,samples", [
    ("C2", dict(layers=2, batch=2, q_heads=4, kv_heads=4, prompt_min=700, prompt_max=700, decode_steps=150,
                window=64, budget=180), [(0, 0, 0), (1, 1, 3)]),
    ("C4", dict(layers=1, batch=2, q_heads=8, kv_heads=2, prompt_min=900, prompt_max=900, decode_steps=130,
                window=64, budget=300), [(0, 1, 0), (0, 0, 1)]),
    ("C5", dict(layers=1, batch=3, q_heads=2, kv_heads=2, prompt_min=130, prompt_max=600, decode_steps=90,
                window=48, budget=120), [(0, 0, 0), (0, 1, 1), (0, 2, 0)]),
])
def test_logn_scaling_on_the_tensor_core_path(cuda_device, name, over, samples):
    """log_512(n) scaling on bf16, d = 128: the TMA/tcgen05 prefill kernels (prompts of several key
    tiles with a ragged tail, MHA and GQA) and the tensor-core decode kernel, through prefill-time
    sampling rounds and decode-time evictions (where tokens seen and retained slots differ). Every
    output row is compared, so the first token of each sequence (scale 0) is covered."""
    w = workloads.scaled(workloads.get(name), **over)
    stats = run_lockstep(w, samples, check_every=7, logn=True)
    assert stats["evictions"] >= 2 and np.isfinite(stats["max_out_err"])


@pytest.mark.parametrize("N", [1, 3, 40, 68, 69, 159, 160, 161, 700])
def test_prompt_length_edges(cuda_device, N):
    """Prompts shorter than sink+window (Remark 1), just below / at / above the budget, and far
    above it (Remark 2: several sampling rounds)."""
    w = workloads.scaled(workloads.get("C1"), prompt_min=N, prompt_max=N, decode_steps=5,
                         budget=160 if N < 700 else 84)
    run_lockstep(w, [(0, 0, 0)])


@pytest.mark.parametrize("dtype,d,g", [("bf16", 64, 1), ("bf16", 64, 2), ("f32", 128, 1), ("f32", 64, 4),
                                       ("bf16", 128, 8)])
def test_dtype_headdim_group_matrix(cuda_device, dtype, d, g):
    w = workloads.scaled(workloads.get("C4"), layers=1, batch=2, q_heads=2 * g, kv_heads=2, head_dim=d,
                         dtype=dtype, prompt_min=200, prompt_max=200, decode_steps=70, window=32,
                         budget=128, segment=5, hitters=2)
    stats = run_lockstep(w, [(0, 0, 0), (0, 1, 1)], check_every=3)
    assert stats["evictions"] >= 2


@pytest.mark.parametrize("name,over", [
    ("C1", dict(prompt_min=3, prompt_max=3, decode_steps=230, sink=2, window=16, segment=4, budget=41)),
    ("C2", dict(layers=1, batch=2, q_heads=2, kv_heads=2, prompt_min=9, prompt_max=9, decode_steps=260, sink=4,
                window=24, segment=5, hitters=2, budget=64)),
    ("C4", dict(layers=1, batch=1, q_heads=4, kv_heads=1, prompt_min=30, prompt_max=30, decode_steps=150, sink=0,
                window=1, segment=3, budget=20)),
])
def test_window_ring_from_empty_to_many_rotations(cuda_device, name, over):
    """The window lives in a ring behind the sink. Starting from a prompt shorter than sink + window,
    the ring first fills in order, then every step replaces its oldest token (which moves to the end
    of the middle region, score and position included), and evictions compact the middle only. The
    ring goes round many times here; every step and every eviction is checked against the oracle,
    whose cache is in plain position order. Also the degenerate ring of one slot with no sink."""
    w = workloads.scaled(workloads.get(name), **over)
    samples = [(0, b, w.kv_heads - 1) for b in range(w.batch)]
    stats = run_lockstep(w, samples, check_every=1)
    assert stats["evictions"] >= 8


def test_export_import_round_trip_with_a_rotated_ring(cuda_device):
    """A cache exported mid-run (ring head somewhere in the middle) and imported into a fresh object
    continues to the same results: the exported arrays are in position order whatever the ring's
    phase. (The import restarts the ring at head 0, so the slot order, and with it the fp32 summation
    order, differs between the two objects: outputs and scores agree to rounding, not bit for bit.)"""
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=1, q_heads=2, kv_heads=2, prompt_min=200,
                         prompt_max=200, decode_steps=120, window=32, budget=100)
    a, b = make_buzz(w), make_buzz(w)
    q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
    a.prefill(0, q, k, v, cu, 200, torch.empty_like(q))
    qd, kd, vd = workloads.decode_inputs(w, 0, "cuda:0")
    o = torch.empty_like(qd[0])
    for t in range(45):                                 # 45 steps: the head is at ring index 13
        a.decode_step(0, qd[t], kd[t], vd[t], o); a.evict(0)
    for h in range(2):
        st = a.export_state(0, 0, h)
        assert torch.all(st["pos"][1:] > st["pos"][:-1])                       # position order
        assert st["pos"][-32:].tolist() == list(range(245 - 32, 245))           # the window, un-rotated
        b.import_state(0, 0, h, st["n_old"], st["total_len"], st["pos"], st["score"], st["k"], st["v"])
    for t in range(45, w.decode_steps):
        oa, ob = torch.empty_like(qd[t]), torch.empty_like(qd[t])
        a.decode_step(0, qd[t], kd[t], vd[t], oa); a.evict(0)
        b.decode_step(0, qd[t], kd[t], vd[t], ob); b.evict(0)
        torch.testing.assert_close(oa.float(), ob.float(), atol=1e-2, rtol=1e-2)
    for h in range(2):
        x, y = a.export_state(0, 0, h), b.export_state(0, 0, h)
        assert (x["n"], x["n_old"], x["total_len"]) == (y["n"], y["n_old"], y["total_len"])
        for key in ("pos", "k", "v"):
            assert torch.equal(x[key], y[key])
        torch.testing.assert_close(x["score"], y["score"], atol=0.0, rtol=1e-4)
    assert a.status() == 0 and b.status() == 0
    a.close(); b.close()


@pytest.mark.parametrize("name,over,layers_call", [
    ("C2", dict(layers=3, batch=2, q_heads=4, kv_heads=4, prompt_min=300, prompt_max=300, decode_steps=160,
                window=32, budget=100), False),
    ("C4", dict(layers=2, batch=3, q_heads=8, kv_heads=2, prompt_min=150, prompt_max=420, decode_steps=140,
                window=48, budget=150, segment=16, hitters=2), True),
    ("C1", dict(layers=2, batch=2, q_heads=2, kv_heads=2, prompt_min=100, prompt_max=100, decode_steps=150,
                window=16, budget=60), False),
])
def test_fused_eviction_matches_separate_calls(cuda_device, name, over, layers_call):
    """Fused mode: a decode step that fills a cache evicts it in the kernel's own tail. Outputs of every
    step and the final caches must equal, bit for bit, decode step + buzz_evict in the default mode
    (which the lock-step tests check against the oracle); in fused mode buzz_evict launches nothing."""
    w = workloads.scaled(workloads.get(name), **over)
    lens = workloads.prompt_lengths(w)
    pre, dec = _stack(w)
    ref, fused = make_buzz(w), make_buzz(w)
    fused.set_fused_evict(True)
    for bz in (ref, fused):
        for l in range(w.layers):
            q, k, v, cu = pre[l]
            bz.prefill(l, q, k, v, cu, max(lens), torch.empty_like(q))
    L = list(range(w.layers))
    evict_launches = 0
    for t in range(w.decode_steps):
        o_ref = [torch.empty_like(dec[l][0][t]) for l in L]
        o_fus = [torch.empty_like(dec[l][0][t]) for l in L]
        for bz, outs in ((ref, o_ref), (fused, o_fus)):
            if layers_call:
                bz.decode_layers(L, [dec[l][0][t] for l in L], [dec[l][1][t] for l in L], [dec[l][2][t] for l in L], outs)
            else:
                for l in L:
                    bz.decode_step(l, dec[l][0][t], dec[l][1][t], dec[l][2][t], outs[l])
        ref.evict(-1)
        before = fused.launch_count()
        fused.evict(-1 if t % 2 else 0)
        evict_launches += fused.launch_count() - before
        for l in L:
            assert torch.equal(o_ref[l], o_fus[l]), f"step {t} layer {l}"
    assert evict_launches == 0
    evicted = False
    for l in L:
        for b in range(w.batch):
            for h in range(w.kv_heads):
                x, y = ref.export_state(l, b, h), fused.export_state(l, b, h)
                assert (x["n"], x["n_old"], x["total_len"]) == (y["n"], y["n_old"], y["total_len"]), (l, b, h)
                for key in ("pos", "score", "k", "v"):
                    assert torch.equal(x[key], y[key]), (l, b, h, key)
                evicted |= x["n"] < lens[b] + w.decode_steps and x["n_old"] > 0
    assert evicted and ref.status() == 0 and fused.status() == 0
    ref.close(); fused.close()


def _random_state(rng, n, d, dtype, quantum):
    pos = np.sort(rng.choice(10 * n, size=n, replace=False)).astype(np.int32)
    score = rng.random(n).astype(np.float32)
    if quantum:
        score = (np.round(score * quantum) / quantum).astype(np.float32)   # exact ties
    k = torch.randn(n, d, generator=torch.Generator().manual_seed(int(rng.integers(1 << 30)))).to(dtype)
    v = torch.randn(n, d, generator=torch.Generator().manual_seed(int(rng.integers(1 << 30)))).to(dtype)
    return pos, score, k, v


@pytest.mark.parametrize("segment,hitters,quantum", [(8, 1, 0), (8, 1, 4), (16, 2, 3), (5, 3, 2), (40, 7, 5),
                                                    (3, 1, 2), (100, 33, 6)])
def test_eviction_bit_exact_on_planted_states(cuda_device, segment, hitters, quantum):
    """Planted cache states with exact score ties: indices, positions, scores and rows must match
    the oracle bit for bit, for full caches with every possible n_old class and for caches below
    the budget (which must be left alone)."""
    rng = np.random.default_rng(segment * 131 + hitters)
    sink, window, budget, d = 3, 17, 3 + 17 + 3 * segment + 57, 64
    w = workloads.scaled(workloads.get("C1"), batch=6, q_heads=2, kv_heads=2, sink=sink, window=window,
                         segment=segment, hitters=hitters, budget=budget, head_dim=d, dtype="bf16")
    bz = make_buzz(w, max_prompt_tokens=64)
    T = budget - sink - window
    cases = []
    for b in range(6):
        for h in range(2):
            n = budget if b < 5 else budget - 1 - h
            n_old = [0, T, T // 2, 1, T - 1, 5][b]
            n_old = min(n_old, n - sink - window)
            pos, score, k, v = _random_state(rng, n, d, torch.bfloat16, quantum)
            bz.import_state(0, b, h, n_old, int(pos[-1]) + 1, torch.from_numpy(pos), torch.from_numpy(score), k, v)
            orc = OracleHead(1, d, sink, window, segment, hitters, budget)
            orc.set_state(n_old, int(pos[-1]) + 1, pos, score.astype(np.float64), k.double().numpy(), v.double().numpy())
            cases.append((b, h, orc, n))
    bz.evict(0)
    assert bz.status() == 0
    for b, h, orc, n in cases:
        r = orc.evict()
        assert r == (1 if n >= budget else 0)
        compare_state(bz, orc, 0, b, h, f"planted b{b} h{h}", exact_scores=True)
    bz.evict(-1)                       # a second call must be a no-op everywhere
    for b, h, orc, n in cases:
        compare_state(bz, orc, 0, b, h, f"planted again b{b} h{h}", exact_scores=True)
    bz.close()


@pytest.mark.parametrize("topk", [False, True])
def test_eviction_with_a_middle_region_too_large_to_stage(cuda_device, topk):
    """Middle regions beyond the size whose scores and positions the eviction copies to shared memory
    take the path that selects straight from global memory; same bit-exact bar, both policies."""
    rng = np.random.default_rng(77 + topk)
    sink, window, segment, hitters, d = 4, 32, 16, 2, 64
    T = 6000
    budget = sink + window + T
    w = workloads.scaled(workloads.get("C1"), batch=3, q_heads=1, kv_heads=1, sink=sink, window=window,
                         segment=segment, hitters=hitters, budget=budget, head_dim=d, dtype="bf16")
    bz = make_buzz(w, max_prompt_tokens=64)
    bz.set_policy(topk)
    cases = []
    for b, n_old in enumerate([0, T // 2 + 3, T]):
        pos, score, k, v = _random_state(rng, budget, d, torch.bfloat16, 7)
        bz.import_state(0, b, 0, n_old, int(pos[-1]) + 1, torch.from_numpy(pos), torch.from_numpy(score), k, v)
        orc = OracleHead(1, d, sink, window, segment, hitters, budget)
        orc.set_policy(topk)
        orc.set_state(n_old, int(pos[-1]) + 1, pos, score.astype(np.float64), k.double().numpy(), v.double().numpy())
        cases.append((b, orc))
    bz.evict(0)
    assert bz.status() == 0
    for b, orc in cases:
        assert orc.evict() == 1
        compare_state(bz, orc, 0, b, 0, f"large middle region b{b}", exact_scores=True)
    bz.close()


@pytest.mark.parametrize("name,over,samples", [
    ("C2", dict(layers=2, batch=2, q_heads=4, kv_heads=4, prompt_min=700, prompt_max=700, decode_steps=150,
                window=64, budget=180), [(0, 0, 0), (1, 1, 3)]),
    ("C4", dict(layers=1, batch=2, q_heads=8, kv_heads=2, prompt_min=2100, prompt_max=2100, decode_steps=270,
                window=64, budget=300), [(0, 1, 0), (0, 0, 1)]),
    ("C3", dict(layers=1, batch=2, q_heads=2, kv_heads=2, prompt_min=300, prompt_max=1500, decode_steps=400,
                window=96, budget=420), [(0, 0, 1), (0, 1, 0)]),
    ("C1", dict(prompt_min=512, prompt_max=512, decode_steps=256), [(0, 0, 0)]),
])
def test_global_topk_policy_lockstep(cuda_device, name, over, samples):
    """The heavy-hitter policy (global top-k of the accumulated scores instead of the sampling module):
    prefill-time rounds (one and several) and decode-time evictions, lock-step against the oracle --
    selected positions bit-exact when the oracle decides on the GPU's scores."""
    w = workloads.scaled(workloads.get(name), **over)
    stats = run_lockstep(w, samples, check_every=7, topk=True)
    assert stats["prefill_rounds"] >= 1 and stats["evictions"] >= 2


@pytest.mark.parametrize("T,segment,hitters,quantum", [(200, 8, 1, 3), (1500, 16, 2, 5), (700, 5, 1, 1), (300, 40, 7, 0)])
def test_global_topk_bit_exact_on_planted_states(cuda_device, T, segment, hitters, quantum):
    """Planted full caches, middle regions of several hundred slots with heavily tied scores (down to
    two distinct values, so the cut falls inside a run of equal scores): positions, scores and rows
    must match the oracle bit for bit; both in a separate eviction call and in the fused tail."""
    rng = np.random.default_rng(T + segment)
    sink, window, d = 3, 17, 64
    budget = sink + window + T
    w = workloads.scaled(workloads.get("C1"), batch=4, q_heads=2, kv_heads=2, sink=sink, window=window,
                         segment=segment, hitters=hitters, budget=budget, head_dim=d, dtype="bf16")
    bz = make_buzz(w, max_prompt_tokens=64)
    bz.set_policy(True)
    cases = []
    for b in range(4):
        for h in range(2):
            n = budget if b < 3 else budget - 1
            n_old = min([0, T, T // 3, 7][b], n - sink - window)
            pos, score, k, v = _random_state(rng, n, d, torch.bfloat16, quantum)
            bz.import_state(0, b, h, n_old, int(pos[-1]) + 1, torch.from_numpy(pos), torch.from_numpy(score), k, v)
            orc = OracleHead(1, d, sink, window, segment, hitters, budget)
            orc.set_policy(True)
            orc.set_state(n_old, int(pos[-1]) + 1, pos, score.astype(np.float64), k.double().numpy(), v.double().numpy())
            cases.append((b, h, orc, n))
    bz.evict(0)
    assert bz.status() == 0
    for b, h, orc, n in cases:
        assert orc.evict() == (1 if n >= budget else 0)
        compare_state(bz, orc, 0, b, h, f"planted top-k b{b} h{h}", exact_scores=True)
    # sequence 3 is one token short of its budget: one fused decode step fills and evicts it in the tail
    bz.set_fused_evict(True)
    q = torch.randn(4, 2, d, device="cuda:0").to(torch.bfloat16)
    kn, vn = torch.randn(4, 2, d, device="cuda:0").to(torch.bfloat16), torch.randn(4, 2, d, device="cuda:0").to(torch.bfloat16)
    out = torch.empty_like(q)
    bz.decode_step(0, q, kn, vn, out)
    assert bz.status() == 0
    for b, h, orc, n in cases:
        orc.decode(q[b, h:h + 1].double().cpu().numpy(), kn[b, h].double().cpu().numpy(), vn[b, h].double().cpu().numpy())
        st = bz.export_state(0, b, h)
        if b == 3:                                       # evicted in the tail: only the post-eviction state exists
            assert st["n"] < budget
            # the oracle decides on its own scores here; with ~T candidates a near-tie flip is possible,
            # so compare what is unique: counts, sink and window positions
            assert orc.evict() == 1
            assert (st["n"], st["n_old"]) == orc.counts()[:2]
            opos = orc.state(with_kv=False)[0]
            assert st["pos"][:sink].tolist() == opos[:sink].tolist() and st["pos"][-window:].tolist() == opos[-window:].tolist()
        else:
            compare_state(bz, orc, 0, b, h, f"planted top-k after a step b{b} h{h}", exact_scores=False)
    bz.close()


def test_fused_mode_with_very_large_budgets(cuda_device):
    """Fused mode keeps the eviction's work area in the decode CTA's shared memory. A budget of 20000
    slots still fits (instance split over 8 CTAs, selection straight from global memory): one fused
    step on a cache one token short of full evicts in the kernel's tail, and the counters follow the
    oracle's schedule. A budget of 32768 with 8 query heads per KV head does not fit: refused."""
    from paper_2410_23079_b200 import BuzzError
    rng = np.random.default_rng(5)
    sink, window, segment, hitters, d, budget = 4, 64, 16, 1, 128, 20000
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=1, q_heads=4, kv_heads=1, sink=sink, window=window,
                         segment=segment, hitters=hitters, budget=budget)
    bz = make_buzz(w, max_prompt_tokens=64)
    bz.set_fused_evict(True)
    n = budget - 1
    pos, score, k, v = _random_state(rng, n, d, torch.bfloat16, 0)
    n_old = 5000
    bz.import_state(0, 0, 0, n_old, int(pos[-1]) + 1, torch.from_numpy(pos), torch.from_numpy(score), k, v)
    orc = OracleHead(4, d, sink, window, segment, hitters, budget)
    orc.set_state(n_old, int(pos[-1]) + 1, pos, score.astype(np.float64), k.double().numpy(), v.double().numpy())
    q = torch.randn(1, 4, d, device="cuda:0").to(torch.bfloat16)
    kn, vn = torch.randn(1, 1, d, device="cuda:0").to(torch.bfloat16), torch.randn(1, 1, d, device="cuda:0").to(torch.bfloat16)
    out = torch.empty_like(q)
    bz.decode_step(0, q, kn, vn, out)
    assert bz.status() == 0
    ref = orc.decode(q[0].double().cpu().numpy(), kn[0, 0].double().cpu().numpy(), vn[0, 0].double().cpu().numpy())
    assert_close(out[0].double().cpu().numpy(), ref, what="fused step output", atol=2e-2, rtol=1e-2)
    assert orc.evict() == 1
    st = bz.export_state(0, 0, 0)
    assert (st["n"], st["n_old"], st["total_len"]) == orc.counts()
    opos = orc.state(with_kv=False)[0]
    assert st["pos"][:sink].tolist() == opos[:sink].tolist() and st["pos"][-window:].tolist() == opos[-window:].tolist()
    assert np.all(np.diff(st["pos"].numpy()) > 0)
    bz.close()
    big = workloads.scaled(workloads.get("C2"), layers=1, batch=1, q_heads=8, kv_heads=1, budget=32768)
    bz = make_buzz(big, max_prompt_tokens=64)
    with pytest.raises(BuzzError) as ei:
        bz.set_fused_evict(True)
    assert ei.value.code == -6
    bz.close()


def test_policy_validation(cuda_device):
    from paper_2410_23079_b200 import BuzzError
    w = workloads.scaled(workloads.get("C1"))
    bz = make_buzz(w, max_prompt_tokens=64)
    with pytest.raises(BuzzError):
        bz._lib.buzz_set_policy  # noqa: B018  (symbol exists)
        from paper_2410_23079_b200.binding import _check
        _check(bz._lib.buzz_set_policy(bz._h, 7), "buzz_set_policy")
    bz.set_policy(True); bz.set_policy(False)
    bz.close()


def test_decode_cluster_sizes_agree(cuda_device):
    """The split of an instance over 1, 2, 4 or 8 CTAs changes only the fp32 summation order."""
    w = workloads.scaled(workloads.get("C4"), layers=1, batch=2, q_heads=8, kv_heads=2,
                         prompt_min=333, prompt_max=333, decode_steps=3, window=64, budget=400)
    ref = None
    for cs in (1, 2, 4, 8):
        bz = make_buzz(w)
        bz.set_decode_cluster(cs)
        run_lockstep(w, [(0, 1, 1)], bz=bz)
        st = bz.export_state(0, 1, 1)
        if ref is None:
            ref = st
        else:
            assert torch.equal(st["pos"], ref["pos"])
            assert_scores_close(st["score"].numpy(), ref["score"].numpy(), f"cluster {cs}")
        bz.close()


def test_deterministic(cuda_device):
    """Two runs on the same inputs give bit-identical caches and outputs."""
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=2, q_heads=2, kv_heads=2,
                         prompt_min=500, prompt_max=500, decode_steps=90, window=32, budget=150)
    snaps = []
    for _ in range(2):
        bz = make_buzz(w)
        q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
        out = torch.empty_like(q)
        bz.prefill(0, q, k, v, cu, 500, out)
        qd, kd, vd = workloads.decode_inputs(w, 0, "cuda:0")
        outs = [out.clone()]
        for t in range(w.decode_steps):
            o = torch.empty_like(qd[t])
            bz.decode_step(0, qd[t], kd[t], vd[t], o)
            bz.evict(0)
            outs.append(o)
        assert bz.status() == 0
        snaps.append((outs, [bz.export_state(0, b, h) for b in range(2) for h in range(2)]))
        bz.close()
    for a, b in zip(snaps[0][0], snaps[1][0]):
        assert torch.equal(a, b)
    for a, b in zip(snaps[0][1], snaps[1][1]):
        assert a["n"] == b["n"] and a["n_old"] == b["n_old"]
        for key in ("pos", "score", "k", "v"):
            assert torch.equal(a[key], b[key])


def test_overflow_status(cuda_device):
    w = workloads.scaled(workloads.get("C1"), prompt_min=100, prompt_max=100, budget=104, window=64)
    bz = make_buzz(w)
    q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
    bz.prefill(0, q, k, v, cu, 100, torch.empty_like(q))
    qd, kd, vd = workloads.decode_inputs(w, 0, "cuda:0", steps=6)
    o = torch.empty_like(qd[0])
    for t in range(4):
        bz.decode_step(0, qd[t], kd[t], vd[t], o)
    assert bz.status() == 0 and bz.export_state(0, 0, 0)["n"] == 104
    bz.decode_step(0, qd[4], kd[4], vd[4], o)          # cache full and no evict: must be refused
    assert bz.status() == -2
    assert bz.status() == 0                            # reading clears it
    assert bz.export_state(0, 0, 0)["n"] == 104        # and the sequence was left untouched
    bz.close()


def test_bounded_wait_expiry_is_reported_and_survivable(cuda_device):
    """A bounded on-device wait that nobody satisfies gives up by itself: the kernel ends, the status
    word reports BUZZ_ERR_TIMEOUT once, and the same object then runs a normal prefill + decode +
    evict to the oracle's result."""
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=1, q_heads=2, kv_heads=2, prompt_min=300,
                         prompt_max=300, decode_steps=30, window=32, budget=96)
    bz = make_buzz(w)
    bz.selftest_wait_expiry(1024)
    assert bz.status() == -4                           # BUZZ_ERR_TIMEOUT
    assert bz.status() == 0                            # reading clears it
    stats = run_lockstep(w, [(0, 0, 1)], bz=bz)        # the context and the object are intact
    assert stats["evictions"] >= 1 and bz.status() == 0
    bz.close()


def test_no_progress_status(cuda_device):
    """segment = 2 gives s_hat = 1: a cache full of old tokens cannot shrink; reported, not looped."""
    w = workloads.scaled(workloads.get("C1"), sink=1, window=2, segment=2, hitters=1, budget=8,
                         head_dim=64, dtype="f32")
    bz = make_buzz(w, max_prompt_tokens=16)
    n = 8
    pos = torch.arange(n, dtype=torch.int32)
    bz.import_state(0, 0, 0, n - 3, n, pos, torch.rand(n), torch.randn(n, 64), torch.randn(n, 64))
    bz.evict(0)
    assert bz.status() == -3
    bz.close()


def test_invalid_arguments_are_rejected(cuda_device):
    from paper_2410_23079_b200 import Buzz, BuzzError
    base = dict(sink=4, window=8, segment=4, hitters=1, budget=32, layers=1, max_batch=1, q_heads=2,
                kv_heads=2, head_dim=64, dtype=torch.float32, max_prompt_tokens=64)
    for bad in [dict(segment=1), dict(hitters=4), dict(window=0), dict(budget=15), dict(head_dim=96),
                dict(q_heads=3), dict(sink=-1)]:
        with pytest.raises(BuzzError):
            Buzz(**{**base, **bad})
    bz = Buzz(**base)
    t = torch.zeros(64, 2, 64, device="cuda:0")
    cu = torch.tensor([0, 64], dtype=torch.int32, device="cuda:0")
    with pytest.raises(BuzzError):
        bz.prefill(1, t, t, t, cu, 64, t)              # layer out of range
    with pytest.raises(BuzzError):
        bz.prefill(0, t[:1].expand(65, 2, 64), t, t, cu, 64, t)   # more tokens than sized for
    bz.close()


def test_full_size_c2_layer_sampled(cuda_device):
    """One layer at the benchmark's full C2 shape (batch 8, 32 heads, 4096-token prompts, budget
    1843), in the launch configuration bench.py times; the oracle checks three sampled instances,
    and a conservation law checks every head: the prompt scores of a head sum to g * tokens."""
    w = workloads.scaled(workloads.get("C2"), layers=1, decode_steps=3)
    bz = make_buzz(w)
    run_lockstep(w, [(0, 0, 0), (0, 7, 31), (0, 3, 17)], bz=bz)
    total = w.batch * w.prompt_min
    for h in range(0, w.kv_heads, 5):
        s = bz.export_prefill_scores(h, total).double().sum().item()
        assert abs(s - w.group * total) <= 1e-4 * total
    bz.close()


def test_prefill_is_reproducible_at_full_size(cuda_device):
    """Three prefills of one full-size C2 layer (8 x 32 heads x 4096 tokens, every SM busy with many
    tiles in flight) must agree bit for bit in outputs, prompt scores and caches: an ordering
    mistake between asynchronous tensor-core operations shows up here as run-to-run noise."""
    w = workloads.scaled(workloads.get("C2"), layers=1)
    bz = make_buzz(w)
    q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
    ref_out = ref_sc = ref_st = None
    for run in range(3):
        out = torch.zeros_like(q)
        bz.prefill(0, q, k, v, cu, 4096, out)
        assert bz.status() == 0
        sc = torch.stack([bz.export_prefill_scores(h, 8 * 4096) for h in range(0, 32, 3)])
        st = bz.export_state(0, 5, 11)
        if run == 0:
            ref_out, ref_sc, ref_st = out, sc, st
        else:
            assert torch.equal(out, ref_out), f"run {run}: {(out != ref_out).sum().item()} outputs differ"
            assert torch.equal(sc, ref_sc)
            assert torch.equal(st["pos"], ref_st["pos"]) and torch.equal(st["score"], ref_st["score"])
    bz.close()


@pytest.mark.parametrize("sampling", [(False, 4, 8), (True, 8, 4), (True, 5, 3)])
def test_sampling_variants_of_the_ablation_study(cuda_device, sampling):
    """Section 4.3 variants (swapped strides; interval sampling for new tokens) through prefill-time
    rounds and decode-time evictions, lock-step against the oracle."""
    w = workloads.scaled(workloads.get("C2"), layers=2, batch=2, q_heads=2, kv_heads=2, prompt_min=650,
                         prompt_max=650, decode_steps=120, window=48, budget=150, hitters=1)
    stats = run_lockstep(w, [(0, 0, 0), (1, 1, 1)], check_every=7, sampling=sampling)
    assert stats["evictions"] >= 2


def test_sampling_variant_validation(cuda_device):
    from paper_2410_23079_b200 import BuzzError
    w = workloads.scaled(workloads.get("C1"), hitters=3, segment=8, budget=120)
    bz = make_buzz(w, max_prompt_tokens=64)
    for bad in [(False, 1, 2), (False, 3, 2), (False, 8, 0), (False, 60, 2)]:
        with pytest.raises(BuzzError):
            bz.set_sampling(*bad)
    bz.set_sampling(True, 8, 4)
    bz.close()


def test_decode_step_host_matches_device_entry(cuda_device):
    """The host-buffer entry point (separate and packed q|k|v records) gives bit-identical outputs and
    caches to the device-pointer entry point."""
    w = workloads.scaled(workloads.get("C4"), layers=1, batch=2, q_heads=8, kv_heads=2, prompt_min=260,
                         prompt_max=260, decode_steps=6, window=32, budget=300)
    q, k, v, cu = workloads.prefill_inputs(w, 0, "cuda:0")
    qd, kd, vd = workloads.decode_inputs(w, 0, "cuda:0")
    ref, sep, packed, paged = make_buzz(w), make_buzz(w), make_buzz(w), make_buzz(w)
    for bz in (ref, sep, packed, paged):
        bz.prefill(0, q, k, v, cu, 260, torch.empty_like(q))
    nq, nk = qd[0].numel(), kd[0].numel()
    for t in range(w.decode_steps):
        o_ref = torch.empty_like(qd[t])
        ref.decode_step(0, qd[t], kd[t], vd[t], o_ref)
        hq, hk, hv = qd[t].cpu().pin_memory(), kd[t].cpu().pin_memory(), vd[t].cpu().pin_memory()
        o_sep = torch.empty_like(hq).pin_memory()
        sep.decode_step_host(0, hq, hk, hv, o_sep)
        rec = torch.cat([hq.reshape(-1), hk.reshape(-1), hv.reshape(-1)]).pin_memory()
        o_pk = torch.empty_like(hq).pin_memory()
        packed.decode_step_host(0, rec[:nq], rec[nq:nq + nk], rec[nq + nk:], o_pk)
        rec_p = torch.empty(rec.shape, dtype=rec.dtype).copy_(rec)      # pageable memory: staged copies
        o_pg = torch.empty(hq.shape, dtype=hq.dtype)
        paged.decode_step_host(0, rec_p[:nq], rec_p[nq:nq + nk], rec_p[nq + nk:], o_pg)
        torch.cuda.synchronize()
        assert torch.equal(o_sep, o_ref.cpu()) and torch.equal(o_pk, o_ref.cpu()) and torch.equal(o_pg, o_ref.cpu())
    for bz in (sep, packed, paged):
        for b in range(2):
            a, c = ref.export_state(0, b, 1), bz.export_state(0, b, 1)
            assert a["n"] == c["n"] and torch.equal(a["score"], c["score"]) and torch.equal(a["k"], c["k"])
        assert bz.status() == 0
    for bz in (ref, sep, packed, paged):
        bz.close()


def _stack(w, device="cuda:0"):
    pre = [workloads.prefill_inputs(w, l, device) for l in range(w.layers)]
    dec = [workloads.decode_inputs(w, l, device) for l in range(w.layers)]
    return pre, dec


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [dict(batch=2, q_heads=8, kv_heads=2), dict(batch=1, q_heads=2, kv_heads=2),
                                   dict(batch=3, q_heads=16, kv_heads=16)])
def test_decode_layers_matches_single_layer_calls(cuda_device, shape):
    """One multi-layer call per step (device pointers, and packed host buffers) leaves bit-identical
    outputs, scores and caches to one buzz_decode_step per layer, across evictions, for any order of
    the layers, with and without an eviction call between steps."""
    w = workloads.scaled(workloads.get("C4"), layers=4, prompt_min=150, prompt_max=150, decode_steps=40,
                         window=32, budget=180, **shape)
    pre, dec = _stack(w)
    ref, multi, host, paged = make_buzz(w), make_buzz(w), make_buzz(w), make_buzz(w)
    for bz in (ref, multi, host, paged):
        bz.set_decode_cluster(2)          # same split of the slots in both entry points: bit-identical sums
        for l in range(w.layers):
            q, k, v, cu = pre[l]
            bz.prefill(l, q, k, v, cu, 150, torch.empty_like(q))
    orders = [[0, 1, 2, 3], [3, 1, 0, 2], [2, 0, 3, 1]]
    for t in range(w.decode_steps):
        order = orders[t % 3]
        o_ref = {l: torch.empty_like(dec[l][0][t]) for l in order}
        for l in order:
            ref.decode_step(l, dec[l][0][t], dec[l][1][t], dec[l][2][t], o_ref[l])
        o_m = {l: torch.empty_like(dec[l][0][t]) for l in order}
        multi.decode_layers(order, [dec[l][0][t] for l in order], [dec[l][1][t] for l in order],
                            [dec[l][2][t] for l in order], [o_m[l] for l in order])
        rec = torch.cat([torch.cat([dec[l][i][t].reshape(-1) for i in range(3)]) for l in order]).cpu().pin_memory()
        o_h = torch.empty(sum(o_ref[l].numel() for l in order), dtype=rec.dtype).pin_memory()
        host.decode_layers_host(order, rec, o_h)          # pinned: read and written in place by the kernels
        rec_p = torch.empty(rec.shape, dtype=rec.dtype).copy_(rec)      # pageable: through the staging area
        o_p = torch.empty(o_h.shape, dtype=o_h.dtype)
        assert not rec_p.is_pinned() and not o_p.is_pinned()
        paged.decode_layers_host(order, rec_p, o_p)
        if t % 2 == 0 or t >= 20:            # early odd steps: the next call follows the last one directly
            for bz in (ref, multi, host, paged):
                bz.evict(-1)
        torch.cuda.synchronize()
        flat = torch.cat([o_ref[l].reshape(-1) for l in order]).cpu()
        assert torch.equal(torch.cat([o_m[l].reshape(-1) for l in order]).cpu(), flat), f"step {t}"
        assert torch.equal(o_h, flat), f"host entry, pinned buffers, step {t}"
        assert torch.equal(o_p, flat), f"host entry, pageable buffers, step {t}"
    for bz in (multi, host, paged):
        for l in range(w.layers):
            for b in range(w.batch):
                a, c = ref.export_state(l, b, w.kv_heads - 1), bz.export_state(l, b, w.kv_heads - 1)
                assert (a["n"], a["n_old"], a["total_len"]) == (c["n"], c["n_old"], c["total_len"])
                assert torch.equal(a["pos"], c["pos"]) and torch.equal(a["score"], c["score"])
                assert torch.equal(a["k"], c["k"]) and torch.equal(a["v"], c["v"])
        assert bz.status() == 0
    for bz in (ref, multi, host, paged):
        bz.close()


@pytest.mark.gpu
def test_two_small_layers_alternating_without_eviction_calls(cuda_device):
    """Small grids let several launches be resident at once. Alternating two layers call after call,
    with nothing between the calls, must give what fully serialised calls give."""
    w = workloads.scaled(workloads.get("C4"), layers=2, batch=1, q_heads=4, kv_heads=1, prompt_min=100,
                         prompt_max=100, decode_steps=60, window=16, budget=400)
    pre, dec = _stack(w)
    ref, fast = make_buzz(w), make_buzz(w)
    for bz in (ref, fast):
        for l in range(2):
            q, k, v, cu = pre[l]
            bz.prefill(l, q, k, v, cu, 100, torch.empty_like(q))
    o_ref = [[torch.empty_like(dec[l][0][t]) for l in range(2)] for t in range(w.decode_steps)]
    o_fast = [[torch.empty_like(dec[l][0][t]) for l in range(2)] for t in range(w.decode_steps)]
    for t in range(w.decode_steps):
        for l in range(2):
            ref.decode_step(l, dec[l][0][t], dec[l][1][t], dec[l][2][t], o_ref[t][l])
            torch.cuda.synchronize()
    for t in range(w.decode_steps):              # enqueued back to back, no synchronisation
        for l in range(2):
            fast.decode_step(l, dec[l][0][t], dec[l][1][t], dec[l][2][t], o_fast[t][l])
    torch.cuda.synchronize()
    for t in range(w.decode_steps):
        for l in range(2):
            assert torch.equal(o_ref[t][l], o_fast[t][l]), f"step {t} layer {l}"
    for l in range(2):
        a, c = ref.export_state(l, 0, 0), fast.export_state(l, 0, 0)
        assert a["n"] == c["n"] == 160 and torch.equal(a["score"], c["score"])
    ref.close(); fast.close()


@pytest.mark.gpu
def test_decode_layers_rejects_bad_layer_lists(cuda_device):
    from paper_2410_23079_b200 import BuzzError
    w = workloads.scaled(workloads.get("C4"), layers=2, batch=1, q_heads=4, kv_heads=1, prompt_min=64,
                         prompt_max=64, decode_steps=1, window=16, budget=100)
    bz = make_buzz(w)
    qd, kd, vd = workloads.decode_inputs(w, 0, "cuda:0")
    o = torch.empty_like(qd[0])
    for bad in ([0, 0], [0, 2], [-1], [0, 1, 0]):
        n = len(bad)
        with pytest.raises(BuzzError):
            bz.decode_layers(bad, [qd[0]] * n, [kd[0]] * n, [vd[0]] * n, [o] * n)
    with pytest.raises(BuzzError):
        bz.decode_layers_host([1, 1], qd[0].cpu(), o.cpu())
    bz.close()


@pytest.mark.gpu
def test_step_replayed_from_a_cuda_graph(cuda_device):
    """One decode step of a layer stack plus the eviction call, captured once in a CUDA graph and
    replayed with fresh inputs in static buffers, leaves the same outputs and caches as direct calls
    (evictions included: the trigger is a device predicate, so the captured launches need no host
    decision)."""
    w = workloads.scaled(workloads.get("C4"), layers=3, batch=2, q_heads=8, kv_heads=2, prompt_min=150,
                         prompt_max=150, decode_steps=45, window=32, budget=180)
    pre, dec = _stack(w)
    ref, cap = make_buzz(w), make_buzz(w)
    for bz in (ref, cap):
        for l in range(w.layers):
            q, k, v, cu = pre[l]
            bz.prefill(l, q, k, v, cu, 150, torch.empty_like(q))
    L = list(range(w.layers))
    sq = [torch.empty_like(dec[l][0][0]) for l in L]
    sk = [torch.empty_like(dec[l][1][0]) for l in L]
    sv = [torch.empty_like(dec[l][2][0]) for l in L]
    so = [torch.empty_like(dec[l][0][0]) for l in L]

    def load(t):
        for l in L:
            sq[l].copy_(dec[l][0][t]); sk[l].copy_(dec[l][1][t]); sv[l].copy_(dec[l][2][t])

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    load(0)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):        # step 0 is only recorded here, not run
            cap.decode_layers(L, sq, sk, sv, so, stream=side)
            cap.evict(-1, stream=side)
    torch.cuda.synchronize()
    for t in range(w.decode_steps):
        o_ref = [torch.empty_like(so[l]) for l in L]
        ref.decode_layers(L, [dec[l][0][t] for l in L], [dec[l][1][t] for l in L], [dec[l][2][t] for l in L], o_ref)
        ref.evict(-1)
        load(t)
        graph.replay()
        torch.cuda.synchronize()
        for l in L:
            assert torch.equal(so[l], o_ref[l]), f"step {t} layer {l}"
    for l in L:
        for b in range(w.batch):
            a, c = ref.export_state(l, b, 1), cap.export_state(l, b, 1)
            assert (a["n"], a["n_old"], a["total_len"]) == (c["n"], c["n_old"], c["total_len"])
            assert torch.equal(a["pos"], c["pos"]) and torch.equal(a["score"], c["score"]) and torch.equal(a["k"], c["k"])
    assert ref.export_state(0, 0, 0)["n"] < 150 + w.decode_steps      # evictions happened on the way
    assert ref.status() == 0 and cap.status() == 0
    ref.close(); cap.close()


@pytest.mark.gpu
def test_decode_layers_with_uneven_and_empty_layers(cuda_device):
    """Layers prefilled with different batch sizes, and a layer that was never prefilled, in one
    multi-layer call: each layer steps its own sequences, the empty one launches nothing; a full
    cache inside the call is reported and skipped like in a single-layer call."""
    w = workloads.scaled(workloads.get("C4"), layers=3, batch=3, q_heads=8, kv_heads=2, prompt_min=120,
                         prompt_max=120, decode_steps=8, window=16, budget=124)
    pre, dec = _stack(w)
    ref, multi = make_buzz(w), make_buzz(w)
    nb = {0: 3, 1: 0, 2: 2}                                    # sequences per layer (layer 1 stays empty)
    for bz in (ref, multi):
        bz.set_decode_cluster(1)
        for l, b in nb.items():
            if b:
                q, k, v, cu = pre[l]
                bz.prefill(l, q[:b * 120], k[:b * 120], v[:b * 120], cu[:b + 1], 120, torch.empty_like(q[:b * 120]))
    for t in range(w.decode_steps):
        o_ref = {l: torch.zeros_like(dec[l][0][t]) for l in nb}
        o_m = {l: torch.zeros_like(dec[l][0][t]) for l in nb}
        for l, b in nb.items():
            if b:
                ref.decode_step(l, dec[l][0][t][:b], dec[l][1][t][:b], dec[l][2][t][:b], o_ref[l][:b])
        L = [2, 1, 0]
        multi.decode_layers(L, [dec[l][0][t][:max(nb[l], 1)] for l in L], [dec[l][1][t][:max(nb[l], 1)] for l in L],
                            [dec[l][2][t][:max(nb[l], 1)] for l in L], [o_m[l][:max(nb[l], 1)] for l in L])
        torch.cuda.synchronize()
        for l in nb:
            assert torch.equal(o_ref[l], o_m[l]), f"step {t} layer {l}"
    # 120 + 8 steps against a budget of 124 and no eviction call: the last steps found the caches full
    assert ref.status() == -2 and multi.status() == -2          # BUZZ_ERR_OVERFLOW
    for l, b in nb.items():
        for s in range(b):
            a, c = ref.export_state(l, s, 0), multi.export_state(l, s, 0)
            assert a["n"] == c["n"] == 124 and torch.equal(a["score"], c["score"]) and torch.equal(a["k"], c["k"])
    ref.close(); multi.close()
