"""Lock-step comparison of libbuzz (CUDA) against the CPU oracle on one workload.

Both sides receive the same seeded inputs (the GPU tensors' bytes, copied to the host). For every
sampled (layer, sequence, KV head) instance:
  * prefill outputs and pre-eviction prompt scores are compared within tolerance;
  * selection parity is lock-step: the GPU's fp32 scores are loaded into a second oracle instance,
    which then takes every arg-max decision on exactly the values the GPU holds; retained
    positions, counters, scores and K/V rows must then match bit for bit;
  * every decode step's output is compared within tolerance, the running scores to rel 1e-3, and
    before each eviction the oracle's scores are replaced by the GPU's (lock-step again);
  * where the oracle ran the whole prefill, a third, FREE-RUNNING oracle instance never sees the
    GPU's scores: at every eviction its retained positions are compared with the GPU's, and every
    difference must be a near-tie (the two candidates' scores, in the oracle's own fp64, within rel
    1e-3 of each other, inside one segment); after a difference it is re-aligned with the lock-step
    instance, because the trajectories legitimately part from there.
"""
from __future__ import annotations

import numpy as np
import torch

import workloads
from oracle.buzz_oracle import OracleHead
from paper_2410_23079_b200 import Buzz

TOL = {"bf16": dict(atol=2e-2, rtol=1e-2), "f32": dict(atol=1e-4, rtol=1e-4)}
SCORE_RTOL = 1e-3


def make_buzz(w: workloads.Workload, device="cuda:0", max_prompt_tokens=None, logn=False) -> Buzz:
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    lens = workloads.prompt_lengths(w)
    return Buzz(sink=w.sink, window=w.window, segment=w.segment, hitters=w.hitters, budget=w.budget,
                layers=w.layers, max_batch=w.batch, q_heads=w.q_heads, kv_heads=w.kv_heads,
                head_dim=w.head_dim, dtype=dt, max_prompt_tokens=max_prompt_tokens or sum(lens),
                logn=logn, device=device)


def _np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def assert_close(got, ref, atol, rtol, what):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    bad = err > atol + rtol * np.abs(ref)
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} off, max abs err {err.max():.3e}"


def assert_scores_close(got, ref, what):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    rel = np.abs(got - ref) / np.maximum(np.abs(ref), 1e-30)
    assert rel.max(initial=0.0) <= SCORE_RTOL, f"{what}: max rel err {rel.max():.3e}"


def compare_state(bz: Buzz, orc: OracleHead, layer, seq, head, what, exact_scores):
    st = bz.export_state(layer, seq, head)
    n, n_old, tot = orc.counts()
    assert (st["n"], st["n_old"], st["total_len"]) == (n, n_old, tot), f"{what}: counters {st['n'], st['n_old'], st['total_len']} vs {(n, n_old, tot)}"
    pos, score, K, V = orc.state()
    assert np.array_equal(st["pos"].numpy(), pos), f"{what}: retained positions differ"
    assert np.array_equal(_np64(st["k"]), K) and np.array_equal(_np64(st["v"]), V), f"{what}: K/V rows differ"
    if exact_scores:
        assert np.array_equal(st["score"].numpy().astype(np.float64), score), f"{what}: scores differ"
    else:
        assert_scores_close(st["score"].numpy(), score, what + " scores")
    return st


def check_free_running(fr: OracleHead, before, gpu_pos, w, what, stats):
    """`before` = (pos, score) of the free-running oracle just before its eviction, `gpu_pos` the
    positions the GPU retained. Counts are score-independent, so the two retained sets have the same
    size; positions only one side kept are paired in order and each pair must be a near-tie."""
    pos_b, sc_b = before
    score_of = dict(zip(pos_b.tolist(), sc_b.tolist()))
    slot_of = {p: i for i, p in enumerate(pos_b.tolist())}
    mine = fr.state(with_kv=False)[0].tolist()
    only_f = sorted(set(mine) - set(gpu_pos))
    only_g = sorted(set(gpu_pos) - set(mine))
    assert len(only_f) == len(only_g), f"{what}: free-running oracle and GPU kept different counts"
    for pf, pg in zip(only_f, only_g):
        a, b = score_of[pf], score_of[pg]
        assert abs(a - b) <= SCORE_RTOL * max(abs(a), abs(b)), \
            f"{what}: GPU kept position {pg} (score {b}) where the oracle kept {pf} (score {a}): not a near-tie"
        if not getattr(fr, "global_topk", False):           # the sampling module decides inside one segment
            assert abs(slot_of[pf] - slot_of[pg]) < fr.segment, f"{what}: positions {pf}, {pg} are not in one segment"
    stats["free_running_evictions"] += 1
    stats["free_running_near_ties"] += len(only_f)
    return len(only_f) == 0


def check_prefill_sampled(w, Q, K, V, got, gpu_scores, rows, tail_keys, tol, logn, what, stats):
    """Full-size prefill check without the O(N^2) oracle prefill. Row i of causal attention is one
    decode step of the oracle over the prefix [0, i) (Eq. 3 for one query), so sampled output rows
    are checked one by one; the column sums of the last `tail_keys` keys only involve the last
    `tail_keys` rows, which the oracle replays in order, accumulating their probabilities."""
    g, N, d = Q.shape
    huge = 1 << 30
    for i in rows:
        i = int(min(max(i, 0), N - 1))
        o = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, huge, logn=logn)
        o.set_state(0, i, np.arange(i), np.zeros(i), K[:i], V[:i])
        ref = o.decode(Q[:, i], K[i], V[i])
        assert_close(got[:, i], ref, what=f"prefill out row {i} {what}", **tol)
        stats["max_out_err"] = max(stats["max_out_err"], float(np.abs(got[:, i] - ref).max()))
    R = min(tail_keys, N)
    o = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, huge, logn=logn)
    o.set_state(0, N - R, np.arange(N - R), np.zeros(N - R), K[:N - R], V[:N - R])
    for i in range(N - R, N):
        ref = o.decode(Q[:, i], K[i], V[i])
        if i % 16 == 0 or i == N - 1:
            assert_close(got[:, i], ref, what=f"prefill out row {i} {what}", **tol)
    _, sc = o.state(with_kv=False)
    assert_scores_close(gpu_scores[N - R:], sc[N - R:], f"prefill scores of the last {R} keys {what}")
    total = float(np.sum(gpu_scores.astype(np.float64)))
    assert abs(total - g * N) <= 1e-4 * g * N, f"{what}: prompt scores sum to {total}, expected {g * N}"


def run_lockstep(w: workloads.Workload, samples, decode_steps=None, layers=None, check_every=1,
                 device="cuda:0", logn=False, bz: Buzz | None = None, sampled_rows=None, tail_keys=64,
                 sampling=None, layers_call=False, topk=False):
    """Runs prefill + decode/evict on the GPU for the whole workload and the oracle on `samples`
    (a list of (layer, seq, kv_head)). Returns a dict of summary counters."""
    tol = TOL[w.dtype]
    S = w.decode_steps if decode_steps is None else decode_steps
    layers = list(range(w.layers)) if layers is None else layers
    own = bz is None
    bz = bz or make_buzz(w, device, logn=logn)
    if sampling is not None:                     # (interval_new, new_stride, old_stride): Section 4.3 variants
        bz.set_sampling(*sampling)
    if topk:                                     # global top-k policy instead of the sampling module
        bz.set_policy(True)

    def new_oracle(budget=w.budget):
        o = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, budget, logn=logn)
        if sampling is not None:
            o.set_sampling(*sampling)
        if topk:
            o.set_policy(True)
            o.global_topk = True
        return o

    lens = workloads.prompt_lengths(w)
    offs = np.concatenate([[0], np.cumsum(lens)])
    g, d = w.group, w.head_dim
    stats = dict(evictions=0, prefill_rounds=0, max_out_err=0.0, free_running_evictions=0, free_running_near_ties=0)
    lock = {}
    frees = {}
    dec = {}
    for layer in layers:
        q, k, v, cu = workloads.prefill_inputs(w, layer, device)
        out = torch.empty_like(q)
        bz.prefill(layer, q, k, v, cu, max(lens), out)
        assert bz.status() == 0
        dec[layer] = workloads.decode_inputs(w, layer, device, steps=S)
        pscore = {}
        for (ll, b, h) in samples:
            if ll != layer:
                continue
            a, e = int(offs[b]), int(offs[b + 1])
            Q = _np64(q[a:e, h * g:(h + 1) * g]).transpose(1, 0, 2)
            K, V = _np64(k[a:e, h]), _np64(v[a:e, h])
            got = _np64(out[a:e, h * g:(h + 1) * g]).transpose(1, 0, 2)
            if h not in pscore:
                pscore[h] = bz.export_prefill_scores(h, int(offs[-1])).numpy()
            gs = pscore[h][a:e]
            if sampled_rows is None:
                free = new_oracle()
                O, full, rounds = free.prefill(Q, K, V)
                stats["prefill_rounds"] = max(stats["prefill_rounds"], rounds)
                assert_close(got, O, what=f"prefill out L{layer} b{b} h{h}", **tol)
                stats["max_out_err"] = max(stats["max_out_err"], float(np.abs(got - O).max()))
                assert_scores_close(gs, full, f"prefill scores L{layer} b{b} h{h}")
                frees[(layer, b, h)] = free
            else:
                check_prefill_sampled(w, Q, K, V, got, gs, sampled_rows, tail_keys, tol, logn,
                                      f"L{layer} b{b} h{h}", stats)
            # lock-step instance: selection decided on the GPU's fp32 scores
            ls = new_oracle()
            N = e - a
            ls.set_state(0, N, np.arange(N), gs.astype(np.float64), K, V)
            while ls.counts()[0] >= w.budget:
                assert ls.evict() == 1
            st0 = compare_state(bz, ls, layer, b, h, f"after prefill L{layer} b{b} h{h}", exact_scores=True)
            lock[(layer, b, h)] = ls
            fr = frees.get((layer, b, h))
            if fr is not None and fr.counts()[0] != e - a:      # the free-running oracle sampled at prefill too
                if rounds == 1:                                 # one round: every difference must be a near-tie
                    same = check_free_running(fr, (np.arange(N), full), st0["pos"].tolist(), w,
                                              f"prefill sampling L{layer} b{b} h{h}", stats)
                else:                                           # later rounds thin by index: one near-tie shifts the rest
                    same = fr.state(with_kv=False)[0].tolist() == st0["pos"].tolist()
                    stats["free_running_evictions"] += 1
                    stats["free_running_near_ties"] += 0 if same else 1
                if not same:
                    fr.set_state(ls.counts()[1], ls.counts()[2], *ls.state())
    for t in range(S):
        outs = {layer: torch.empty_like(dec[layer][0][t]) for layer in layers}
        if layers_call:                          # the whole stack in one multi-layer call
            bz.decode_layers(layers, [dec[l][0][t] for l in layers], [dec[l][1][t] for l in layers],
                             [dec[l][2][t] for l in layers], [outs[l] for l in layers])
        else:
            for layer in layers:
                qd, kd, vd = dec[layer]
                bz.decode_step(layer, qd[t], kd[t], vd[t], outs[layer])
        pre = {}
        for key, ls in lock.items():
            layer, b, h = key
            qd, kd, vd = dec[layer]
            ref = ls.decode(_np64(qd[t, b, h * g:(h + 1) * g]), _np64(kd[t, b, h]), _np64(vd[t, b, h]))
            got = _np64(outs[layer][b, h * g:(h + 1) * g])
            assert_close(got, ref, what=f"decode out step {t} {key}", **tol)
            stats["max_out_err"] = max(stats["max_out_err"], float(np.abs(got - ref).max()))
            will_evict = ls.counts()[0] >= w.budget
            if will_evict or (t % check_every == 0) or t == S - 1:
                st = compare_state(bz, ls, layer, b, h, f"decode step {t} {key}", exact_scores=False)
                if will_evict:
                    ls.set_scores(st["score"].numpy().astype(np.float64))
            pre[key] = will_evict
            fr = frees.get(key)
            if fr is not None:
                ref_f = fr.decode(_np64(qd[t, b, h * g:(h + 1) * g]), _np64(kd[t, b, h]), _np64(vd[t, b, h]))
                assert_close(got, ref_f, what=f"decode out step {t} {key} (free-running oracle)", **tol)
        for layer in layers:
            bz.evict(layer)
        assert bz.status() == 0, f"device status after step {t}"
        for key, ls in lock.items():
            r = ls.evict()
            assert r == (1 if pre[key] else 0)
            if pre[key]:
                stats["evictions"] += 1
                st = compare_state(bz, ls, *key, f"after eviction step {t} {key}", exact_scores=True)
                fr = frees.get(key)
                if fr is not None:
                    before = fr.state(with_kv=False)
                    assert fr.evict() == 1
                    if not check_free_running(fr, before, st["pos"].tolist(), w, f"eviction step {t} {key}", stats):
                        fr.set_state(ls.counts()[1], ls.counts()[2], *ls.state())
    if own:
        bz.close()
    return stats
