"""Pins for the oracle's eviction (Algorithms 1 and 2, Remarks 1-2) and its integer schedule."""
import json
import math
import os

import numpy as np
import pytest

from oracle.buzz_oracle import BO_NO_PROGRESS, OracleHead

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load_state(h, pos, score, n_old):
    pos = np.asarray(pos, dtype=np.int32)
    n = len(pos)
    K = np.repeat(pos[:, None].astype(np.float64), h.d, axis=1)         # row content = its position
    V = -K
    h.set_state(n_old, int(pos[-1]) + 1, pos, np.asarray(score, dtype=np.float64), K, V)


def test_handworked_case():
    with open(os.path.join(GOLD, "handworked_evict.json")) as f:
        gold = json.load(f)
    h = OracleHead(1, 2, **gold["params"])
    a = gold["first"]
    _load_state(h, a["pos"], a["score"], a["n_old"])
    assert h.evict() == 1
    pos, score, K, V = h.state()
    assert pos.tolist() == a["expect_pos"]
    assert h.counts()[:2] == (len(a["expect_pos"]), a["expect_n_old"])
    assert K[:, 0].tolist() == a["expect_pos"] and V[:, 0].tolist() == [-p for p in a["expect_pos"]]
    keep = [a["pos"].index(p) for p in a["expect_pos"]]
    assert score.tolist() == [a["score"][i] for i in keep]
    assert h.evict() == 0                       # below budget: the trigger must not fire
    b = gold["second"]
    pos2 = a["expect_pos"] + b["append_pos"]
    _load_state(h, pos2, b["score"], a["expect_n_old"])
    assert h.evict() == 1
    assert h.state(with_kv=False)[0].tolist() == b["expect_pos"]
    assert h.counts()[:2] == (len(b["expect_pos"]), b["expect_n_old"])


def _evict_full_cache(h, sink, window, budget, n_old, rng):
    """Plants a full cache (n = budget, of which n_old slots are old, random scores) and runs ONE
    eviction of the oracle; returns the retained original slot indices."""
    pos = np.arange(budget, dtype=np.int32)
    K = pos[:, None].astype(np.float64)
    h.set_state(n_old, budget, pos, rng.random(budget), K, -K)
    assert h.evict() == 1
    return h.state(with_kv=False)[0].tolist()


def test_paper_printed_values():
    """The two numbers the paper prints for stride 5, observed on the oracle's behaviour: s_hat = 3
    (which old slots survive one eviction) and the optimum T/w = 4.33 (the ratio of the middle
    region's capacity to the steady-state number of old tokens, which the theorem equates with w)."""
    with open(os.path.join(GOLD, "paper_values.json")) as f:
        gold = json.load(f)
    s = gold["t_over_w_s5"]["s"]
    assert s == gold["s_hat_formula"]["s"]
    s_hat = gold["s_hat_formula"]["s_hat"]
    rng = np.random.default_rng(0)
    sink, window, T = 2, 7, 26000
    budget = sink + window + T
    h = OracleHead(1, 1, sink, window, s, 1, budget)
    kept = _evict_full_cache(h, sink, window, budget, 100, rng)
    old_kept = [p - sink for p in kept if sink <= p < sink + 100]
    assert old_kept == list(range(0, 100, s_hat))                  # every s_hat-th old slot, from offset 0
    a = h.counts()[1]
    for _ in range(60):                                            # iterate eviction on a full cache to steady state
        _evict_full_cache(h, sink, window, budget, a, rng)
        a = h.counts()[1]
    assert abs(T / a - gold["t_over_w_s5"]["value"]) <= gold["t_over_w_s5"]["abs_tol"]


def _run_schedule(sink, window, s, hitters, budget, evictions, seed=0):
    """Drive the oracle with random scores only (d = 1) and return the n_old after each eviction."""
    rng = np.random.default_rng(seed)
    h = OracleHead(1, 1, sink, window, s, hitters, budget)
    n0 = sink + window
    h.set_state(0, n0, np.arange(n0), rng.random(n0), np.zeros((n0, 1)), np.zeros((n0, 1)))
    seq = []
    while len(seq) < evictions:
        h.decode(np.zeros((1, 1)), np.zeros(1), np.zeros(1))
        n, n_old, tot = h.counts()
        h.set_scores(rng.random(n))
        r = h.evict()
        assert r in (0, 1)
        if r:
            seq.append(h.counts()[1])
            assert h.counts()[0] == sink + seq[-1] + window < budget
    return seq


@pytest.mark.parametrize("s", [3, 4, 5, 8, 16])
def test_count_recursion_and_steady_state(s):
    """n_old follows a_n = ceil(a_{n-1}/s_hat) + ceil((T - a_{n-1})/s) (the appendix recursion with
    this oracle's rounding), independent of the scores; its limit obeys the theorem's fixed point
    T (s+1)/(s^2+1) for odd s and T/(s-1) for even s within the proof's slack."""
    sink, window, T = 4, 32, 600
    budget = sink + window + T
    s_hat = (s + 1) // 2
    seq = _run_schedule(sink, window, s, 1, budget, 60, seed=s)
    a = math.ceil(T / s)
    assert seq[0] == a
    for got in seq[1:]:
        a = math.ceil(a / s_hat) + math.ceil((T - a) / s)
        assert got == a
    assert seq == _run_schedule(sink, window, s, 1, budget, 60, seed=s + 100)   # score-independent
    fixed = T * (s + 1) / (s * s + 1) if s % 2 else T / (s - 1)
    assert abs(seq[-1] - fixed) <= 3.0


@pytest.mark.parametrize("s,hitters", [(3, 1), (4, 1), (5, 1), (5, 2), (8, 1), (16, 2), (31, 3)])
def test_count_recursion_over_1000_evictions(s, hitters):
    """1000 consecutive evictions of a refilled cache: after every one, n_old equals the integer
    recursion a' = ceil(a/s_hat) + kept((T - a), s, h) with kept(m) = (ceil(m/s) - 1) h + min(h, last
    segment), whatever the scores; for one hitter per segment the sequence settles within the proof's
    slack of the theorem's fixed point (Appendix C.1)."""
    sink, window, T = 3, 20, 997
    budget = sink + window + T
    s_hat = (s + 1) // 2
    rng = np.random.default_rng(s * 7 + hitters)
    h = OracleHead(1, 1, sink, window, s, hitters, budget)
    a = 0
    for it in range(1000):
        _evict_full_cache(h, sink, window, budget, a, rng)
        m = T - a
        nseg = math.ceil(m / s)
        kept_new = 0 if nseg == 0 else (nseg - 1) * hitters + min(hitters, m - (nseg - 1) * s)
        a = math.ceil(a / s_hat) + kept_new
        n, n_old, _ = h.counts()
        assert n_old == a and n == sink + a + window < budget, f"eviction {it}"
    if hitters == 1:
        fixed = T * (s + 1) / (s * s + 1) if s % 2 else T / (s - 1)
        assert abs(a - fixed) <= 3.0


def test_first_eviction_shrinks_middle_by_s_minus_1_over_s():
    sink, window, s, T = 4, 16, 8, 800
    seq = _run_schedule(sink, window, s, 1, sink + window + T, 1)
    assert seq[0] == T // s                       # kept 1/s => removed (s-1)/s of the middle


def test_remark1_short_sequences_keep_everything():
    h = OracleHead(1, 1, 4, 8, 4, 1, 16)
    n = 12                                        # = sink + window exactly
    h.set_state(0, n, np.arange(n), np.arange(n, dtype=float), np.zeros((n, 1)), np.zeros((n, 1)))
    assert h.evict() == 0 and h.counts()[0] == n


def test_remark2_prefill_samples_until_it_fits():
    """N = 2000, budget 100: round 1 local-max (stride 8), later rounds interval (stride 4)."""
    sink, window, s, budget, N, d = 4, 32, 8, 100, 2000, 2
    rng = np.random.default_rng(5)
    Q, K, V = rng.standard_normal((1, N, d)), rng.standard_normal((N, d)), rng.standard_normal((N, d))
    h = OracleHead(1, d, sink, window, s, 1, budget)
    _, full, rounds = h.prefill(Q, K, V)
    mid = N - sink - window
    counts = [math.ceil(mid / s)]
    while sink + counts[-1] + window >= budget:
        counts.append(math.ceil(counts[-1] / 4))
    assert rounds == len(counts) and h.counts() == (sink + counts[-1] + window, counts[-1], N)
    pos, sc = h.state(with_kv=False)
    # survivors of round 1 = per-segment argmax; survivors overall = every 4^(rounds-1)-th of them
    winners = [sink + c * s + int(np.argmax(full[sink + c * s: min(sink + (c + 1) * s, N - window)]))
               for c in range(counts[0])]
    expect = list(range(sink)) + winners[:: 4 ** (rounds - 1)] + list(range(N - window, N))
    assert pos.tolist() == expect
    np.testing.assert_array_equal(sc, full[expect])


def _segment_winners_reference(score, lo, hi, s, hmax):
    out = []
    for a in range(lo, hi, s):
        idx = list(range(a, min(a + s, hi)))
        order = sorted(idx, key=lambda j: (-score[j], j))
        out += sorted(order[: min(hmax, len(idx))])
    return out


@pytest.mark.parametrize("seed", range(12))
def test_random_evictions_against_independent_selection_and_invariants(seed):
    rng = np.random.default_rng(seed)
    sink = int(rng.integers(0, 5)); window = int(rng.integers(1, 20)); s = int(rng.integers(3, 12))
    hit = int(rng.integers(1, min(s, 4))); budget = sink + window + s + int(rng.integers(0, 120))
    d = 2
    h = OracleHead(1, d, sink, window, s, hit, budget)
    rows = {}
    def row(p):
        rows.setdefault(p, rng.standard_normal(2 * d))
        return rows[p][:d], rows[p][d:]
    n0 = 1
    k0, v0 = row(0)
    h.prefill(rng.standard_normal((1, 1, d)), k0[None], v0[None])
    quant = rng.random() < 0.5                        # force exact score ties half of the time
    for t in range(1, 400):
        k, v = row(t)
        h.decode(rng.standard_normal((1, d)), k, v)
        n, n_old, tot = h.counts()
        assert tot == t + 1 and n <= budget                                   # I1
        pos, sc = h.state(with_kv=False)
        if quant:
            sc = np.round(sc * 4) / 4
            h.set_scores(sc)
        r = h.evict()
        if n < budget:
            assert r == 0
            continue
        assert r == 1
        s_hat = (s + 1) // 2
        old_keep = list(range(sink, sink + n_old, s_hat))
        new_keep = _segment_winners_reference(sc, sink + n_old, n - window, s, hit)
        expect_idx = list(range(sink)) + old_keep + new_keep + list(range(n - window, n))
        pos2, sc2, K2, V2 = h.state()
        assert pos2.tolist() == pos[expect_idx].tolist()
        np.testing.assert_array_equal(sc2, sc[expect_idx])
        n2, n_old2, _ = h.counts()
        assert n2 < budget and n_old2 == len(old_keep) + len(new_keep)        # I1, count rule
        assert np.all(np.diff(pos2) > 0)                                      # I4
        assert pos2[:sink].tolist() == list(range(sink))                      # I2 sink
        assert pos2[-window:].tolist() == list(range(t + 1 - window, t + 1))  # I2 window
        for i, p in enumerate(pos2):                                          # I5 rows travel intact
            kk, vv = row(int(p))
            assert np.array_equal(K2[i], kk) and np.array_equal(V2[i], vv)


def test_no_progress_is_reported_not_looped():
    """s = 2 gives s_hat = 1: old tokens never thin, so a cache full of old tokens cannot shrink."""
    sink, window, budget = 1, 2, 8
    h = OracleHead(1, 1, sink, window, 2, 1, budget)
    n = budget
    h.set_state(n - sink - window, n, np.arange(n), np.zeros(n), np.zeros((n, 1)), np.zeros((n, 1)))
    assert h.evict() == BO_NO_PROGRESS


def test_overflow_is_an_error():
    h = OracleHead(1, 1, 1, 2, 3, 1, 6)
    n = 6
    h.set_state(0, n, np.arange(n), np.zeros(n), np.zeros((n, 1)), np.zeros((n, 1)))
    with pytest.raises(RuntimeError):
        h.decode(np.zeros((1, 1)), np.zeros(1), np.zeros(1))


def test_parameter_validation():
    for bad in [dict(segment=1), dict(hitters=0), dict(hitters=4), dict(window=0), dict(budget=10)]:
        p = dict(sink=4, window=8, segment=4, hitters=1, budget=32)
        p.update(bad)
        with pytest.raises(ValueError):
            OracleHead(1, 4, **p)


def _interval_reference(lo, hi, s, hmax):
    out = []
    for a in range(lo, hi, s):
        out += list(range(a, min(a + min(hmax, s), hi)))
    return out


@pytest.mark.parametrize("interval_new,new_stride,old_stride", [(False, 3, 5), (True, 6, 3), (True, 4, 1), (False, 7, 2)])
def test_sampling_variants_of_the_ablation_study(interval_new, new_stride, old_stride):
    """Section 4.3: swapped / free strides and interval sampling for new tokens, against a selection
    written independently here; counts follow a_n = ceil(a/s_old) + kept(T - a) whatever the scores."""
    rng = np.random.default_rng(new_stride * 10 + old_stride)
    sink, window, hit, T = 3, 11, 2 if new_stride > 2 else 1, 90
    budget = sink + window + T
    h = OracleHead(1, 1, sink, window, 16, hit, budget)
    h.set_sampling(interval_new, new_stride, old_stride)
    n0 = sink + window
    h.set_state(0, n0, np.arange(n0), rng.random(n0), np.zeros((n0, 1)), np.zeros((n0, 1)))
    evictions = 0
    for t in range(n0, n0 + 600):
        h.decode(np.zeros((1, 1)), np.zeros(1), np.zeros(1))
        n, n_old, _ = h.counts()
        sc = np.round(rng.random(n) * 5) / 5
        h.set_scores(sc)
        pos, _ = h.state(with_kv=False)
        r = h.evict()
        if n < budget:
            assert r == 0
            continue
        old_keep = list(range(sink, sink + n_old, old_stride))
        lo, hi = sink + n_old, n - window
        new_keep = _interval_reference(lo, hi, new_stride, hit) if interval_new else \
            _segment_winners_reference(sc, lo, hi, new_stride, hit)
        expect = list(range(sink)) + old_keep + new_keep + list(range(n - window, n))
        if len(expect) >= n:                      # nothing can be dropped (old stride 1): reported, not looped
            assert r == BO_NO_PROGRESS
            break
        assert r == 1
        evictions += 1
        assert h.state(with_kv=False)[0].tolist() == pos[expect].tolist()
        assert h.counts()[1] == len(old_keep) + len(new_keep)
    assert evictions >= 3 or old_stride == 1


def test_sampling_variant_validation():
    h = OracleHead(1, 1, 2, 4, 8, 3, 40)
    for bad in [(False, 1, 2), (False, 3, 2), (False, 8, 0), (False, 40, 2)]:
        with pytest.raises(ValueError):
            h.set_sampling(*bad)


# ---- global top-k policy (the heavy-hitter baseline, Sections 3.2 and 4.3) ----------------------

def test_topk_policy_handworked_case():
    with open(os.path.join(GOLD, "handworked_topk.json")) as f:
        gold = json.load(f)
    h = OracleHead(1, 2, **gold["params"])
    h.set_policy(True)
    a = gold["first"]
    _load_state(h, a["pos"], a["score"], a["n_old"])
    assert h.evict() == 1
    pos, score, K, V = h.state()
    assert pos.tolist() == a["expect_pos"] and h.counts()[:2] == (len(a["expect_pos"]), a["expect_n_old"])
    assert K[:, 0].tolist() == a["expect_pos"]
    assert score.tolist() == [a["score"][a["pos"].index(p)] for p in a["expect_pos"]]
    b = gold["second"]
    pos2 = a["expect_pos"] + b["append_pos"]
    _load_state(h, pos2, b["score"], a["expect_n_old"])
    assert h.evict() == 1
    assert h.state(with_kv=False)[0].tolist() == b["expect_pos"]
    assert h.counts()[:2] == (len(b["expect_pos"]), b["expect_n_old"])


@pytest.mark.parametrize("seed", range(10))
def test_topk_policy_against_a_sort_and_same_schedule_as_sampling(seed):
    """Random runs with forced ties: the survivors equal a selection written independently here (sort
    the middle slots by (score descending, slot ascending), cut at M, restore slot order), M follows
    the sampling module's count rule, and so the (n, n_old) trajectory is the one the sampling
    policy produces on the same lengths."""
    rng = np.random.default_rng(100 + seed)
    sink = int(rng.integers(0, 5)); window = int(rng.integers(1, 20)); s = int(rng.integers(3, 12))
    hit = int(rng.integers(1, min(s, 4))); budget = sink + window + s + int(rng.integers(0, 120))
    top, ref = OracleHead(1, 1, sink, window, s, hit, budget), OracleHead(1, 1, sink, window, s, hit, budget)
    top.set_policy(True)
    z = np.zeros((1, 1))
    for head in (top, ref):
        head.prefill(z[None], z, z)
    s_hat = (s + 1) // 2
    evictions = 0
    for t in range(1, 500):
        for head in (top, ref):
            head.decode(z, z[0], z[0])
        n, n_old, tot = top.counts()
        assert ref.counts() == (n, n_old, tot)                       # same schedule under both policies
        sc = np.round(rng.random(n) * 6) / 6                         # many exact ties
        top.set_scores(sc); ref.set_scores(sc)
        pos, _ = top.state(with_kv=False)
        r = top.evict()
        assert ref.evict() == r
        if n < budget:
            assert r == 0
            continue
        assert r == 1
        evictions += 1
        lo, hi = sink, n - window
        M = len(range(0, n_old, s_hat)) + sum(min(hit, min(a + s, hi) - a) for a in range(sink + n_old, hi, s))
        chosen = sorted(sorted(range(lo, hi), key=lambda j: (-sc[j], j))[:M])
        expect = list(range(sink)) + chosen + list(range(hi, n))
        pos2, sc2 = top.state(with_kv=False)
        assert pos2.tolist() == pos[expect].tolist()
        np.testing.assert_array_equal(sc2, sc[expect])
        assert top.counts()[1] == M
        assert np.all(np.diff(pos2) > 0) and pos2[-window:].tolist() == list(range(t + 1 - window, t + 1))
        # every survivor's score is >= every evicted middle token's score
        evicted = sorted(set(range(lo, hi)) - set(chosen))
        if evicted and chosen:
            assert min(sc[j] for j in chosen) >= max(sc[j] for j in evicted)
    assert evictions >= 3


def test_topk_policy_at_prefill_keeps_the_overall_heaviest():
    """Remark 2's repeated rounds under the top-k policy: top-k sets are nested, so after any number
    of rounds the middle survivors are the M_final heaviest prompt tokens between sink and window."""
    sink, window, s, budget, N, d = 4, 32, 8, 100, 1500, 2
    rng = np.random.default_rng(9)
    Q, K, V = rng.standard_normal((1, N, d)), rng.standard_normal((N, d)), rng.standard_normal((N, d))
    h = OracleHead(1, d, sink, window, s, 1, budget)
    h.set_policy(True)
    _, full, rounds = h.prefill(Q, K, V)
    assert rounds >= 2
    M = h.counts()[1]
    mid = range(sink, N - window)
    chosen = sorted(sorted(mid, key=lambda j: (-full[j], j))[:M])
    assert h.state(with_kv=False)[0].tolist() == list(range(sink)) + chosen + list(range(N - window, N))
