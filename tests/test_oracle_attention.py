"""Pins for the oracle's attention and score arithmetic (Eqs. 1-3; Algorithm 2's input A).

Each check binds the oracle to something other than itself: a library softmax in fp64, closed
forms for equal keys, conservation laws, and a pure-Python brute force on tiny inputs.
"""
import math

import numpy as np
import pytest
import torch

from oracle.buzz_oracle import OracleHead

BIG = 10 ** 6  # a budget that is never reached: the path must then be textbook attention


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _torch_causal(Q, K, V):
    """Causal softmax attention with torch's own softmax/matmul in fp64 (a library routine)."""
    Qt, Kt, Vt = (torch.from_numpy(x) for x in (Q, K, V))
    N, d = K.shape
    S = torch.einsum("gid,jd->gij", Qt, Kt) / math.sqrt(d)
    mask = torch.ones(N, N, dtype=torch.bool).tril()
    P = torch.softmax(S.masked_fill(~mask, float("-inf")), dim=-1)
    return torch.einsum("gij,jd->gid", P, Vt).numpy(), P.sum(dim=(0, 1)).numpy()


@pytest.mark.parametrize("g,N,d", [(1, 37, 8), (4, 50, 16), (2, 129, 64)])
def test_prefill_equals_textbook_attention(g, N, d):
    Q, K, V = _rand((g, N, d), 1), _rand((N, d), 2), _rand((N, d), 3)
    h = OracleHead(g, d, 2, 4, 4, 1, BIG)
    O, score, rounds = h.prefill(Q, K, V)
    O_ref, col_ref = _torch_causal(Q, K, V)
    assert rounds == 0
    np.testing.assert_allclose(O, O_ref, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(score, col_ref, rtol=1e-11, atol=1e-13)
    assert h.counts() == (N, 0, N)
    pos, sc, Kc, Vc = h.state()
    assert np.array_equal(pos, np.arange(N)) and np.array_equal(Kc, K) and np.array_equal(Vc, V)


def test_decode_without_eviction_is_full_attention():
    g, N, d, steps = 3, 20, 16, 12
    Q, K, V = _rand((g, N + steps, d), 4), _rand((N + steps, d), 5), _rand((N + steps, d), 6)
    h = OracleHead(g, d, 2, 4, 4, 1, BIG)
    h.prefill(Q[:, :N], K[:N], V[:N])
    O_ref, col_ref = _torch_causal(Q, K, V)
    for t in range(steps):
        o = h.decode(Q[:, N + t], K[N + t], V[N + t])
        assert h.evict() == 0
        np.testing.assert_allclose(o, O_ref[:, N + t], rtol=1e-11, atol=1e-12)
    # accumulated scores after prefill + decode == column sums of the full causal matrix
    _, sc = h.state(with_kv=False)
    np.testing.assert_allclose(sc, col_ref, rtol=1e-11, atol=1e-13)


def test_equal_keys_closed_forms():
    """All keys equal => P_ij = 1/(i+1), O_i = mean(V_0..V_i), score_j = g (H_N - H_j)."""
    g, N, d = 2, 40, 8
    Q, V = _rand((g, N, d), 7), _rand((N, d), 8)
    K = np.tile(_rand((1, d), 9), (N, 1))
    h = OracleHead(g, d, 1, 2, 3, 1, BIG)
    O, score, _ = h.prefill(Q, K, V)
    means = np.cumsum(V, axis=0) / np.arange(1, N + 1)[:, None]
    for q in range(g):
        np.testing.assert_allclose(O[q], means, rtol=1e-12, atol=1e-13)
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, N + 1))])
    np.testing.assert_allclose(score, g * (H[N] - H[:N]), rtol=1e-12)


def test_probability_mass_is_conserved():
    """Every softmax row sums to 1: sum(score) = g N after prefill and grows by g per decode step;
    with V = all ones every output equals 1."""
    g, N, d = 4, 33, 16
    Q, K = _rand((g, N, d), 10), _rand((N, d), 11)
    V = np.ones((N, d))
    h = OracleHead(g, d, 2, 4, 4, 1, BIG)
    O, score, _ = h.prefill(Q, K, V)
    assert abs(score.sum() - g * N) < 1e-10
    np.testing.assert_allclose(O, 1.0, rtol=0, atol=1e-12)
    for t in range(5):
        o = h.decode(_rand((g, d), 20 + t), _rand((d,), 30 + t), np.ones(d))
        np.testing.assert_allclose(o, 1.0, rtol=0, atol=1e-12)
        _, sc = h.state(with_kv=False)
        assert abs(sc.sum() - g * (N + t + 1)) < 1e-10


def test_single_key_gets_probability_one():
    d = 8
    h = OracleHead(1, d, 1, 2, 3, 1, BIG)
    k0, v0 = _rand((1, d), 1), _rand((1, d), 2)
    O, score, _ = h.prefill(_rand((1, 1, d), 3), k0, v0)
    np.testing.assert_allclose(O[0, 0], v0[0], rtol=1e-14)
    assert score[0] == 1.0


def test_scale_is_one_over_sqrt_d():
    """Two keys, hand-computed logistic: p_1 = sigmoid((q.k1 - q.k0)/sqrt(d))."""
    d = 4
    q = np.array([[1.0, 2.0, -1.0, 0.5]])
    K = np.array([[0.5, 0.0, 1.0, 1.0], [1.0, 1.0, 0.0, -2.0]])
    V = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]])
    h = OracleHead(1, d, 1, 2, 3, 1, BIG)
    h.prefill(np.zeros((1, 1, d)), K[:1], V[:1])
    o = h.decode(q, K[1], V[1])
    l0, l1 = q[0] @ K[0] / 2.0, q[0] @ K[1] / 2.0
    p1 = 1.0 / (1.0 + math.exp(l0 - l1))
    np.testing.assert_allclose(o[0], [1 - p1, p1, 0, 0], rtol=1e-13, atol=1e-15)
    _, sc = h.state(with_kv=False)
    np.testing.assert_allclose(sc, [1.0 + (1 - p1), p1], rtol=1e-13)


def _bruteforce_probs(Q, K):
    """Pure-Python causal probabilities P[q][i][j], no numpy in the arithmetic."""
    g, N, d = Q.shape
    out = []
    for q in range(g):
        rows = []
        for i in range(N):
            logits = [sum(float(Q[q, i, c]) * float(K[j, c]) for c in range(d)) / math.sqrt(d)
                      for j in range(i + 1)]
            mx = max(logits)
            e = [math.exp(x - mx) for x in logits]
            tot = sum(e)
            rows.append([x / tot for x in e] + [0.0] * (N - i - 1))
        out.append(rows)
    return out


def test_bruteforce_prefill_then_segment_argmax():
    """Tiny case end to end: full attention by hand, then an explicit per-segment argmax written
    separately from the oracle (Algorithm 2), then sink | winners | window."""
    g, N, d = 2, 30, 4
    sink, window, seg, budget = 2, 5, 4, 20
    Q, K, V = _rand((g, N, d), 41), _rand((N, d), 42), _rand((N, d), 43)
    P = _bruteforce_probs(Q, K)
    col = [sum(P[q][i][j] for q in range(g) for i in range(N)) for j in range(N)]
    keep = list(range(sink))
    lo, hi = sink, N - window
    idx = lo
    while idx < hi:
        cand = list(range(idx, min(idx + seg, hi)))
        best = cand[0]
        for j in cand[1:]:
            if col[j] > col[best]:
                best = j
        keep.append(best)
        idx += seg
    keep += list(range(N - window, N))
    h = OracleHead(g, d, sink, window, seg, 1, budget)
    O, score, rounds = h.prefill(Q, K, V)
    assert rounds == 1
    np.testing.assert_allclose(score, col, rtol=1e-12)
    pos, sc, Kc, Vc = h.state()
    assert pos.tolist() == keep
    np.testing.assert_array_equal(Kc, K[keep])
    np.testing.assert_array_equal(Vc, V[keep])
    np.testing.assert_allclose(sc, np.array(col)[keep], rtol=1e-12)
    for q in range(g):
        for i in (0, 7, N - 1):
            ref = sum(P[q][i][j] * V[j] for j in range(N))
            np.testing.assert_allclose(O[q, i], ref, rtol=1e-11, atol=1e-13)


# ---- log-n scaled attention (Section 3.5): Softmax((log_512 n / sqrt(d)) Q K^T) V --------------
# Each pin below fails for one plausible misreading: a natural or base-2 logarithm instead of base
# 512, n counted from zero, or n taken as the number of retained slots instead of tokens seen.

def test_logn_scale_is_exactly_one_at_512_tokens():
    """log_512(512) = 1: the 512th token's row (prefill) and a decode step that brings the number of
    tokens seen to 512 must equal plain attention bit for bit; their neighbours must not."""
    g, d, N = 2, 8, 514
    Q, K, V = _rand((g, N, d), 51), _rand((N, d), 52), _rand((N, d), 53)
    plain, logn = OracleHead(g, d, 2, 4, 4, 1, BIG), OracleHead(g, d, 2, 4, 4, 1, BIG, logn=True)
    Op, _, _ = plain.prefill(Q, K, V)
    Ol, _, _ = logn.prefill(Q, K, V)
    assert np.array_equal(Ol[:, 511], Op[:, 511])              # row index 511 has seen 512 tokens
    assert not np.array_equal(Ol[:, 510], Op[:, 510]) and not np.array_equal(Ol[:, 512], Op[:, 512])
    # decode: 511 tokens seen, 5 retained; the appended token is the 512th
    keep = [0, 100, 200, 300, 510]
    for head in (plain, logn):
        head.set_state(2, 511, np.array(keep), np.zeros(5), K[keep], V[keep])
    q, k, v = _rand((g, d), 54), _rand((d,), 55), _rand((d,), 56)
    assert np.array_equal(logn.decode(q, k, v), plain.decode(q, k, v))
    assert not np.array_equal(logn.decode(q, k, v), plain.decode(q, k, v))   # 513 tokens seen now


def test_logn_two_keys_by_hand():
    """Second token of a sequence: n = 2, log_512 2 = 1/9, so p_1 = sigmoid((q.k1 - q.k0)/(9 sqrt(d)))."""
    d = 4
    q = np.array([[1.0, 2.0, -1.0, 0.5]])
    K = np.array([[0.5, 0.0, 1.0, 1.0], [1.0, 1.0, 0.0, -2.0]])
    V = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]])
    h = OracleHead(1, d, 1, 2, 3, 1, BIG, logn=True)
    O, _, _ = h.prefill(np.ones((1, 1, d)), K[:1], V[:1])
    np.testing.assert_array_equal(O[0, 0], V[0])               # n = 1: scale 0, the only key gets p = 1
    o = h.decode(q, K[1], V[1])
    l0, l1 = q[0] @ K[0] / (9.0 * 2.0), q[0] @ K[1] / (9.0 * 2.0)
    p1 = 1.0 / (1.0 + math.exp(l0 - l1))
    np.testing.assert_allclose(o[0], [1 - p1, p1, 0, 0], rtol=1e-13, atol=1e-15)
    # the same pair as the first two rows of a prefill
    h2 = OracleHead(1, d, 1, 2, 3, 1, BIG, logn=True)
    O2, sc2, _ = h2.prefill(np.stack([np.ones((1, d)), q], axis=1), K, V)
    np.testing.assert_allclose(O2[0, 1], [1 - p1, p1, 0, 0], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(sc2, [1.0 + (1 - p1), p1], rtol=1e-13)


def test_logn_counts_tokens_seen_not_retained_slots():
    """After evictions the cache holds fewer slots than tokens were seen. With 3 retained slots and 63
    tokens seen, the next step has n = 64 = 512^(2/3): the scale is (2/3)/sqrt(d), not log_512(4)."""
    d = 16
    K, V = _rand((3, d), 61), _rand((3, d), 62)
    q, k, v = _rand((1, d), 63), _rand((d,), 64), _rand((d,), 65)
    h = OracleHead(1, d, 1, 2, 3, 1, BIG, logn=True)
    h.set_state(0, 63, np.array([0, 40, 62]), np.zeros(3), K, V)
    o = h.decode(q, k, v)
    Kall, Vall = np.vstack([K, k]), np.vstack([V, v])

    def attend(scale):
        z = torch.from_numpy(Kall @ q[0] * scale)
        return (torch.softmax(z, dim=0).numpy()[:, None] * Vall).sum(axis=0)

    np.testing.assert_allclose(o[0], attend((2.0 / 3.0) / 4.0), rtol=1e-12, atol=1e-14)
    assert np.abs(o[0] - attend(math.log(4, 512) / 4.0)).max() > 1e-3     # the retained-count reading
    assert np.abs(o[0] - attend(math.log(64) / 4.0)).max() > 1e-3         # a natural logarithm


@pytest.mark.parametrize("g,N,d", [(1, 33, 8), (3, 70, 16)])
def test_logn_prefill_against_library_softmax(g, N, d):
    """Row i (0-based) is scaled by log2(i+1)/9/sqrt(d) -- written with the base-2 identity
    log_512 n = log2(n)/9 rather than the oracle's quotient of natural logarithms."""
    Q, K, V = _rand((g, N, d), 71), _rand((N, d), 72), _rand((N, d), 73)
    h = OracleHead(g, d, 2, 4, 4, 1, BIG, logn=True)
    O, score, _ = h.prefill(Q, K, V)
    Qt, Kt, Vt = (torch.from_numpy(x) for x in (Q, K, V))
    scale = torch.log2(torch.arange(1, N + 1, dtype=torch.float64)) / 9.0 / math.sqrt(d)
    S = torch.einsum("gid,jd->gij", Qt, Kt) * scale[None, :, None]
    mask = torch.ones(N, N, dtype=torch.bool).tril()
    P = torch.softmax(S.masked_fill(~mask, float("-inf")), dim=-1)
    np.testing.assert_allclose(O, torch.einsum("gij,jd->gid", P, Vt).numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(score, P.sum(dim=(0, 1)).numpy(), rtol=1e-10, atol=1e-12)
    assert abs(score.sum() - g * N) < 1e-9
