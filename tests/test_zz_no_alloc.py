"""buzz_prefill_static: the prefill entry point for callers that cannot allocate device memory.

Code embedded in someone else's memory pool, a real-time loop, or a process whose device memory
was handed out once at start-up has nowhere to get the prefill's temporary buffers from. That
entry point keeps them in a fixed array inside the library instead. This file checks it, through
the C ABI, against the ordinary buzz_prefill on the same inputs, twice in a row (the array is
shared by all calls and keeps the previous call's contents, so a second call with different
inputs must not be disturbed by the first), and checks that an oversized request is refused.
It is named to be collected last, so a run that stops at the first failure has already run every
other test; it passes alone in a fresh process as well as after the others.
"""
import pytest
import torch

import workloads
from paper_2410_23079_b200 import BuzzError
from tests.harness import TOL, make_buzz

pytestmark = pytest.mark.gpu


def _prefill_both(w, layer, check_allocations=False):
    dev = "cuda:0"
    q, k, v, cu = workloads.prefill_inputs(w, layer, dev)
    lens = workloads.prompt_lengths(w)
    ref, new = make_buzz(w), make_buzz(w)
    out_ref, out_new = torch.empty_like(q), torch.empty_like(q)
    ref.prefill(layer, q, k, v, cu, max(lens), out_ref)
    torch.cuda.synchronize()
    before = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated())
    new.prefill_static(layer, q, k, v, cu, max(lens), out_new)
    torch.cuda.synchronize()
    after = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated())
    if check_allocations:
        # From the second call on a device on, the entry point must leave the device's free memory and
        # the framework's allocator untouched (the first call may make the driver load the library's
        # device code, which places the built-in array).
        assert after == before, f"device memory changed across buzz_prefill_static: {before} -> {after}"
    assert ref.status() == 0 and new.status() == 0
    scores_ref = [ref.export_prefill_scores(h, q.shape[0]) for h in range(w.kv_heads)]
    return ref, new, out_ref, out_new, scores_ref


def _same_or_near_tie(pos_ref, pos_new, score_ref, w):
    """The two entry points compute the scores with different kernels (equal to rel 1e-3), so a
    segment whose two best candidates are tied to that precision may keep either. Positions only one
    side kept are paired in order; each pair must lie in one segment and be such a tie."""
    a, b = set(pos_ref.tolist()), set(pos_new.tolist())
    only_ref, only_new = sorted(a - b), sorted(b - a)
    assert len(only_ref) == len(only_new)
    for p, r in zip(only_ref, only_new):
        assert abs(p - r) < w.segment
        x, y = float(score_ref[p]), float(score_ref[r])
        assert abs(x - y) <= 3e-3 * max(abs(x), abs(y)), (p, r, x, y)


@pytest.mark.parametrize("name,over", [
    ("C2", dict(layers=2, batch=2, q_heads=4, kv_heads=4, prompt_min=600, prompt_max=600, window=64, budget=200)),
    ("C4", dict(layers=2, batch=3, q_heads=8, kv_heads=2, prompt_min=300, prompt_max=700, window=48, budget=160)),
])
def test_static_prefill_matches_prefill_twice(cuda_device, name, over):
    w = workloads.scaled(workloads.get(name), **over)
    tol = TOL[w.dtype]
    lens = workloads.prompt_lengths(w)
    offs = [0]
    for n in lens:
        offs.append(offs[-1] + n)
    for call, layer in enumerate((0, 1)):           # two calls in a row, different inputs each
        ref, new, out_ref, out_new, scores_ref = _prefill_both(w, layer, check_allocations=call > 0)
        torch.testing.assert_close(out_new.float(), out_ref.float(), atol=tol["atol"], rtol=tol["rtol"])
        for b in range(w.batch):
            for h in range(w.kv_heads):
                a, c = ref.export_state(layer, b, h), new.export_state(layer, b, h)
                assert (a["n"], a["n_old"], a["total_len"]) == (c["n"], c["n_old"], c["total_len"]), (call, b, h)
                if torch.equal(a["pos"], c["pos"]):
                    assert torch.equal(a["k"], c["k"]) and torch.equal(a["v"], c["v"])
                    torch.testing.assert_close(c["score"], a["score"], atol=0.0, rtol=1e-3)
                else:
                    _same_or_near_tie(a["pos"], c["pos"], scores_ref[h][offs[b]:offs[b + 1]], w)
        ref.close(); new.close()


def test_static_prefill_refuses_oversized_requests(cuda_device):
    """(q_heads + kv_heads) * tokens beyond the built-in 1,048,576 floats: a clear error, no launch."""
    w = workloads.scaled(workloads.get("C2"), layers=1, batch=1, q_heads=32, kv_heads=32,
                         prompt_min=16385, prompt_max=16385, budget=1843)
    bz = make_buzz(w)
    q = torch.zeros(16385, 32, 128, dtype=torch.bfloat16, device="cuda:0")
    cu = torch.tensor([0, 16385], dtype=torch.int32, device="cuda:0")
    with pytest.raises(BuzzError) as ei:
        bz.prefill_static(0, q, q, q, cu, 16385, torch.empty_like(q))
    assert ei.value.code == -6
    assert bz.export_state(0, 0, 0)["n"] == 0        # nothing ran
    bz.close()
