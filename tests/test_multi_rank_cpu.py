"""The N > 1 path of the benchmark is "replicas only": ranks run independent copies of the workload
and only the timing is combined (max over ranks, aggregate = world x per-rank units / that time).
That host logic is exercised here with two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    agg = bench.max_over_ranks(ms, dist, "cpu")
    rate = bench.whole_job_rate(8 * 100, world, agg)
    dist.barrier()
    if rank == 0:
        print(json.dumps(dict(agg=agg, rate=rate, world=world)))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29513", str(script)],
                         capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2 and res["agg"] == 15.0
    assert abs(res["rate"] - 2 * 800 / 0.015) < 1e-6


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_rate(100, 1, 1000.0) == 100.0


def test_cache_length_schedule_matches_the_oracle():
    """bench.py's integer schedule (used only to count algorithmic bytes) against the oracle's counters."""
    import numpy as np
    import bench
    import workloads
    from oracle.buzz_oracle import OracleHead
    w = workloads.scaled(workloads.get("C2"), prompt_min=700, prompt_max=700, window=64, budget=180)
    n, n_old = bench._after_prefill(700, w)
    h = OracleHead(1, 1, w.sink, w.window, w.segment, w.hitters, w.budget)
    N = 700
    h.set_state(0, N, np.arange(N), np.random.default_rng(0).random(N), np.zeros((N, 1)), np.zeros((N, 1)))
    while h.counts()[0] >= w.budget:
        h.evict()
    assert h.counts()[:2] == (n, n_old)
    for t in range(300):
        h.decode(np.zeros((1, 1)), np.zeros(1), np.zeros(1))
        h.evict()
        n, n_old, _ = bench._after_evict(n + 1, n_old, w)
        assert h.counts()[:2] == (n, n_old)
