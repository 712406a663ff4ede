#!/usr/bin/env python
"""Benchmark of the BUZZ hot path on B200: decode tokens/s with attention + eviction.

A "step" is one decode step of the whole attention stack: ``buzz_decode_layers`` over all layers
(per layer: append, attention over the compacted cache, score update; one kernel launch per layer,
the launches of a call overlap on the GPU), then ``buzz_evict`` for all layers.
The caches are first filled by ``buzz_prefill`` of the workload's prompts (timed as its own leg and
reported under ``prefill``); after the timed steps the run continues until the first decode-time
eviction and times that call (``evict``).

Prints ONE JSON line. ``--impl reference`` times the CPU oracle instead (a deliberately slow
program; the line then carries ``"impl": "reference"``).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=p["hbm_gbs"], bf16=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def _ncu_traffic(slots_per_launch):
    """DRAM bytes per launch of the decode kernel from the committed ncu capture, scaled by the slots
    one launch processes; None if there is no capture or the kernel source changed since it."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if slots_per_launch is None or not os.path.exists(path):
        return None
    kv = {}
    for line in open(path):
        if "=" in line and not line.startswith("#"):
            a, b = line.split("=", 1)
            kv[a.strip()] = b.strip()
    try:
        src = os.path.join(ROOT, kv["kernel_source"])
        if hashlib.sha1(open(src, "rb").read()).hexdigest() != kv["kernel_source_sha1"]:
            return None
        return float(kv["dram_bytes_per_slot"]) * slots_per_launch
    except (KeyError, OSError, ValueError):
        return None


# ---- integer schedule of the cache length (no scores involved) ---------------------------------
def _after_prefill(N, w):
    if N < w.budget:
        return N, 0
    mid = N - w.sink - w.window
    nseg = -(-mid // w.segment)
    last = mid - (nseg - 1) * w.segment
    m = (nseg - 1) * w.hitters + min(w.hitters, last)
    s_hat = (w.segment + 1) // 2
    while w.sink + m + w.window >= w.budget:
        m = -(-m // s_hat)
    return w.sink + m + w.window, m


def _after_evict(n, n_old, w):
    if n < w.budget:
        return n, n_old, False
    s_hat = (w.segment + 1) // 2
    n_new = n - w.sink - w.window - n_old
    nseg = -(-n_new // w.segment)
    kept_new = 0 if nseg == 0 else (nseg - 1) * w.hitters + min(w.hitters, n_new - (nseg - 1) * w.segment)
    m = -(-n_old // s_hat) + kept_new
    return w.sink + m + w.window, m, True


def _workload_name(w) -> str:
    return (f"{w.name}: {w.layers} layers x {w.batch} seqs x {w.q_heads}/{w.kv_heads} heads, d={w.head_dim}, "
            f"prompt {w.prompt_min}..{w.prompt_max}, sink {w.sink} window {w.window} segment {w.segment} "
            f"hitters {w.hitters} budget {w.budget}")


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's time: every multi-GPU number is the max over ranks (replicas run independently)."""
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Aggregate throughput of `world` replicas that each processed units_per_rank in ms (max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1]))
                except ValueError:
                    continue
                for nm, val in zip(names, p[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def _warm_library(w, dt, dev):
    """One throw-away pass of every kernel on a tiny object of the same head shape, so that module
    loading and one-time attribute set-up are not charged to the first timed call."""
    from paper_2410_23079_b200 import Buzz
    n = 512
    small = Buzz(sink=w.sink, window=w.window, segment=w.segment, hitters=w.hitters, budget=w.budget, layers=2,
                 max_batch=1, q_heads=w.q_heads, kv_heads=w.kv_heads, head_dim=w.head_dim, dtype=dt,
                 max_prompt_tokens=n, device=dev)
    cu = torch.tensor([0, n], dtype=torch.int32, device=dev)
    q = torch.randn((n, w.q_heads, w.head_dim), device=dev).to(dt)
    k = torch.randn((n, w.kv_heads, w.head_dim), device=dev).to(dt)
    for layer in range(2):
        small.prefill(layer, q, k, k, cu, n, torch.empty_like(q))
    o = [torch.empty_like(q[:1]) for _ in range(2)]
    small.decode_layers([0, 1], [q[:1]] * 2, [k[:1]] * 2, [k[:1]] * 2, o)
    small.evict(-1)
    torch.cuda.synchronize()
    assert small.status() == 0
    small.close()


def run_ours(args):
    from paper_2410_23079_b200 import Buzz
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    w = workloads.get(args.workload)
    if args.layers:
        w = workloads.scaled(w, layers=args.layers)
    K, W = args.steps, args.warmup
    peaks = _peaks()
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    esize = 2 if w.dtype == "bf16" else 4
    lens = workloads.prompt_lengths(w)
    total = sum(lens)
    bz = Buzz(sink=w.sink, window=w.window, segment=w.segment, hitters=w.hitters, budget=w.budget,
              layers=w.layers, max_batch=w.batch, q_heads=w.q_heads, kv_heads=w.kv_heads,
              head_dim=w.head_dim, dtype=dt, max_prompt_tokens=total, device=dev)
    stream = torch.cuda.current_stream()
    _warm_library(w, dt, dev)

    # ---- prefill leg (fills the caches; timed per layer around the library call only) --------
    pre_ms = 0.0
    l0 = bz.launch_count()
    for layer in range(w.layers):
        q, k, v, cu = workloads.prefill_inputs(w, layer, dev)
        out = torch.empty_like(q)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        bz.prefill(layer, q, k, v, cu, max(lens), out)
        b.record(stream)
        torch.cuda.synchronize()
        pre_ms += a.elapsed_time(b)
        del q, k, v, out
    prefill_launches = bz.launch_count() - l0
    assert bz.status() == 0
    flops = sum(2.0 * n * n * w.head_dim for n in lens) * w.q_heads * w.layers   # 2 N^2 d per query head (causal)
    prefill = dict(ms=pre_ms, tokens_per_s=total * 1e3 / pre_ms * 1.0,
                   tflops_algorithmic=flops / (pre_ms * 1e-3) / 1e12,
                   frac_of_bf16_peak=flops / (pre_ms * 1e-3) / 1e12 / peaks["bf16_sustained"],
                   peak_tflops=peaks["bf16_sustained"], launches=prefill_launches)

    # ---- decode inputs: a pool of distinct steps per layer, reused cyclically ----------------
    pool = min(K + W, 64)
    dec = [workloads.decode_inputs(w, layer, dev, steps=pool) for layer in range(w.layers)]
    outs = [torch.empty_like(dec[layer][0][0]) for layer in range(w.layers)]
    counts = [_after_prefill(n, w) for n in lens]

    all_layers = list(range(w.layers))

    def step(t):
        i = t % pool
        bz.decode_layers(all_layers, [d[0][i] for d in dec], [d[1][i] for d in dec], [d[2][i] for d in dec], outs)

    def advance_counts():
        nonlocal counts
        tot, ev = 0, 0
        new = []
        for (n, n_old) in counts:
            n += 1
            tot += n
            n, n_old, fired = _after_evict(n, n_old, w)
            ev += fired
            new.append((n, n_old))
        counts = new
        return tot, ev

    t = 0
    for _ in range(W):
        step(t); bz.evict(-1); advance_counts(); t += 1
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    ev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = bz.launch_count()
    slot_sum, timed_evictions = 0, 0
    torch.cuda.synchronize()
    start.record(stream)
    for i in range(K):
        ev_pairs[i][0].record(stream)
        step(t)
        ev_pairs[i][1].record(stream)
        bz.evict(-1)
        s, e = advance_counts()
        slot_sum += s; timed_evictions += e
        t += 1
    end.record(stream)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.stop()
    launches = bz.launch_count() - l0
    ms = start.elapsed_time(end)
    assert bz.status() == 0
    ms = max_over_ranks(ms, dist, dev)
    decode_ms = sum(a.elapsed_time(b) for a, b in ev_pairs)
    # algorithmic bytes of all decode launches in the timed region (per layer the same lengths)
    per_slot = 2 * w.head_dim * esize + 8
    io = w.batch * (2 * w.q_heads + 2 * w.kv_heads) * w.head_dim * esize
    bytes_all = w.layers * (slot_sum * w.kv_heads * per_slot + K * io)
    n_launch = w.layers * K
    achieved = bytes_all / (decode_ms * 1e-3) / 1e9
    traffic = _ncu_traffic(bytes_all / n_launch / per_slot if w.dtype == "bf16" else None)
    roofline = dict(bound="hbm", kernel="decode_bf16_kernel" if w.dtype == "bf16" else "decode_kernel", achieved=achieved, peak=peaks["hbm"], unit="GB/s",
                    frac=achieved / peaks["hbm"], frac_of_nominal_8000=achieved / 8000.0, peak_source=peaks["source"],
                    traffic=traffic, bytes_per_launch=bytes_all / n_launch,
                    us_per_launch=decode_ms * 1e3 / n_launch)

    # ---- end-to-end leg: the same step through the host-buffer entry point -------------------
    Ke = min(K, args.e2e_steps)
    # pinned host inputs: per step one packed buffer, for each layer q | k_new | v_new, so that a step's
    # inputs go down in one copy and its outputs come back in one
    nq = w.batch * w.q_heads * w.head_dim
    nk = w.batch * w.kv_heads * w.head_dim
    hin = torch.empty((pool, w.layers, nq + 2 * nk), dtype=dt).pin_memory()
    ho = torch.empty((w.layers, nq), dtype=dt).pin_memory()
    for l in range(w.layers):
        hin[:, l, :nq].copy_(dec[l][0].reshape(pool, nq))
        hin[:, l, nq:nq + nk].copy_(dec[l][1].reshape(pool, nk))
        hin[:, l, nq + nk:].copy_(dec[l][2].reshape(pool, nk))
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(Ke):
        bz.decode_layers_host(all_layers, hin[t % pool], ho)
        bz.evict(-1)
        advance_counts(); t += 1
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    h2d = w.layers * w.batch * (w.q_heads + 2 * w.kv_heads) * w.head_dim * esize
    d2h = w.layers * w.batch * w.q_heads * w.head_dim * esize
    e2e = dict(value=whole_job_rate(w.batch * Ke, world, e2e_ms), unit="tokens/s", steps=Ke,
               h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h)
    assert bz.status() == 0

    # ---- eviction leg: keep decoding until the first, then the second, decode-time eviction; time those calls ----
    def timed_eviction():
        nonlocal t
        guard = 0
        while max(n for n, _ in counts) + 1 < w.budget and guard < 5000:
            step(t); bz.evict(-1); advance_counts(); t += 1; guard += 1
        step(t)
        before = [(n + 1, n_old) for n, n_old in counts]
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        bz.evict(-1)
        b.record(stream)
        torch.cuda.synchronize()
        advance_counts(); t += 1
        ev_ms = a.elapsed_time(b)
        moved = 0
        for (n, n_old) in before:
            n2, m2, fired = _after_evict(n, n_old, w)
            if fired:
                moved += 4 * (n - w.sink - w.window) + 2 * (n2 - w.sink) * per_slot   # scan + rows read and written
        ev_bytes = moved * w.kv_heads * w.layers
        return dict(ms=ev_ms, sequences_evicting=sum(1 for n, _ in before if n >= w.budget),
                    gbs=ev_bytes / (ev_ms * 1e-3) / 1e9, frac_of_hbm_peak=ev_bytes / (ev_ms * 1e-3) / 1e9 / peaks["hbm"],
                    bytes=ev_bytes, at_step=t)

    evict = None
    if not args.no_evict_leg:
        evict = timed_eviction()
        evict["second"] = timed_eviction()             # old and new tokens both present this time
        assert bz.status() == 0

    line = dict(metric="decode tokens/s (attention + BUZZ eviction)", value=whole_job_rate(w.batch * K, world, ms),
                unit="tokens/s", n_gpus=world, steps=K, warmup=W, ms_per_step=ms / K, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype=w.dtype, data="synthetic",
                config=dict(workload=_workload_name(w),
                            parallelism="replicas only" if world > 1 else "single GPU",
                            l2="per-step K/V working set (GBs) exceeds the 126 MB L2; no flush needed",
                            decode_input_pool=pool, evictions_in_timed_region=timed_evictions),
                clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roofline, prefill=prefill, evict=evict)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, seconds=args.cpu_seconds)
        print(json.dumps(line))
    bz.close()
    if dist:
        dist.destroy_process_group()


def cpu_baseline(w, seconds=15.0, steps=4):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload's decode steps:
    as many (layer, sequence, head) instances as fit the time box, one thread per host core."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    from oracle.buzz_oracle import OracleHead
    cores = os.cpu_count() or 1
    n0, n_old0 = _after_prefill(w.prompt_min, w)
    n_mid = min(n0 + w.decode_steps // 2, w.budget - steps - 1)
    g, d = w.group, w.head_dim
    rng = np.random.default_rng(0)

    def one_instance(seed):
        r = np.random.default_rng(seed)
        h = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, w.budget)
        h.set_state(min(n_old0, n_mid - w.sink - w.window) if n_mid > w.sink + w.window else 0, n_mid + 10,
                    np.arange(n_mid), r.random(n_mid), r.standard_normal((n_mid, d)), r.standard_normal((n_mid, d)))
        q, k, v = r.standard_normal((steps, g, d)), r.standard_normal((steps, d)), r.standard_normal((steps, d))
        t0 = time.perf_counter()
        for s in range(steps):
            h.decode(q[s], k[s], v[s])
            h.evict()
        return time.perf_counter() - t0

    one_instance(1)   # warm the library
    t0 = time.perf_counter()
    done = 0
    with ThreadPoolExecutor(max_workers=cores) as ex:
        batch_id = 0
        while time.perf_counter() - t0 < seconds:
            list(ex.map(one_instance, range(batch_id * cores, (batch_id + 1) * cores)))
            done += cores
            batch_id += 1
    wall = time.perf_counter() - t0
    inst_steps_per_s = done * steps / wall
    tokens_per_s = inst_steps_per_s / (w.layers * w.kv_heads)     # one token = L x Hkv instance-steps
    return dict(value=tokens_per_s, unit="tokens/s", cores=cores, kind="oracle",
                sample=f"{done} (layer, sequence, head) instances x {steps} decode+evict steps at n={n_mid} slots, "
                       f"scaled by the {w.layers * w.kv_heads} instances one token needs; includes generating each instance's random state",
                wall_s=wall)


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    w = workloads.get(args.workload)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        cpu_baseline(w, seconds=per_step)
    vals = [cpu_baseline(w, seconds=per_step) for _ in range(args.steps)]
    v = statistics.mean(x["value"] for x in vals)
    base = dict(vals[-1]); base["value"] = v
    line = dict(impl="reference", metric="decode tokens/s (attention + BUZZ eviction)", value=v, unit="tokens/s",
                n_gpus=int(os.environ.get("WORLD_SIZE", 1)), steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * w.batch / v, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload=_workload_name(w), sample="each step is a bounded sample of this workload, see cpu_baseline.sample"),
                cpu_baseline=base, e2e=dict(value=v, unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling small cases)")
    ap.add_argument("--e2e-steps", type=int, default=64)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-evict-leg", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
