#!/usr/bin/env python
"""Benchmark of the BUZZ hot path on B200: decode tokens/s with attention + eviction.

A "step" is one decode step of the whole attention stack (per layer: append, attention over the
compacted cache, score update, eviction trigger and, when a cache is full, its eviction). The
headline times it as one ``buzz_decode_layers`` call over all layers in fused-eviction mode (one
kernel launch per layer, the launches of a call overlap on the GPU, an instance that fills up is
evicted in the tail of the kernel that filled it). Beside it, on the same caches:

  * ``separate_evict``    the same call followed by ``buzz_evict(-1)`` as a launch of its own;
  * ``decode_step_loop``  one ``buzz_decode_step`` call per layer with an unrelated small kernel
                          between consecutive layers (what a transformer's decoder does: layer l+1's
                          inputs exist only after layer l's output), direct and replayed from a CUDA graph;
  * ``prefill``           the ``buzz_prefill`` calls that fill the caches;
  * ``evict``             each sequence's first and second decode-time eviction, timed as
                          ``buzz_evict`` calls of their own;
  * ``e2e``               the headline step through the host-buffer entry point.

The headline workload is the largest one that fits one GPU (C5, the multi-document QA shape);
``per_workload`` repeats the device-side legs on C2, C3 (long-context summarisation shape) and C4.

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

METRIC = "decode tokens/s (attention + BUZZ eviction)"


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
                                          "-i", str(self.index), "-lms", "50"],
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
    for fused in (False, True):
        small.set_fused_evict(fused)
        for layer in range(2):
            small.prefill(layer, q, k, k, cu, n, torch.empty_like(q))
        o = [torch.empty_like(q[:1]) for _ in range(2)]
        small.decode_layers([0, 1], [q[:1]] * 2, [k[:1]] * 2, [k[:1]] * 2, o)
        small.decode_step(0, q[:1], k[:1], k[:1], o[0])
        small.evict(-1)
    torch.cuda.synchronize()
    assert small.status() == 0
    small.close()


class Leg:
    """CUDA-event timing of a run of steps on the launching stream."""

    def __init__(self, stream, name=None):
        self.stream, self.name = stream, name              # name: an NVTX range a profiler can filter on
        self.a, self.b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def __enter__(self):
        torch.cuda.synchronize()
        if self.name:
            torch.cuda.nvtx.range_push(self.name)
        self.a.record(self.stream)
        return self

    def __exit__(self, *exc):
        self.b.record(self.stream)
        if self.name:
            torch.cuda.nvtx.range_pop()
        torch.cuda.synchronize()
        self.ms = self.a.elapsed_time(self.b)


def measure(w, K, W, peaks, dev, dist, world, *, headline, e2e_steps=0, evict_leg=True, loop_leg=True):
    """All device-side legs of one workload on one GPU. Returns a dict; the caller builds the JSON line."""
    from paper_2410_23079_b200 import Buzz
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    esize = 2 if w.dtype == "bf16" else 4
    lens = workloads.prompt_lengths(w)
    total = sum(lens)
    bz = Buzz(sink=w.sink, window=w.window, segment=w.segment, hitters=w.hitters, budget=w.budget,
              layers=w.layers, max_batch=w.batch, q_heads=w.q_heads, kv_heads=w.kv_heads,
              head_dim=w.head_dim, dtype=dt, max_prompt_tokens=total, device=dev)
    stream = torch.cuda.current_stream()
    _warm_library(w, dt, dev)
    res = dict(workload=_workload_name(w), state_gb=bz.state_bytes / 1e9)
    per_slot = 2 * w.head_dim * esize + 8                      # one K row, one V row, score read + write
    io = w.batch * (2 * w.q_heads + 2 * w.kv_heads) * w.head_dim * esize
    kernel = "decode_bf16_kernel" if w.dtype == "bf16" else "decode_kernel"

    # ---- prefill leg (fills the caches; timed per layer around the library call only) --------
    pre_ms = 0.0
    l0 = bz.launch_count()
    for layer in range(w.layers):
        q, k, v, cu = workloads.prefill_inputs(w, layer, dev)
        out = torch.empty_like(q)
        with Leg(stream, "prefill") as leg:
            bz.prefill(layer, q, k, v, cu, max(lens), out)
        pre_ms += leg.ms
        del q, k, v, out
    prefill_launches = bz.launch_count() - l0
    assert bz.status() == 0
    flops = sum(2.0 * n * n * w.head_dim for n in lens) * w.q_heads * w.layers   # 2 N^2 d per query head (causal)
    tf = flops / (pre_ms * 1e-3) / 1e12
    # each layer's prefill is a burst of a few ms between synchronisations: the burst peak is the fair
    # denominator; the sustained one is given beside it
    res["prefill"] = dict(ms=pre_ms, tokens_per_s=total * 1e3 / pre_ms, tflops_algorithmic=tf,
                          frac_of_bf16_peak=tf / peaks["bf16"], peak_tflops=peaks["bf16"],
                          frac_of_bf16_sustained=tf / peaks["bf16_sustained"],
                          frac_of_nominal_2250=tf / 2250.0, launches=prefill_launches)

    # ---- decode inputs: a pool of distinct steps per layer, reused cyclically ----------------
    pool = min(K + W, 16 if w.batch * w.q_heads > 512 else 64)
    dec = [workloads.decode_inputs(w, layer, dev, steps=pool) for layer in range(w.layers)]
    outs = [torch.empty_like(dec[layer][0][0]) for layer in range(w.layers)]
    counts = [_after_prefill(n, w) for n in lens]
    all_layers = list(range(w.layers))
    t = 0

    def step_layers():
        i = t % pool
        bz.decode_layers(all_layers, [d[0][i] for d in dec], [d[1][i] for d in dec], [d[2][i] for d in dec], outs)

    filler = torch.zeros(1 << 16, device=dev)

    def step_loop():
        i = t % pool
        for l in all_layers:
            bz.decode_step(l, dec[l][0][i], dec[l][1][i], dec[l][2][i], outs[l])
            filler.add_(1.0)                                  # stand-in for the caller's work between two attention calls

    def advance_counts():
        nonlocal counts, t
        slots, fired = 0, []
        new = []
        for b, (n, n_old) in enumerate(counts):
            n += 1
            slots += n
            n2, m2, f = _after_evict(n, n_old, w)
            if f:
                fired.append((b, n, n_old, m2))
            new.append((n2, m2))
        counts = new
        t += 1
        return slots, fired

    def decode_bytes(slot_sum, steps):
        return w.layers * (slot_sum * w.kv_heads * per_slot + steps * io)

    def own_evict_bytes(fired):
        # the method's own work per evicting instance: the score scan plus every surviving middle row read and written
        return sum(4 * (n - w.sink - w.window) + 2 * m2 * per_slot for (_, n, _, m2) in fired) * w.kv_heads * w.layers

    def run_leg(step_fn, fused, steps, evict_call, name=None):
        """`steps` steps; returns (ms, slot_sum, launches, evictions)."""
        bz.set_fused_evict(fused)
        slot_sum, ev = 0, 0
        l0 = bz.launch_count()
        with Leg(stream, name) as leg:
            for _ in range(steps):
                step_fn()
                if evict_call:
                    bz.evict(-1)
                s, f = advance_counts()
                slot_sum += s; ev += len(f)
        assert bz.status() == 0
        return leg.ms, slot_sum, bz.launch_count() - l0, ev

    def decode_summary(ms, slot_sum, steps, launches_per_step):
        b = decode_bytes(slot_sum, steps)
        gbs = b / (ms * 1e-3) / 1e9
        return dict(ms_per_step=ms / steps, us_per_launch=ms * 1e3 / (steps * launches_per_step), gbs=gbs,
                    frac_of_hbm_peak=gbs / peaks["hbm"], frac_of_nominal_8000=gbs / 8000.0,
                    tokens_per_s=w.batch * steps / (ms * 1e-3), steps=steps)

    # warm-up in both modes and both call patterns
    run_leg(step_layers, False, max(W - W // 2, 1), True)
    run_leg(step_layers, True, max(W // 2, 1), False)
    if loop_leg:
        run_leg(step_loop, True, 2, False)

    # ---- headline: fused eviction, one multi-layer call per step ------------------------------
    if dist:
        dist.barrier()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.3)
    ms, slot_sum, launches, ev = run_leg(step_layers, True, K, False, "headline")
    if dist:
        dist.barrier()
    res["clocks"] = sampler.stop()
    ms = max_over_ranks(ms, dist, dev)
    res["headline"] = dict(ms=ms, launches=launches, evictions=ev, **decode_summary(ms, slot_sum, K, w.layers))
    b_launch = decode_bytes(slot_sum, K) / (K * w.layers)
    res["roofline"] = dict(bound="hbm", kernel=kernel, achieved=res["headline"]["gbs"], peak=peaks["hbm"], unit="GB/s",
                           frac=res["headline"]["gbs"] / peaks["hbm"], frac_of_nominal_8000=res["headline"]["gbs"] / 8000.0,
                           peak_source=peaks["source"],
                           above_measured_peak=res["headline"]["gbs"] > peaks["hbm"],
                           traffic=_ncu_traffic(b_launch / per_slot if w.dtype == "bf16" else None),
                           bytes_per_launch=b_launch, us_per_launch=res["headline"]["us_per_launch"])

    # ---- the same step with the eviction as a launch of its own ------------------------------
    ms2, ss2, _, _ = run_leg(step_layers, False, K, True)
    res["separate_evict"] = decode_summary(ms2, ss2, K, w.layers)

    # ---- one call per layer, something else enqueued in between ------------------------------
    if loop_leg:
        ms3, ss3, _, _ = run_leg(step_loop, True, K, False)
        loop = dict(pattern="buzz_decode_step per layer, an unrelated small kernel after each, fused eviction",
                    **decode_summary(ms3, ss3, K, w.layers))
        # The same enqueue pattern replayed from a CUDA graph (no host time between launches), and the
        # filler kernels alone the same way: the difference is what a decode launch costs when it cannot
        # overlap with its neighbours (its duration plus one kernel boundary).
        try:
            side = torch.cuda.Stream()
            g_loop, g_fill = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
            i = t % pool
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g_fill, stream=side):
                    for l in all_layers:
                        filler.add_(1.0)
                with torch.cuda.graph(g_loop, stream=side):
                    for l in all_layers:
                        bz.decode_step(l, dec[l][0][i], dec[l][1][i], dec[l][2][i], outs[l], stream=side)
                        filler.add_(1.0)
            torch.cuda.synchronize()
            for _ in range(3):
                g_fill.replay()
            with Leg(stream) as leg_f:
                for _ in range(K):
                    g_fill.replay()
            slot_sum4 = 0
            with Leg(stream) as leg:
                for _ in range(K):
                    g_loop.replay()
                    s, _f = advance_counts()
                    slot_sum4 += s
            assert bz.status() == 0
            loop["graph_replay"] = decode_summary(leg.ms, slot_sum4, K, w.layers)
            loop["filler_us"] = leg_f.ms * 1e3 / (K * w.layers)
            loop["net_of_filler"] = decode_summary(leg.ms - leg_f.ms, slot_sum4, K, w.layers)
            del g_loop, g_fill
        except RuntimeError as e:                              # capture refused: report, do not fail the run
            loop["graph_replay"] = dict(error=str(e)[:200])
        res["decode_step_loop"] = loop

    # ---- host schedule against the device: lengths of a few instances ------------------------
    torch.cuda.synchronize()
    for (l, b, h) in {(0, 0, 0), (w.layers - 1, w.batch - 1, w.kv_heads - 1), (w.layers // 2, w.batch // 2, 0)}:
        st = bz.export_state(l, b, h)
        assert (st["n"], st["n_old"]) == counts[b], f"length schedule: device {st['n'], st['n_old']} host {counts[b]}"
    res["schedule_checked"] = True

    # ---- end-to-end leg: the headline step through the host-buffer entry point ---------------
    if e2e_steps:
        Ke = min(K, e2e_steps)
        nq = w.batch * w.q_heads * w.head_dim
        nk = w.batch * w.kv_heads * w.head_dim
        hin = torch.empty((pool, w.layers, nq + 2 * nk), dtype=dt).pin_memory()
        ho = torch.empty((w.layers, nq), dtype=dt).pin_memory()
        for l in range(w.layers):
            hin[:, l, :nq].copy_(dec[l][0].reshape(pool, nq))
            hin[:, l, nq:nq + nk].copy_(dec[l][1].reshape(pool, nk))
            hin[:, l, nq + nk:].copy_(dec[l][2].reshape(pool, nk))

        def step_host():
            bz.decode_layers_host(all_layers, hin[t % pool], ho)

        run_leg(step_host, True, 2, False)
        e2e_ms, _, _, _ = run_leg(step_host, True, Ke, False)
        e2e_ms = max_over_ranks(e2e_ms, dist, dev)
        res["e2e"] = dict(value=whole_job_rate(w.batch * Ke, world, e2e_ms), unit="tokens/s", steps=Ke,
                          h2d_bytes_per_step=w.layers * w.batch * (w.q_heads + 2 * w.kv_heads) * w.head_dim * esize,
                          d2h_bytes_per_step=w.layers * w.batch * w.q_heads * w.head_dim * esize)
        del hin, ho

    # ---- eviction leg: every sequence's first and second decode-time eviction -----------------
    if evict_leg:
        bz.set_fused_evict(False)
        rounds = [dict(calls=0, ms=0.0, ms_max=0.0, sequences=0, bytes=0) for _ in range(2)]
        seen = [0] * w.batch
        cycle = []                                   # steps from a sequence's second eviction to its next one
        idle_ms, idle_calls, guard = 0.0, 0, 0
        while min(seen) < 2 and guard < 20000:
            guard += 1
            due = any(n + 1 >= w.budget for n, _ in counts)
            step_layers()
            timed = due or idle_calls < 8
            if timed:
                with Leg(stream, "evict_due" if due else None) as leg:
                    bz.evict(-1)
            else:
                bz.evict(-1)
            _, fired = advance_counts()
            assert bool(fired) == due
            if not fired:
                if timed:
                    idle_ms += leg.ms; idle_calls += 1
                continue
            for r in (0, 1):
                part = [f for f in fired if seen[f[0]] == r]
                if part:
                    d = rounds[r]
                    d["calls"] += 1; d["ms"] += leg.ms * len(part) / len(fired); d["ms_max"] = max(d["ms_max"], leg.ms)
                    d["sequences"] += len(part); d["bytes"] += own_evict_bytes(part)
                    if r == 1:
                        cycle += [w.budget - (w.sink + f[3] + w.window) for f in part]
            for f in fired:
                seen[f[0]] += 1
        assert bz.status() == 0
        for d in rounds:
            d["gbs"] = d["bytes"] / (d["ms"] * 1e-3) / 1e9 if d["ms"] else None
            d["frac_of_hbm_peak"] = d["gbs"] / peaks["hbm"] if d["ms"] else None
        res["evict"] = dict(first=rounds[0], second=rounds[1], at_step=t,
                            bytes_counted="score scan + surviving middle rows read and written (the window ring is not moved)",
                            idle_call_us=(idle_ms / idle_calls * 1e3) if idle_calls else None,
                            steps_between_evictions=statistics.mean(cycle) if cycle else None,
                            amortised_us_per_step=(rounds[1]["ms"] * 1e3 / statistics.mean(cycle)) if cycle else None)
    bz.close()
    del bz, dec, outs
    torch.cuda.empty_cache()
    return res


def run_ours(args):
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
    K, W = args.steps, max(args.warmup, 3)
    peaks = _peaks()
    head = measure(w, K, W, peaks, dev, dist, world, headline=True, e2e_steps=args.e2e_steps,
                   evict_leg=not args.no_evict_leg, loop_leg=not args.no_loop_leg)
    per = {}
    if world == 1:
        for name in [x for x in args.legs.split(",") if x and x != w.name]:
            wl = workloads.get(name)
            if args.layers:
                wl = workloads.scaled(wl, layers=args.layers)
            r = measure(wl, K, W, peaks, dev, None, 1, headline=False, evict_leg=not args.no_evict_leg,
                        loop_leg=not args.no_loop_leg)
            r.pop("clocks", None)
            per[name] = r
    hl = head["headline"]
    line = dict(metric=METRIC, value=whole_job_rate(w.batch * K, world, hl["ms"]),
                unit="tokens/s", n_gpus=world, steps=K, warmup=W, ms_per_step=hl["ms"] / K, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype=w.dtype, data="synthetic",
                config=dict(workload=head["workload"],
                            parallelism="replicas only" if world > 1 else "single GPU",
                            step="buzz_decode_layers over all layers, fused eviction (an instance that fills up is evicted in the tail of the kernel that filled it)",
                            l2="per-step K/V working set (GBs) exceeds the 126 MB L2; no flush needed",
                            state_gb=head["state_gb"], evictions_in_timed_region=hl["evictions"],
                            schedule_checked_against_device=head["schedule_checked"]),
                clocks=head["clocks"], e2e=head.get("e2e"), gpu_launches=hl["launches"], roofline=head["roofline"],
                prefill=head["prefill"], separate_evict=head["separate_evict"],
                decode_step_loop=head.get("decode_step_loop"), evict=head.get("evict"), per_workload=per)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, seconds=args.cpu_seconds, extras=True)
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def cpu_baseline(w, seconds=15.0, steps=4, extras=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload's decode steps: as
    many (layer, sequence, head) instances as fit the time box, one thread per host core. Each
    instance's state is generated before its clock starts. With `extras`, also one firing eviction
    per instance at the workload's shape and the oracle's prefill of all of C1 and of one C2 instance."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    from oracle.buzz_oracle import OracleHead
    cores = os.cpu_count() or 1
    n0, n_old0 = _after_prefill(w.prompt_min, w)
    n_mid = min(n0 + w.decode_steps // 2, w.budget - steps - 1)
    g, d = w.group, w.head_dim

    def planted(seed, n, n_old):
        r = np.random.default_rng(seed)
        h = OracleHead(g, d, w.sink, w.window, w.segment, w.hitters, w.budget)
        h.set_state(n_old, n + 10, np.arange(n), r.random(n), r.standard_normal((n, d)), r.standard_normal((n, d)))
        return h, r

    def one_instance(seed):
        h, r = planted(seed, n_mid, min(n_old0, n_mid - w.sink - w.window) if n_mid > w.sink + w.window else 0)
        q, k, v = r.standard_normal((steps, g, d)), r.standard_normal((steps, d)), r.standard_normal((steps, d))
        t0 = time.perf_counter()
        for s in range(steps):
            h.decode(q[s], k[s], v[s])
            h.evict()
        return time.perf_counter() - t0

    one_instance(1)   # warm the library
    t0 = time.perf_counter()
    done, busy = 0, 0.0
    with ThreadPoolExecutor(max_workers=cores) as ex:
        batch_id = 0
        while time.perf_counter() - t0 < seconds:
            busy += sum(ex.map(one_instance, range(batch_id * cores, (batch_id + 1) * cores)))
            done += cores
            batch_id += 1
    wall = time.perf_counter() - t0
    inst_steps_per_s = done * steps / (busy / cores)            # `cores` instances run side by side
    tokens_per_s = inst_steps_per_s / (w.layers * w.kv_heads)   # one token = L x Hkv instance-steps
    out = dict(value=tokens_per_s, unit="tokens/s", cores=cores, kind="oracle",
               sample=f"{done} (layer, sequence, head) instances x {steps} decode+evict steps at n={n_mid} slots on random "
                      f"state of the workload's shape, scaled by the {w.layers * w.kv_heads} instances one token needs; "
                      f"state generation is outside the clock",
               wall_s=wall)
    if extras:
        # one firing eviction per instance (full cache, old and new tokens both present)
        def one_eviction(seed):
            h, _ = planted(seed, w.budget, n_old0)
            t0 = time.perf_counter()
            fired = h.evict()
            dt = time.perf_counter() - t0
            assert fired == 1
            return dt
        with ThreadPoolExecutor(max_workers=cores) as ex:
            ts = list(ex.map(one_eviction, range(4 * cores)))
        per_inst = sum(ts) / len(ts)
        out["evict"] = dict(ms_per_instance=per_inst * 1e3,
                            s_all_instances=per_inst * w.layers * w.batch * w.kv_heads / cores,
                            sample=f"{len(ts)} instances with a full cache (n = budget = {w.budget}, n_old = {n_old0}), "
                                   f"scaled to the {w.layers * w.batch * w.kv_heads} instances of one eviction of the whole batch over {cores} cores")
        # prefill: all of C1, and one (layer, sequence, head) instance of C2
        pre = {}
        for name in ("C1", "C2"):
            wl = workloads.get(name)
            small = workloads.scaled(wl, layers=1, batch=1, q_heads=wl.group, kv_heads=1)
            q, k, v, _cu = workloads.prefill_inputs(small, 0, "cpu")
            Q = q.to(torch.float64).numpy().transpose(1, 0, 2)
            h = OracleHead(wl.group, wl.head_dim, wl.sink, wl.window, wl.segment, wl.hitters, wl.budget)
            t0 = time.perf_counter()
            h.prefill(Q, k[:, 0].to(torch.float64).numpy(), v[:, 0].to(torch.float64).numpy())
            dt = time.perf_counter() - t0
            inst = wl.layers * wl.batch * wl.kv_heads
            pre[name] = dict(s_one_instance=dt, tokens=wl.prompt_min, instances_in_workload=inst,
                             s_whole_workload_scaled=dt * inst / min(cores, inst))
        out["prefill"] = pre
    return out


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
    line = dict(impl="reference", metric=METRIC, value=v, unit="tokens/s",
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
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", help="headline workload (default: the largest that fits one GPU)")
    ap.add_argument("--legs", default="C2,C3,C4", help="further workloads measured into per_workload (single GPU only)")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling small cases)")
    ap.add_argument("--e2e-steps", type=int, default=32)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-evict-leg", action="store_true")
    ap.add_argument("--no-loop-leg", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
