#!/usr/bin/env python
"""Benchmark of the sink+window attention hot path (one JSON line on stdout).

A *step* is one pass of the whole hot path over one chunk of synthetic input at
the Wan-1.3B-shaped single-layer workload: fused 3-D RoPE + K/V append of a new
3-frame chunk (4680 tokens x 12 heads x 128), then sink+window attention of its
queries over the full cache (18720 keys).  The caches of several layers are
rotated from step to step so that every step finds its K/V cold in L2.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

value      : attention TFLOP/s over the whole step time (append included), inputs
             resident in HBM.
e2e        : the same with pinned host Q/K/V copied in and the output copied out
             inside the timed region (copies of neighbouring steps overlap the kernels).
roofline   : the attention kernel alone against the measured dense bf16 peak.
cpu_baseline / --impl reference: the fp64 CPU oracle on a bounded sample of the
             same workload's query rows.
extra.in_loop: the same step repeated for at least two seconds, whatever --steps
             is: the GPU then sits at its power limit and the figure is the one a long
             stream sees; the --steps region of a short run is a burst.
With N > 1 every rank runs an independent replica (the path has no exchange
step); value is the sum over ranks divided by the slowest rank's time.  Started
without a launcher (no WORLD_SIZE in the environment), --gpus N > 1 starts the N
ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_22622_b200 import synth  # noqa: E402

WL = synth.CONFIGS[1]
N_LAYERS = 4               # caches rotated across steps (4 x 115 MB > L2)
N_INPUT_SETS = 4
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def steady_keys(wl):
    return (wl.sink_frames + wl.window_frames) * wl.tokens_per_frame


def attn_flops(wl, n_rows=None):
    nq = wl.chunk_tokens if n_rows is None else n_rows
    return 4.0 * nq * steady_keys(wl) * wl.head_dim * wl.heads


def append_bytes(wl):
    # Q in + Q out + K in + K cache + V in + V cache
    return 6.0 * wl.chunk_tokens * wl.heads * wl.head_dim * 2


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """Per-launch DRAM bytes of the kernels from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    out = {}
    if os.path.exists(path):
        with open(path) as fh:
            for line in fh:
                parts = line.split("#")[0].split()
                if len(parts) == 2:
                    out[parts[0]] = float(parts[1])
    return out


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""

    def __init__(self, index: int):
        self.path = "/tmp/llattn_clocks_%d_%d.csv" % (os.getpid(), index)
        self.proc = None
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + CLOCK_QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as fh:
            for line in fh:
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); smax.append(float(f[2])); power.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [c for c, p in zip(sm, power) if p > 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# ---------------------------------------------------------------------------
# the oracle leg (CPU baseline / reference arm)
# ---------------------------------------------------------------------------

def oracle_sample(target_seconds: float, steps: int = 1, warmup: int = 0):
    """Time the fp64 oracle on a bounded sample of query rows of one steady-state
    attention call of the workload.  Returns (tflops, cores, description, ms_per_step)."""
    import oracle
    oracle.build()
    wl = WL
    C, P = wl.chunk_frames, wl.tokens_per_frame
    cores = len(os.sched_getaffinity(0))
    orc = oracle.Oracle(1, wl.heads, wl.head_dim, P, C, wl.sink_frames, wl.window_frames)
    n_fill = (wl.sink_frames + wl.window_frames) // C
    t_append = 0.0
    for chunk in range(n_fill):
        _, k, v = synth.chunk_qkv(wl, chunk)
        t0 = time.perf_counter()
        orc.append(0, synth.bf16_bits_to_f64(k), synth.bf16_bits_to_f64(v), chunk * C, wl.grid_h, wl.grid_w)
        t_append = time.perf_counter() - t0
    q, _, _ = synth.chunk_qkv(wl, n_fill - 1)
    qr = orc.rope_q(synth.bf16_bits_to_f64(q), (n_fill - 1) * C, wl.grid_h, wl.grid_w)
    # calibrate: rows the oracle gets through in about target_seconds
    probe = synth.sample_rows(C * P, 2 * cores, seed=1, edges=False)
    t0 = time.perf_counter()
    orc.attn(0, qr, (n_fill - 1) * C, rows=probe)
    per_row = (time.perf_counter() - t0) / len(probe)
    n_rows = int(max(cores, min(C * P, target_seconds / per_row)))
    n_rows = max(cores, n_rows // cores * cores)
    rows = synth.sample_rows(C * P, n_rows, seed=2, edges=False)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.attn(0, qr, (n_fill - 1) * C, rows=rows)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    dt = sum(times) / len(times)
    tflops = attn_flops(wl, len(rows)) / dt / 1e12
    what = ("%d of %d query rows x all %d heads x %d keys of one steady-state attention call, fp64, "
            "%d OpenMP threads; one oracle append of a chunk took %.2f s"
            % (len(rows), C * P, wl.heads, steady_keys(wl), cores, t_append))
    orc.close()
    return tflops, cores, what, dt * 1e3


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # about two minutes of oracle time in all, whatever the step count (a step never samples
    # fewer query rows than there are cores)
    per_step = min(20.0, 120.0 / max(1, args.steps + args.warmup))
    tflops, cores, what, ms = oracle_sample(per_step, steps=args.steps, warmup=args.warmup)
    line = {
        "impl": "reference", "metric": "sink_window_attn_tflops", "value": tflops, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WL.name, "sample": what},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# multi-rank aggregation (replicas only: no data-path collective)
# ---------------------------------------------------------------------------

def reduce_max(values, dist, device="cpu"):
    """Element-wise max over ranks of a short list of per-rank timings (ms)."""
    if dist is None:
        return list(values)
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tflops(world: int, steps: int, flops_per_step: float, slowest_ms: float) -> float:
    """Every rank ran `steps` independent steps; the job took as long as its slowest rank."""
    return world * steps * flops_per_step / (slowest_ms * 1e-3) / 1e12


def spawn_ranks(args, argv):
    """`bench.py --gpus N` started by hand: launch N ranks of this script (one per GPU) and
    pass rank 0's JSON line through.  Returns the launcher's exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_dry(args):
    """The multi-rank plumbing without a GPU (gloo): every rank contributes made-up device
    times, the line is assembled as in the real run.  Measures nothing; for tests."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    total_ms = 10.0 + rank                      # the last rank is the slowest
    red = reduce_max([total_ms], dist if world > 1 else None, "cpu")
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"dry_run": True, "metric": "sink_window_attn_tflops", "n_gpus": world, "steps": args.steps,
                          "ms_per_step": red[0] / args.steps,
                          "value": whole_job_tflops(world, args.steps, attn_flops(WL), red[0])}))


# ---------------------------------------------------------------------------
# the CUDA leg
# ---------------------------------------------------------------------------

def run_ours(args):
    import torch
    from paper_2509_22622_b200 import binding as B
    from paper_2509_22622_b200 import build as _build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        _build.build()
    if dist is not None:
        dist.barrier()
    B.lib()

    wl = WL
    C, P, H, D = wl.chunk_frames, wl.tokens_per_frame, wl.heads, wl.head_dim
    nq = C * P
    n_fill = (wl.sink_frames + wl.window_frames) // C
    warmup = max(args.warmup, 3)
    stream = torch.cuda.current_stream()

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    cache = B.Cache(N_LAYERS, H, D, P, C, wl.sink_frames, wl.window_frames, device="cuda:%d" % local_rank)
    host_sets = [synth.chunk_qkv(wl, 100 + i, stream=rank) for i in range(N_INPUT_SETS)]
    dev_sets = [tuple(dev(t) for t in s) for s in host_sets]
    pinned = [tuple(torch.from_numpy(t.view(np.int16)).view(torch.bfloat16).pin_memory() for t in s)
              for s in host_sets]
    q_roped = torch.empty(nq, H, D, device="cuda", dtype=torch.bfloat16)
    out = torch.empty_like(q_roped)
    out_host = torch.empty(nq, H, D, dtype=torch.bfloat16).pin_memory()
    stage = tuple(torch.empty_like(q_roped) for _ in range(3))

    # untimed prefill: every layer reaches the steady state (ring full)
    for layer in range(N_LAYERS):
        for chunk in range(n_fill):
            q, k, v = dev_sets[(layer + chunk) % N_INPUT_SETS]
            cache.rope_append_kv(layer, q, k, v, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped)
    cache.check_device()
    step_no = [0]

    def step(ev=None):
        s = step_no[0]
        step_no[0] += 1
        layer = s % N_LAYERS
        fs = cache.state(layer)["end"]
        q, k, v = dev_sets[s % N_INPUT_SETS]
        cache.rope_append_kv(layer, q, k, v, fs, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped)
        if ev:
            ev[0].record(stream)
        cache.sink_window_attn(layer, q_roped, fs, out)
        if ev:
            ev[1].record(stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step()
    cache.check_device()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    time.sleep(0.3)
    launches0 = B.ll_launch_count()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record(stream)
    for i in range(args.steps):
        step(ev=events[i])
    t_end.record(stream)
    barrier()
    launches = B.ll_launch_count() - launches0
    total_ms = t_begin.elapsed_time(t_end)
    attn_ms = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    append_ms = total_ms / args.steps - attn_ms          # the rest of a step: the append, two launch gaps, two event records
    cache.check_device()

    # End to end: every step's Q/K/V come from pinned host memory and its output goes back
    # to the host, all inside the timed region.  The copies of neighbouring steps overlap the
    # kernels on two more streams (two sets of staging buffers), as a serving loop would do
    # it; a step still cannot start before its own inputs have landed.
    h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()
    stages = [stage, tuple(torch.empty_like(q_roped) for _ in range(3))]
    outs = [out, torch.empty_like(out)]
    outs_host = [out_host, torch.empty(nq, H, D, dtype=torch.bfloat16).pin_memory()]
    in_ready = [torch.cuda.Event() for _ in range(2)]      # inputs of the step using buffer b are on the device
    in_free = [torch.cuda.Event() for _ in range(2)]       # the kernels that read buffer b are done
    out_ready = [torch.cuda.Event() for _ in range(2)]
    out_free = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        s = step_no[0]
        step_no[0] += 1
        b = i % 2
        layer = s % N_LAYERS
        fs = cache.state(layer)["end"]
        with torch.cuda.stream(h2d_stream):
            if i >= 2:
                h2d_stream.wait_event(in_free[b])
            for dst, src in zip(stages[b], pinned[s % N_INPUT_SETS]):
                dst.copy_(src, non_blocking=True)
            in_ready[b].record(h2d_stream)
        stream.wait_event(in_ready[b])
        if i >= 2:
            stream.wait_event(out_free[b])
        q, k, v = stages[b]
        cache.rope_append_kv(layer, q, k, v, fs, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped)
        cache.sink_window_attn(layer, q_roped, fs, outs[b])
        in_free[b].record(stream)
        out_ready[b].record(stream)
        with torch.cuda.stream(d2h_stream):
            d2h_stream.wait_event(out_ready[b])
            outs_host[b].copy_(outs[b], non_blocking=True)
            out_free[b].record(d2h_stream)

    for i in range(4):
        e2e_step(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    h2d_stream.wait_event(e0)
    for i in range(args.steps):
        e2e_step(i)
    d2h_stream.wait_stream(stream)
    e1.record(d2h_stream)                                  # after the last output has reached the host
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    cache.check_device()

    # The same step for a fixed length of time, whatever --steps was: after about a second the
    # GPU sits at its power limit and the SM clock settles below its maximum, which is what a
    # long stream sees.  Its own clock samples are reported with it.
    in_loop = None
    if args.in_loop_seconds > 0:
        slowest_ms = reduce_max([total_ms], dist, "cuda")[0]            # every rank runs the same number of steps
        n_loop = max(args.steps, int(args.in_loop_seconds * 1e3 / max(slowest_ms / args.steps, 1e-3)) + 1)
        loop_sampler = ClockSampler(local_rank) if rank == 0 else None
        lev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_loop)]
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        l0.record(stream)
        for i in range(n_loop):
            step(ev=lev[i])
        l1.record(stream)
        barrier()
        loop_ms = l0.elapsed_time(l1)
        # the second half of the loop: the clock has settled by then
        half = lev[n_loop // 2:]
        loop_attn_ms = sum(e[0].elapsed_time(e[1]) for e in half) / len(half)
        loop_clocks = loop_sampler.stop() if loop_sampler else None
        cache.check_device()
        in_loop = {"steps": n_loop, "ms_total": loop_ms, "ms_per_step": loop_ms / n_loop,
                   "attn_ms_per_launch_second_half": loop_attn_ms, "clocks": loop_clocks}

    # The append kernel alone: launches back to back on rotating layers and input sets (each
    # overwrites its layer's newest chunk in place), one pair of events around all of them, so
    # that no launch gap is counted.
    n_app = 200
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def appends(n):
        for i in range(n):
            layer = i % N_LAYERS
            q, k, v = dev_sets[(i + i // N_LAYERS) % N_INPUT_SETS]
            cache.rope_append_kv(layer, q, k, v, cache.state(layer)["end"] - C, wl.grid_h, wl.grid_w, wl.rope_theta,
                                 q_roped)
    appends(8)
    barrier()
    a0.record(stream)
    appends(n_app)
    a1.record(stream)
    barrier()
    append_b2b_ms = a0.elapsed_time(a1) / n_app
    cache.check_device()


    # recache of the full window (one launch pair), reported beside the headline
    n_w = wl.window_frames
    rq, rk, rv = (dev(t) for t in synth.chunk_qkv(wl, 200, pass_id=synth.RECACHE_PASS, n_frames=n_w, stream=rank))
    rq_out, r_out = torch.empty_like(rq), torch.empty_like(rq)
    rc = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    cache.recache(0, rq, rk, rv, n_w, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, r_out)
    torch.cuda.synchronize()
    rc[0].record(stream)
    for _ in range(3):
        cache.recache(0, rq, rk, rv, n_w, wl.grid_h, wl.grid_w, wl.rope_theta, rq_out, r_out)
    rc[1].record(stream)
    torch.cuda.synchronize()
    recache_ms = rc[0].elapsed_time(rc[1]) / 3
    cache.check_device()

    # The other entry points at the same layer shape, a few launches each, reported beside the
    # headline: eight streams at ragged positions in one launch, a 21-frame clip in one call,
    # cross-attention over a 512-token prompt.
    def median_ms(fn, reps=10):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        return sorted(times)[len(times) // 2]

    others = {}
    if rank == 0:
        q, k, v = dev_sets[0]
        positions = synth.SWEEP_POSITIONS
        streams, items, flops8 = [], [], 0.0
        for pos in positions:
            c = B.Cache(1, H, D, P, C, wl.sink_frames, wl.window_frames, device="cuda:%d" % local_rank)
            qr = torch.empty_like(q)
            for chunk in range(pos + 1):
                c.rope_append_kv(0, q, k, v, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, qr)
            streams.append(c)
            items.append((c, 0, qr, pos * C, torch.empty_like(q), None))
            ring = min(pos + 1, wl.window_frames // C) * C
            sink = wl.sink_frames if pos + 1 > wl.window_frames // C else 0
            flops8 += 4.0 * nq * (ring + sink) * P * D * H
        ms = median_ms(lambda: B.Cache.sink_window_attn_batched(items))
        others["batched_8_ragged_streams"] = {"ms": ms, "tflops": flops8 / ms / 1e9, "positions": list(positions)}
        for c in streams:
            c.check_device()
            c.close()
        del streams, items
        clip_chunks = 7
        T = clip_chunks * C
        big = B.Cache(1, H, D, P, C, wl.sink_frames, wl.window_frames + T - C, device="cuda:%d" % local_rank)
        for chunk in range(n_fill):
            big.rope_append_kv(0, None, k, v, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta)
        cq, ck, cv = (torch.cat([dev_sets[i % N_INPUT_SETS][j] for i in range(clip_chunks)]) for j in range(3))
        cq_out, c_out = torch.empty_like(cq), torch.empty_like(cq)
        c_lse = torch.empty(H, T * P, device="cuda", dtype=torch.float32)
        pos = [n_fill * C]

        def clip():
            big.clip_append_attn(0, cq, ck, cv, pos[0], T, wl.window_frames, wl.grid_h, wl.grid_w, wl.rope_theta,
                                 cq_out, c_out, c_lse)
            pos[0] += T
        ms = median_ms(clip)
        others["clip_21_frames"] = {"ms": ms, "tflops_attention_over_append_plus_attention":
                                    clip_chunks * attn_flops(wl) / ms / 1e9}
        # backward of that clip (gradients for the clip's q, k, v; sink and context detached)
        d_out = torch.randn_like(cq)
        dq_g, dk_g, dv_g = (torch.empty_like(cq) for _ in range(3))
        bws = torch.empty(B.ll_clip_backward_workspace_bytes(big.h, T) + 256, dtype=torch.uint8, device="cuda")
        bws = bws[(-bws.data_ptr()) % 256:]
        ms = median_ms(lambda: B.ll_clip_attn_backward(big.h, 0, cq_out, c_out, d_out, c_lse, pos[0] - T, T, wl.window_frames,
                                                       wl.grid_h, wl.grid_w, wl.rope_theta, dq_g, dk_g, dv_g, bws), reps=5)
        all_f = clip_chunks * (wl.sink_frames + wl.window_frames)
        own_f = sum(min((g + 1) * C, wl.window_frames) for g in range(clip_chunks))
        bwd_flops = 2.0 * nq * P * D * H * (3 * all_f + 2 * own_f)      # S, dP, dQ over all keys; dK, dV over the clip's
        others["clip_21_frames_backward"] = {"ms": ms, "tflops_algorithmic": bwd_flops / ms / 1e9,
                                             "note": "S and dP are formed twice (dq kernel and dk/dv kernel): 7 products "
                                                     "run where 5 are counted"}
        big.check_device()
        big.close()
        gains = torch.ones(H * D, device="cuda")
        layer_i = [0]

        def norm_append(n=20):
            for _ in range(n):
                layer_i[0] = (layer_i[0] + 1) % N_LAYERS
                fs = cache.state(layer_i[0])["end"] - C                  # overwrite the newest chunk in place
                qq, kk, vv = dev_sets[layer_i[0] % N_INPUT_SETS]
                cache.norm_rope_append_kv(layer_i[0], qq, kk, vv, gains, gains, 1e-6, fs, wl.grid_h, wl.grid_w,
                                          wl.rope_theta, q_roped)
        ms = median_ms(norm_append) / 20
        others["norm_rope_append"] = {"us": ms * 1e3, "gbs": append_bytes(wl) / ms / 1e6,
                                      "frac_of_copy_peak": append_bytes(wl) / ms / 1e6 / load_peaks()[0]["hbm_gbs"]}
        # the layer's QKV projection with the path's front end in its epilogue (d_model 1536)
        d_model = 1536
        xs = torch.randn(nq, d_model, device="cuda").bfloat16()
        wq = (torch.randn(3 * H * D, d_model, device="cuda") / d_model ** 0.5).bfloat16()
        bq = torch.randn(3 * H * D, device="cuda") * 0.1
        rs = torch.empty(nq, device="cuda")
        wsb = torch.empty(B.ll_qkv_proj_workspace_bytes(cache.h) + 256, dtype=torch.uint8, device="cuda")
        wsb = wsb[(-wsb.data_ptr()) % 256:]

        def proj(norm, n=10):
            for _ in range(n):
                layer_i[0] = (layer_i[0] + 1) % N_LAYERS
                fs = cache.state(layer_i[0])["end"] - C
                B.ll_qkv_proj_append(cache.h, layer_i[0], xs, wq, bq, gains if norm else None, gains if norm else None,
                                     1e-6, fs, C, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped, rs if norm else None,
                                     wsb if norm else None)
        gemm_flops = 2.0 * nq * d_model * 3 * H * D
        for norm in (False, True):
            ms = median_ms(lambda: proj(norm)) / 10
            others["qkv_proj_append" + ("_with_norm" if norm else "")] = {"us": ms * 1e3, "gemm_tflops": gemm_flops / ms / 1e9}
        cache.check_device()
        # the 8-bit cache: append that quantises on write, attention = expand to bf16 staging + the same kernel
        c8 = B.Cache(2, H, D, P, C, wl.sink_frames, wl.window_frames, device="cuda:%d" % local_rank, kv_format=B.LL_KV_E4M3)
        for l in range(2):
            c8.set_kv_scales(l, [6.0 / 448.0] * H, [6.0 / 448.0] * H)
            for chunk in range(n_fill):
                c8.rope_append_kv(l, q, k, v, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped)
        lay = [0]

        def app8(n=20):
            for _ in range(n):
                lay[0] ^= 1
                c8.rope_append_kv(lay[0], q, k, v, (n_fill - 1) * C, wl.grid_h, wl.grid_w, wl.rope_theta, q_roped)

        def att8():
            lay[0] ^= 1
            c8.sink_window_attn(lay[0], q_roped, (n_fill - 1) * C, out)
        ms_a = median_ms(app8) / 20
        ms_t = median_ms(att8)
        others["kv_e4m3"] = {"append_us": ms_a * 1e3, "attention_ms_incl_expansion": ms_t,
                             "attention_tflops": attn_flops(wl) / ms_t / 1e9,
                             "storage_bytes_30_layers": None, "bf16_storage_bytes_30_layers": None}
        if args.in_loop_seconds > 0:
            # the same call back to back for about a second: the figure under the power cap
            n8 = int(1e3 / ms_t) + 1
            a8, b8 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(n8 // 2):
                att8()
            a8.record(stream)
            for _ in range(n8 // 2):
                att8()
            b8.record(stream)
            torch.cuda.synchronize()
            ms_loop8 = a8.elapsed_time(b8) / (n8 // 2)
            others["kv_e4m3"]["attention_ms_in_a_one_second_loop"] = ms_loop8
            others["kv_e4m3"]["attention_tflops_in_the_loop"] = attn_flops(wl) / ms_loop8 / 1e9
        h8, h16 = B.ll_cache_create(30, H, D, P, C, wl.sink_frames, wl.window_frames), \
            B.ll_cache_create(30, H, D, P, C, wl.sink_frames, wl.window_frames)
        B.ll_cache_set_kv_format(h8, B.LL_KV_E4M3)
        others["kv_e4m3"]["storage_bytes_30_layers"] = B.ll_cache_storage_bytes(h8)
        others["kv_e4m3"]["bf16_storage_bytes_30_layers"] = B.ll_cache_storage_bytes(h16)
        B.ll_cache_destroy(h8)
        B.ll_cache_destroy(h16)
        c8.check_device()
        c8.close()
        n_prompt = 512
        pk = torch.randn(n_prompt, H, D, device="cuda").bfloat16()
        pv = torch.randn(n_prompt, H, D, device="cuda").bfloat16()
        ms_call = median_ms(lambda: cache.cross_attn(q, pk, pv, out))
        # the launch is shorter than a call's host time: ten calls in a captured graph give the device time
        cache.cross_attn(q, pk, pv, out)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(10):
                cache.cross_attn(q, pk, pv, out)
        ms = median_ms(graph.replay) / 10
        cache.check_device()
        # the same grid and width with 24 heads of 64: twice the exponentials per flop
        H64, D64 = 2 * H, D // 2
        c64 = B.Cache(2, H64, D64, P, C, wl.sink_frames, wl.window_frames, device="cuda:%d" % local_rank)
        q64 = torch.randn(nq, H64, D64, device="cuda").bfloat16()
        k64, v64 = torch.randn_like(q64), torch.randn_like(q64)
        qr64, out64 = torch.empty_like(q64), torch.empty_like(q64)
        for l in range(2):
            for chunk in range(n_fill):
                c64.rope_append_kv(l, q64, k64, v64, chunk * C, wl.grid_h, wl.grid_w, wl.rope_theta, qr64)

        def att64():
            lay[0] ^= 1
            c64.sink_window_attn(lay[0], qr64, (n_fill - 1) * C, out64)
        ms64 = median_ms(att64)
        c64.check_device()
        c64.close()
        others["head_dim_64_24_heads"] = {"ms": ms64, "tflops": attn_flops(wl) / ms64 / 1e9}
        others["cross_attn_512_keys"] = {"us": ms * 1e3, "tflops": 4.0 * nq * n_prompt * D * H / ms / 1e9,
                                         "us_one_call_between_events": ms_call * 1e3,
                                         "how": "ten launches in a captured CUDA graph, replayed"}
        cache.check_device()

    loop_vals = [in_loop["ms_total"], in_loop["attn_ms_per_launch_second_half"]] if in_loop else [0.0, 0.0]
    total_ms, e2e_ms, attn_ms, append_ms, append_b2b_ms, loop_total_ms, loop_attn_ms = reduce_max(
        [total_ms, e2e_ms, attn_ms, append_ms, append_b2b_ms] + loop_vals, dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    flops_step = attn_flops(wl)
    peaks, peak_kind = load_peaks()
    traffic = load_traffic()
    value = whole_job_tflops(world, args.steps, flops_step, total_ms)
    e2e_value = whole_job_tflops(world, args.steps, flops_step, e2e_ms)
    attn_tflops = flops_step / (attn_ms * 1e-3) / 1e12
    append_gbs = append_bytes(wl) / (append_b2b_ms * 1e-3) / 1e9
    if in_loop:
        n_loop = in_loop["steps"]
        in_loop.update({
            "ms_total": loop_total_ms, "ms_per_step": loop_total_ms / n_loop,
            "value_tflops": whole_job_tflops(world, n_loop, flops_step, loop_total_ms),
            "attn_ms_per_launch_second_half": loop_attn_ms,
            "attn_tflops": flops_step / (loop_attn_ms * 1e-3) / 1e12,
            "attn_frac_of_burst_peak": flops_step / (loop_attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "attn_frac_of_sustained_peak": flops_step / (loop_attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
            "note": "at least %.1f s of back-to-back steps; sw_power_cap in its clock record is expected and kept; "
                    "the --steps region above is a burst when it is short" % args.in_loop_seconds})
    ms_per_step = total_ms / args.steps
    in_bytes = 3 * nq * H * D * 2
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        tf, cores, what, _ = oracle_sample(15.0)
        cpu = {"value": tf, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": what}
    line = {
        "metric": "sink_window_attn_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "heads": H, "head_dim": D, "tokens_per_frame": P, "chunk_frames": C,
                   "sink_frames": wl.sink_frames, "window_frames": wl.window_frames, "query_rows": nq,
                   "keys": steady_keys(wl), "parallelism": "replicas x%d" % world,
                   "l2": "inputs larger than L2: %d layer caches (115 MB each) and %d q/k/v sets rotate"
                         % (N_LAYERS, N_INPUT_SETS)},
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": in_bytes,
                "d2h_bytes_per_step": nq * H * D * 2, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "attn_sm100_kernel<128>", "achieved": attn_tflops,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": attn_tflops / peaks["bf16_tflops"],
                     "peak_kind": "of %s (burst bf16 GEMM)" % peak_kind, "ms_per_launch": attn_ms,
                     "frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": attn_tflops / 2250.0,
                     "traffic": traffic.get("attn_sm100_kernel")},
        "roofline_append": {"bound": "hbm", "kernel": "rope_append_kernel<128>", "achieved": append_gbs,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": append_gbs / peaks["hbm_gbs"],
                            "peak_kind": "of %s (copy)" % peak_kind, "ms_per_launch": append_b2b_ms,
                            "how": "%d launches back to back on rotating layers between two events" % n_app,
                            "ms_of_a_step_outside_the_attention_events": append_ms,
                            "traffic": traffic.get("rope_append_kernel"),
                            "traffic_note": "DRAM bytes under the profiler are below the 86.3 MB the kernel moves: "
                                            "the cache rows it wrote are still in L2 when it ends"},
        "cpu_baseline": cpu,
        "extra": {"in_loop": in_loop,
                  "latent_frames_per_s_30_layers_5_passes": C / (150 * ms_per_step * 1e-3),
                  "latent_frames_per_s_30_layers_4_passes": C / (120 * ms_per_step * 1e-3),
                  "recache_ms_per_layer": recache_ms,
                  "recache_tflops": 9 * attn_flops(wl) / 4 / (recache_ms * 1e-3) / 1e12,
                  "other_entry_points": others,
                  "paper_context": "20.7 video FPS (about 5.2 latent frames/s) for the whole 1.3B model on one H100"},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--in-loop-seconds", type=float, default=2.0,
                    help="length of the extra power-limited leg reported as extra.in_loop (0 = skip)")
    ap.add_argument("--dry-run", action="store_true", help="multi-rank plumbing only, on CPU (gloo); measures nothing")
    args = ap.parse_args()
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    elif args.dry_run:
        run_dry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
