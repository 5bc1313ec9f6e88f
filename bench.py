"""Benchmark of the residual-binary linear layer on B200.

Workload (``config.workload``): the seven projections of a Llama-2-7B-shaped decoder layer
(q,k,v,o 4096->4096; gate,up 4096->11008; down 11008->4096) as K=2 residual-binary layers,
batch 1, run back to back.  One *step* is one such decoder layer = seven ``rabit_linear``
calls.  To keep the weights cold in HBM the run rotates over ``--copies`` distinct decoder
layers (default 32, i.e. the 224 projections of a 7B-shaped stack, 1.6 GB packed, far
above the 126 MB L2), so every step streams weights that were evicted long ago.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl rabit|reference]

For N > 1 launch under ``torch.distributed.run``; every rank holds its own replica of the
workload (the path has no exchange step), timing is the max over ranks.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "batch-1 residual-binary GEMV us/layer"
UNIT = "us/layer"
WORKLOAD = "llama2-7b decoder layer: 7 residual-binary projections, K=2, batch 1, back to back"
K_PATHS = 2


def layer_bytes(M: int, N: int, batch: int, K: int = K_PATHS) -> int:
    """Algorithmic bytes of one call: sign bits + fp16 scales + x in + y out."""
    return K * M * N // 8 + 2 * K * (M + N) + 2 * batch * (M + N)


# ---------------------------------------------------------------------------------------
# clocks sampler (nvidia-smi in the background, as the profiling recipe prescribes)
# ---------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.samples = []   # (t, sm_mhz, max_mhz, {reason: bool})
        self.proc = None
        self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(gpu_index), "-lms", str(period_ms)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm, mx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
            reasons = {n: parts[5 + i].lower().startswith("active") for i, n in enumerate(names)}
            self.samples.append((time.time(), sm, mx, reasons))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float) -> dict:
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        reasons = sorted({n for s in inside for n, on in s[3].items() if on})
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside)}


# ---------------------------------------------------------------------------------------
# multi-rank bookkeeping (replicas only: the path has no exchange step)
# ---------------------------------------------------------------------------------------
def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: what a job that waits for every replica sees."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_layer(ms_per_step: float, layers_per_step: int, world: int) -> float:
    """Time-like aggregate over N replicas: every rank finishes `layers_per_step` layers per step, so the
    job finishes world * layers_per_step layers in the slowest rank's step time."""
    return ms_per_step * 1e3 / (layers_per_step * world)


# ---------------------------------------------------------------------------------------
# workload
# ---------------------------------------------------------------------------------------
def build_workload(copies: int, batch: int, device: str, tokens: int, seed_cfg: int = 1):
    import torch
    import paper_2602_05367_b200 as rabit
    from synth import llama2_7b_layer_shapes, make_layer, make_x

    shapes = llama2_7b_layer_shapes()
    layers = []            # [copy][proj] -> RabitLayer
    for c in range(copies):
        row = []
        for p, sh in enumerate(shapes):
            L = make_layer(sh.M, sh.N, K_PATHS, key=(seed_cfg, c, p))
            row.append(rabit.rabit_pack(L.planes, L.g, L.h, device=device))
        layers.append(row)
    widths = sorted({sh.N for sh in shapes})
    xs_host = {n: np.stack([make_x(batch, n, key=(seed_cfg, 10_000 + t)) for t in range(tokens)]) for n in widths}
    xs = {n: torch.from_numpy(a).to(device) for n, a in xs_host.items()}            # [tokens][batch][N]
    ys = [torch.zeros((batch, sh.M), dtype=torch.float16, device=device) for sh in shapes]
    return shapes, layers, xs, xs_host, ys


# Projections of a decoder layer that read the same activations: q|k|v and gate|up go through
# rabit_linear_group (one launch each), o and down through rabit_linear.
GROUPS = [[0, 1, 2], [3], [4, 5], [6]]


def run_step(rabit, shapes, layer_row, xs, ys, token: int, grouped: bool = True):
    if not grouped:
        for p, sh in enumerate(shapes):
            rabit.rabit_linear(layer_row[p], xs[sh.N][token], ys[p])
        return
    for grp in GROUPS:
        if len(grp) == 1:
            p = grp[0]
            rabit.rabit_linear(layer_row[p], xs[shapes[p].N][token], ys[p])
        else:
            rabit.rabit_linear_group([layer_row[p] for p in grp], [xs[shapes[p].N][token] for p in grp], [ys[p] for p in grp])


# ---------------------------------------------------------------------------------------
# timing helpers
# ---------------------------------------------------------------------------------------
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", 1590.0)),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 1400.0)), "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def recorded_traffic(key: str):
    """DRAM bytes per step from the ncu capture recorded in profiles/gemv_lut_traffic.json, or None when no capture of
    this workload is on record there (the file names the command and the kernel source it was taken with)."""
    path = os.path.join(ROOT, "profiles", "gemv_lut_traffic.json")
    try:
        rec = json.load(open(path))
    except (OSError, ValueError):
        return None
    entry = rec.get(key)
    return None if entry is None else entry.get("dram_bytes_per_step")


def time_replays(stream, graphs, repeats: int, warm: int = 1):
    """Milliseconds of `repeats` timed passes over the list of CUDA graphs (each pass replays every graph once, in
    order), CUDA events on the launching stream; `warm` untimed passes first."""
    import torch
    out = []
    with torch.cuda.stream(stream):
        for _ in range(warm):
            for g in graphs:
                g.replay()
    stream.synchronize()
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for g in graphs:
                g.replay()
            e1.record(stream)
        stream.synchronize()
        out.append(e0.elapsed_time(e1))
    return out


def capture_graph(stream, fn):
    import torch
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        fn()
    return g


def measure_stream_read(device, stream) -> float:
    """Read-only streaming bandwidth in GB/s: 128-bit loads over 2 GiB, best of 5 (the library's own probe kernel)."""
    import ctypes
    import torch
    from paper_2602_05367_b200 import binding
    lib = binding.raw_lib()
    n = 2 << 30
    buf = torch.empty(n, dtype=torch.uint8, device=device)
    buf.fill_(3)
    best = None
    for _ in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            rc = lib.rabit_selftest_stream_read(ctypes.c_void_p(buf.data_ptr()), n, None, ctypes.c_void_p(stream.cuda_stream))
            e1.record(stream)
        stream.synchronize()
        assert rc == 0
        ms = e0.elapsed_time(e1)
        best = ms if best is None or ms < best else best
    del buf
    torch.cuda.empty_cache()
    return n / (best * 1e-3) / 1e9


# ---------------------------------------------------------------------------------------
# the library arm
# ---------------------------------------------------------------------------------------
def bench_rabit(args) -> dict:
    import torch
    import paper_2602_05367_b200 as rabit

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device(device))
        dist = dist_mod

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    copies, batch, tokens = args.copies, args.batch, 4
    shapes, layers, xs, xs_host, ys = build_workload(copies, batch, device, tokens)
    step_bytes = sum(layer_bytes(sh.M, sh.N, batch) for sh in shapes)
    n_proj = len(shapes)
    stream = torch.cuda.Stream(device)
    grouped = not args.no_group
    launches_per_step = len(GROUPS) if grouped else n_proj
    peaks = load_peaks()

    def steps_fn(first: int, count: int):
        """Steps first .. first+count-1; step s runs decoder-layer copy s % copies on the current token's activations (a
        token's hidden state is re-read by every layer of the stack, so it is warm in L2; the weights are not)."""
        def fn():
            for s in range(first, first + count):
                run_step(rabit, shapes, layers[s % copies], xs, ys, 0, grouped)
        return fn

    with torch.cuda.stream(stream):
        steps_fn(0, copies)()                        # first-call set-up of every kernel variant, outside any capture
    stream.synchronize()

    # The timed region is K steps as whole CUDA graphs, whatever K is: full cycles over the copies replay one graph of
    # `copies` steps, the remainder is one graph of its own, so 20 steps and 32000 steps time the same launch pattern.
    def graphs_for(first: int, count: int):
        out = []
        full, rem = divmod(count, copies)
        if full:
            cyc = capture_graph(stream, steps_fn(first, copies))
            out += [cyc] * full
        if rem:
            out.append(capture_graph(stream, steps_fn(first + full * copies, rem)))
        return out

    warm_graphs = graphs_for(0, args.warmup)
    timed_graphs = graphs_for(args.warmup, args.steps)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    time_replays(stream, warm_graphs, repeats=0, warm=1)
    barrier()
    t_wall0 = time.time()
    times = time_replays(stream, timed_graphs, repeats=args.repeats, warm=0)
    barrier()
    t_wall1 = time.time()
    times = [max_over_ranks(t, dist, device) for t in times]
    ms = float(np.median(times))
    clocks = sampler.summary(t_wall0, t_wall1) if sampler else None
    if sampler and clocks["samples"] < 3:
        # the timed region was shorter than the sampling period: repeat the same work, untimed,
        # for about a second under the sampler and report the clocks seen there
        reps = max(1, int(1.0 / max(ms * 1e-3, 1e-4)))
        t0 = time.time()
        time_replays(stream, timed_graphs, repeats=0, warm=reps)
        clocks = sampler.summary(t0, time.time())
        clocks["note"] = "sampled over an untimed repeat of the timed region (region shorter than the sampler period)"
    if sampler:
        sampler.stop()

    ms_per_step = ms / args.steps
    gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    gbs_best = step_bytes / (min(times) / args.steps * 1e-3) / 1e9

    # ---- warm-L2 figure (labelled; the paper's own latencies are warm-cache): one decoder layer, 51 MB, replayed in place
    warm_l2 = None
    if rank == 0 and world == 1 and not args.no_extras:
        g1 = capture_graph(stream, steps_fn(0, 1))
        t = time_replays(stream, [g1] * 200, repeats=5, warm=2)
        warm_l2 = {"us_per_layer": float(np.median(t)) / 200 * 1e3 / n_proj, "gbs_equivalent": step_bytes / (float(np.median(t)) / 200 * 1e-3) / 1e9,
                   "note": "the same step replayed on ONE decoder layer: its 51 MB stay in the 126 MB L2, no HBM traffic"}

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if rank == 0 or dist is not None:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pin_x = {n: torch.from_numpy(a).pin_memory() for n, a in xs_host.items()}
        pin_y = [torch.empty((batch, sh.M), dtype=torch.float16).pin_memory() for sh in shapes]
        e2e_steps = max(1, min(args.steps, args.e2e_steps))

        plans = None
        if grouped:                                   # arguments checked and marshalled once per (decoder layer, group)
            plans = [[rabit.PreparedGroupHost([layers[c][p] for p in grp], [pin_x[shapes[p].N][c % tokens] for p in grp],
                                              [pin_y[p] for p in grp]) for grp in GROUPS] for c in range(copies)]

        def e2e_step(s):
            c = s % copies
            with torch.cuda.stream(stream):
                if grouped:
                    for plan in plans[c]:
                        plan(stream.cuda_stream)
                else:
                    for p, sh in enumerate(shapes):
                        rabit.rabit_linear_host(layers[c][p], pin_x[sh.N][c % tokens], pin_y[p], stream=stream.cuda_stream)
                stream.synchronize()                  # the caller reads y on the host after every step
        for s in range(min(3 * copies, 100)):
            e2e_step(s)
        barrier()
        with torch.cuda.stream(stream):
            ev0.record(stream)
        for s in range(e2e_steps):
            e2e_step(s)
        with torch.cuda.stream(stream):
            ev1.record(stream)
        barrier()
        e_ms = max_over_ranks(ev0.elapsed_time(ev1), dist, device)
        e2e = {"value": whole_job_us_per_layer(e_ms / e2e_steps, n_proj, world), "unit": UNIT,
               "h2d_bytes_per_step": int(sum(2 * batch * shapes[grp[0]].N for grp in GROUPS) if grouped else sum(2 * batch * sh.N for sh in shapes)),
               "d2h_bytes_per_step": int(sum(2 * batch * sh.M for sh in shapes)),
               "steps": e2e_steps, "note": ("rabit_linear_group_host (prepared calls) per group of projections (a shared input is copied once)" if grouped else
                        "rabit_linear_host per projection") + ": pinned host x -> device stage by copy, kernel, y stored by the kernel straight into pinned (mapped) host memory, host synchronises after every step"}

    read_peak = measure_stream_read(device, stream) if (rank == 0 and not args.no_extras) else None
    peak = peaks["hbm_gbs"]
    traffic_step = recorded_traffic("decoder7b_grouped_batch1") if (grouped and batch == 1) else None
    result = {
        "metric": METRIC, "value": whole_job_us_per_layer(ms_per_step, n_proj, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (table look-up sums in fp32 registers, 64-bit fixed-point reduction across CTAs, fp16 in/out)",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "copies": copies, "batch": batch, "K": K_PATHS,
                   "packed_bytes_total": int(step_bytes * copies),
                   "l2": "inputs larger than L2: rotation over %d distinct decoder layers (%.0f MB of weights); the activations of the "
                         "current token are re-read by every layer and stay warm, as in a decoder" % (copies, step_bytes * copies / 1e6),
                   "launch": "CUDA graph replay: the timed region is whole graphs (one graph per cycle over the copies, one for the remainder)",
                   "launches_per_step": launches_per_step,
                   "grouping": "q|k|v and gate|up (projections that share their input) each go through one rabit_linear_group launch; "
                               "o and down through rabit_linear" if grouped else "one rabit_linear launch per projection",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "repeats": {"n": len(times), "ms_median": ms, "ms_min": min(times), "ms_max": max(times),
                    "us_per_layer_median": ms_per_step * 1e3 / n_proj, "us_per_layer_min": min(times) / args.steps * 1e3 / n_proj},
        "achieved_hbm_gbs": gbs * world,
        "tokens_per_s_32_layer_stack_extrapolated": world * 1.0 / (32 * ms_per_step * 1e-3),
        "gpu_launches": args.steps * launches_per_step * max(1, len(times)),
        "clocks": clocks,
        "e2e": e2e,
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                     "traffic": (traffic_step / launches_per_step) if traffic_step else None,
                     "algorithmic_bytes_per_launch": step_bytes / launches_per_step,
                     "peak_source": peaks["source"] + " hbm_gbs (copy bandwidth, read+write bytes)",
                     "frac_best_repeat": gbs_best / peak,
                     "other_denominators": {"nominal_8000_gbs": gbs / 8000.0,
                                            "read_only_stream_gbs": read_peak, "frac_of_read_only_stream": (gbs / read_peak) if read_peak else None},
                     "note": "per launch of rabit_gemv_lut_kernel, averaged over the launches of a step: algorithmic bytes of the "
                             "step / device time of the step (launch gaps included); traffic = ncu dram bytes of the same launches"},
    }
    if warm_l2:
        result["warm_l2"] = warm_l2
    if rank == 0 and world == 1 and not args.no_extras:
        result["extras"] = bench_extras(args, rabit, device, stream, shapes, layers, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(sample_projections=n_proj, variants=True)
    for row in layers:
        for L in row:
            L.free()
    if dist is not None:
        dist.destroy_process_group()
    return result if rank == 0 else None


def bench_extras(args, rabit, device, stream, shapes, layers, peaks) -> dict:
    """Compact measurements of the other benchmark configurations, each with its own roofline fraction (same protocol:
    cold weights by rotation over distinct copies, graph replay, CUDA events, median of 5)."""
    import torch
    from synth import make_layer, make_x
    out = {}
    hbm = peaks["hbm_gbs"]

    def timed_case(lys, x, y, launches_note=None):
        def fn():
            for L in lys:
                rabit.rabit_linear(L, x, y)
        with torch.cuda.stream(stream):
            fn()
        stream.synchronize()
        g = capture_graph(stream, fn)
        reps = max(1, int(2e-3 / (len(lys) * 20e-6)))
        t = time_replays(stream, [g] * reps, repeats=5, warm=1)
        return float(np.median(t)) * 1e3 / (reps * len(lys))

    def make_copies(M, N, K, n, cfg):
        res = []
        for c in range(n):
            L = make_layer(M, N, K, key=(cfg, c, M, N, K))
            res.append(rabit.rabit_pack(L.planes, L.g, L.h, device=device))
        return res

    def n_copies(M, N, K):
        return max(2, min(32, int(4 * 126e6 / layer_bytes(M, N, 1, K)) + 1))

    def hbm_case(M, N, K, batch, us):
        nb = layer_bytes(M, N, batch, K)
        return {"M": M, "N": N, "K": K, "batch": batch, "us_per_layer": us, "gbs": nb / us / 1e3, "frac": nb / us / 1e3 / hbm}

    # config 0: the 4096 x 4096 layer alone (the q projections of the rotating decoder layers)
    x4096 = torch.from_numpy(make_x(1, 4096, key=(0, 0))).to(device)
    y = torch.zeros((1, 4096), dtype=torch.float16, device=device)
    us = timed_case([row[0] for row in layers], x4096, y)
    out["config0_4096x4096_batch1"] = hbm_case(4096, 4096, K_PATHS, 1, us)

    # config 2 as stated: the whole stack (copies x 7 projections), 256 sequential tokens, one token = one CUDA graph
    if len(layers) >= 32:
        n_tok = 256
        xs_all = {n: torch.from_numpy(np.stack([make_x(1, n, key=(2, 10_000 + t))[0] for t in range(n_tok)])).to(device) for n in (4096, 11008)}
        x_cur = {n: torch.zeros((1, n), dtype=torch.float16, device=device) for n in xs_all}
        idx = torch.zeros(1, dtype=torch.int64, device=device)
        ys2 = [torch.zeros((1, sh.M), dtype=torch.float16, device=device) for sh in shapes]

        def token_fn():
            for n in xs_all:                                   # the token's activations: device-side index, advanced inside the graph
                torch.index_select(xs_all[n], 0, idx, out=x_cur[n])
            idx.add_(1).remainder_(n_tok)
            for row in layers:
                for grp in GROUPS:
                    if len(grp) == 1:
                        rabit.rabit_linear(row[grp[0]], x_cur[shapes[grp[0]].N], ys2[grp[0]])
                    else:
                        rabit.rabit_linear_group([row[p] for p in grp], [x_cur[shapes[p].N] for p in grp], [ys2[p] for p in grp])
        with torch.cuda.stream(stream):
            token_fn()
        stream.synchronize()
        idx.zero_()
        g = capture_graph(stream, token_fn)
        t = time_replays(stream, [g] * n_tok, repeats=3, warm=0)
        sec = float(np.median(t)) * 1e-3
        stack_bytes = len(layers) * sum(layer_bytes(sh.M, sh.N, 1) for sh in shapes)
        out["config2_stack_256_tokens"] = {"layers": len(layers) * len(shapes), "tokens": n_tok, "tokens_per_s": n_tok / sec,
                                            "ms_per_token": sec / n_tok * 1e3, "gbs": stack_bytes * n_tok / sec / 1e9,
                                            "frac": stack_bytes * n_tok / sec / 1e9 / hbm,
                                            "note": "one token = one CUDA graph of %d launches (plus three tiny launches that select the token's "
                                                    "activations by a device-side index); tokens/s = 256 / elapsed" % (len(layers) * len(GROUPS))}

    # config 3 / 4 samples at batch 1, batches 1, 2, 4, 8 and 16 on the 8B shapes, the batch-512 GEMM, and K = 1 / 3 at 7B shapes
    extra_hbm = []
    for (M, N) in [(14336, 4096), (28672, 8192)]:
        lys = make_copies(M, N, K_PATHS, n_copies(M, N, K_PATHS), 4)
        x = torch.from_numpy(make_x(1, N, key=(4, 1, N))).to(device)
        y = torch.zeros((1, M), dtype=torch.float16, device=device)
        extra_hbm.append(hbm_case(M, N, K_PATHS, 1, timed_case(lys, x, y)))
        if (M, N) == (28672, 8192):
            xb = torch.from_numpy(make_x(512, N, key=(4, 512, N))).to(device)
            yb = torch.zeros((512, M), dtype=torch.float16, device=device)
            usb = timed_case(lys, xb, yb)
            tf = 2.0 * 512 * M * N * K_PATHS / usb / 1e6
            out["gemm_28672x8192_batch512"] = {"us_per_layer": usb, "tflops": tf, "bound": "tensor", "peak": peaks["bf16_tflops_sustained"],
                                               "frac": tf / peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " bf16_tflops_sustained"}
        for L in lys:
            L.free()
        del lys
    out["batch1_large_layers"] = extra_hbm
    b16 = []
    for (M, N) in [(4096, 4096), (1024, 4096), (14336, 4096), (4096, 14336)]:
        lys = make_copies(M, N, K_PATHS, n_copies(M, N, K_PATHS), 3)
        for batch in (1, 2, 4, 8, 16):
            x = torch.from_numpy(make_x(batch, N, key=(3, batch, N))).to(device)
            y = torch.zeros((batch, M), dtype=torch.float16, device=device)
            b16.append(hbm_case(M, N, K_PATHS, batch, timed_case(lys, x, y)))
        for L in lys:
            L.free()
        del lys
    out["llama3_8b_shapes_batch_1_to_16"] = b16
    kk = []
    for K in (1, 3):
        for (M, N) in [(4096, 4096), (11008, 4096)]:
            lys = make_copies(M, N, K, n_copies(M, N, K), 5)
            x = torch.from_numpy(make_x(1, N, key=(5, 1, N))).to(device)
            y = torch.zeros((1, M), dtype=torch.float16, device=device)
            kk.append(hbm_case(M, N, K, 1, timed_case(lys, x, y)))
            for L in lys:
                L.free()
            del lys
    out["paths_1_and_3_batch1"] = kk
    torch.cuda.empty_cache()
    return out


# ---------------------------------------------------------------------------------------
# the oracle, timed as it stands on the host cores
# ---------------------------------------------------------------------------------------
def cpu_baseline(sample_projections: int = 7, repeats: int = 1, variants: bool = False) -> dict:
    from oracle import rabit_oracle as orc
    from synth import llama2_7b_layer_shapes, make_layer, make_x

    shapes = llama2_7b_layer_shapes()[:sample_projections]
    inputs = [(make_layer(sh.M, sh.N, K_PATHS, key=(1, 0, p)), make_x(1, sh.N, key=(1, 10_000))) for p, sh in enumerate(shapes)]
    t0 = time.perf_counter()
    for _ in range(repeats):
        for L, x in inputs:
            orc.linear(L.planes, L.g, L.h, x)
    dt = (time.perf_counter() - t0) / repeats
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    res = {"value": dt * 1e6 / len(shapes), "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "decoder-layer copy 0, its %d projections once each, batch 1 (float64: unpack signs, dense W, product)" % len(shapes)}
    if variants:
        # the same oracle restricted to one thread, and its last step alone (float64 product with W already formed)
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                t0 = time.perf_counter()
                for L, x in inputs[:2]:
                    orc.linear(L.planes, L.g, L.h, x)
                res["one_thread_us_per_layer"] = (time.perf_counter() - t0) * 1e6 / 2
                res["one_thread_sample"] = "the first two projections (4096 x 4096), BLAS limited to one thread"
        except ImportError:
            res["one_thread_us_per_layer"] = None
        L, x = inputs[0]
        W = orc.dense_weight(L.planes, L.g, L.h)
        x64 = x.astype(np.float64)
        t0 = time.perf_counter()
        for _ in range(5):
            (x64 @ W.T)
        res["w_preformed_us_per_layer"] = (time.perf_counter() - t0) * 1e6 / 5
        res["w_preformed_sample"] = "4096 x 4096: float64 product alone, dense W formed beforehand by the oracle (not timed)"
    return res


def bench_cases(args) -> dict:
    """Extra workloads (not the default line): one (shape, batch) case at a time, rotating over enough
    distinct copies of the layer to exceed L2, CUDA-graph replay, CUDA-event timing.
      gemm70b : 70B-shaped layers at batch 512 (tensor-core GEMM), roofline = measured bf16 TFLOP/s
      gemm7b  : the three distinct 7B-shaped layers at batch 128, 512 and 2048 (prefill sizes; split and whole-wave launches)
      gemv70b : the same layers at batch 1 (HBM roofline)
      sweep8b : Llama-3-8B shapes at batch 1,2,4,8,16 (HBM roofline per batch)"""
    import torch
    import paper_2602_05367_b200 as rabit
    from synth import llama3_8b_layer_shapes, llama_70b_layer_shapes, make_layer, make_x

    device = "cuda:0"
    torch.cuda.set_device(0)
    if args.workload == "sweep8b":
        seen, shapes = set(), []
        for sh in llama3_8b_layer_shapes():
            if (sh.M, sh.N) not in seen:
                seen.add((sh.M, sh.N)); shapes.append(sh)
        batches, cfg = [1, 2, 4, 8, 16], 3
    elif args.workload == "gemm7b":
        from synth import llama2_7b_layer_shapes
        seen, shapes = set(), []
        for sh in llama2_7b_layer_shapes():
            if (sh.M, sh.N) not in seen:
                seen.add((sh.M, sh.N)); shapes.append(sh)
        batches, cfg = [128, 512, 2048], 1
    else:
        shapes, cfg = llama_70b_layer_shapes(), 4
        batches = [512] if args.workload == "gemm70b" else [1]
    if args.only_shape:
        shapes = [sh for sh in shapes if "%dx%d" % (sh.M, sh.N) == args.only_shape]
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    tc_peak = float(peaks.get("bf16_tflops_sustained", 1400.0))
    stream = torch.cuda.Stream(device)
    cases = []
    sampler = ClockSampler(0)
    t_start = time.time()
    for sh in shapes:
        per_layer = layer_bytes(sh.M, sh.N, 1)
        copies = max(2, min(args.copies, int(4 * 126e6 / per_layer) + 1))
        layers = []
        for c in range(copies):
            L = make_layer(sh.M, sh.N, K_PATHS, key=(cfg, c, sh.M, sh.N))
            layers.append(rabit.rabit_pack(L.planes, L.g, L.h, device=device))
        for batch in batches:
            x = torch.from_numpy(make_x(batch, sh.N, key=(cfg, 10_000, batch))).to(device)
            y = torch.zeros((batch, sh.M), dtype=torch.float16, device=device)
            with torch.cuda.stream(stream):
                for L in layers:
                    rabit.rabit_linear(L, x, y)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for L in layers:
                    rabit.rabit_linear(L, x, y)
            reps = max(3, args.steps // copies) if args.steps < 32000 else max(3, int(0.3 / (copies * 30e-6)))
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                for _ in range(3):
                    g.replay()
                ev0.record(stream)
                for _ in range(reps):
                    g.replay()
                ev1.record(stream)
            stream.synchronize()
            us = ev0.elapsed_time(ev1) * 1e3 / (reps * copies)
            nbytes = layer_bytes(sh.M, sh.N, batch)
            flops = 2.0 * batch * sh.M * sh.N * K_PATHS
            case = {"M": sh.M, "N": sh.N, "batch": batch, "copies": copies, "us_per_layer": us,
                    "gbs": nbytes / us / 1e3, "tflops": flops / us / 1e6}
            if batch > 16:
                case["roofline"] = {"bound": "tensor", "achieved": case["tflops"], "peak": tc_peak, "unit": "TFLOP/s",
                                    "frac": case["tflops"] / tc_peak}
            else:
                case["roofline"] = {"bound": "hbm", "achieved": case["gbs"], "peak": hbm_peak, "unit": "GB/s",
                                    "frac": case["gbs"] / hbm_peak}
            if batch > 16:
                # the same case on the dequantised-tile GEMM (variant 4: one contraction of fp16 weights instead of one per
                # path); tflops counts the layer's algorithmic flops for both, so the two compare by time
                for L in layers:
                    L.set_variant(4)
                with torch.cuda.stream(stream):
                    for L in layers:
                        rabit.rabit_linear(L, x, y)
                stream.synchronize()
                g4 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g4, stream=stream):
                    for L in layers:
                        rabit.rabit_linear(L, x, y)
                with torch.cuda.stream(stream):
                    for _ in range(3):
                        g4.replay()
                    ev0.record(stream)
                    for _ in range(reps):
                        g4.replay()
                    ev1.record(stream)
                stream.synchronize()
                us4 = ev0.elapsed_time(ev1) * 1e3 / (reps * copies)
                case["dequantised_tile_variant"] = {"us_per_layer": us4, "tflops_algorithmic": flops / us4 / 1e6,
                                                    "tensor_flops_executed_tflops": flops / K_PATHS / us4 / 1e6,
                                                    "frac_of_peak_executed": flops / K_PATHS / us4 / 1e6 / tc_peak}
                for L in layers:
                    L.set_variant(0)
                del g4
            cases.append(case)
            del g
        for L in layers:
            L.free()
        del layers
        torch.cuda.empty_cache()
    clocks = sampler.summary(t_start, time.time())
    sampler.stop()
    head = max(cases, key=lambda c: c["M"] * c["N"] * c["batch"])
    gemm = args.workload in ("gemm70b", "gemm7b")
    return {"metric": ("batch-512 residual-binary GEMM TFLOP/s" if args.workload == "gemm70b" else "residual-binary GEMM TFLOP/s (largest case)") if gemm else METRIC,
            "value": head["tflops"] if gemm else head["us_per_layer"], "unit": "TFLOP/s" if gemm else UNIT,
            "n_gpus": 1, "steps": args.steps, "warmup": 3, "ms_per_step": head["us_per_layer"] / 1e3,
            "higher_is_better": gemm, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 tensor-core products, fp32 accumulate" if gemm else "fp32 table sums (batch 1-2), f16 tensor-core products with fp32 accumulate (batch 3-16); 64-bit fixed-point cross-CTA sums",
            "data": "synthetic", "config": {"workload": args.workload, "K": K_PATHS,
                                            "l2": "rotation over distinct copies of each layer, > 4 x L2 in total where the layer is small"},
            "cases": cases, "roofline": head["roofline"], "clocks": clocks,
            "gpu_launches": sum(c["copies"] for c in cases)}


def bench_derive(args) -> dict:
    """Extra workload: on-device derivation of the sign planes fused with packing (rabit_derive_pack) on the
    7B-shaped weights; streams W (fp32) once, so the bound is HBM: 4 bytes in + K/8 bytes out per weight."""
    import torch
    import paper_2602_05367_b200 as rabit
    from synth import llama2_7b_layer_shapes

    torch.cuda.set_device(0)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    cases = []
    for sh in [s for i, s in enumerate(llama2_7b_layer_shapes()) if i in (0, 4, 6)]:
        gen = torch.Generator(device="cuda"); gen.manual_seed(sh.M * 31 + sh.N)
        Ws = [torch.randn((sh.M, sh.N), generator=gen, device="cuda", dtype=torch.float32) * 0.02 for _ in range(3)]   # 3 copies > L2
        rng = np.random.default_rng(sh.M + sh.N)
        h = rng.uniform(0.5, 1.5, (K_PATHS, sh.N)).astype(np.float16)
        g = np.stack([rng.uniform(0.012, 0.02, sh.M), rng.uniform(0.005, 0.009, sh.M)]).astype(np.float16)
        for W in Ws:
            rabit.rabit_derive_pack(W, g, h).free()
        reps = 4
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        # one call at a time, CUDA events around it (includes the upload of header and scales)
        bufs = [torch.empty(rabit.packed_bytes(K_PATHS, sh.M, sh.N), dtype=torch.uint8, device="cuda") for _ in Ws]
        from paper_2602_05367_b200 import binding
        import ctypes
        lib, vp = binding.raw_lib(), ctypes.c_void_p
        g16, h16 = g.view(np.uint16), h.view(np.uint16)
        st = torch.cuda.current_stream().cuda_stream
        handles = []
        ev0.record()
        for r in range(reps):
            for W, buf in zip(Ws, bufs):
                out = vp()
                rc = lib.rabit_derive_pack(vp(W.data_ptr()), g16.ctypes.data, h16.ctypes.data, K_PATHS, sh.M, sh.N,
                                           vp(buf.data_ptr()), buf.numel(), vp(st), ctypes.byref(out))
                assert rc == 0, rabit.last_error()
                handles.append(out)
        ev1.record(); torch.cuda.synchronize()
        for hnd in handles:
            lib.rabit_free(hnd)
        us = ev0.elapsed_time(ev1) * 1e3 / (reps * len(Ws))
        nbytes = 4 * sh.M * sh.N + K_PATHS * sh.M * sh.N // 8 + 2 * K_PATHS * (sh.M + sh.N)
        cases.append({"M": sh.M, "N": sh.N, "us": us, "gbs": nbytes / us / 1e3,
                      "roofline": {"bound": "hbm", "achieved": nbytes / us / 1e3, "peak": hbm_peak, "unit": "GB/s", "frac": nbytes / us / 1e3 / hbm_peak},
                      "note": "back-to-back asynchronous calls through the C ABI, CUDA events around all of them: includes the "
                              "upload of the scales, the second kernel (look-up blocks, scratch fills, header) and the fill of the accumulate words"})
        del Ws
        torch.cuda.empty_cache()
    head = max(cases, key=lambda c: c["M"] * c["N"])
    return {"metric": "sign-plane derivation + packing GB/s", "value": head["gbs"], "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
            "warmup": 3, "ms_per_step": head["us"] / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": {"workload": "derive7b", "K": K_PATHS}, "cases": cases,
            "roofline": head["roofline"], "gpu_launches": len(cases) * 12}


def bench_trace(args) -> dict:
    """Extra workload: where the time of a decoder-layer step goes, from the phase stamps of a library built with
    -DRABIT_TRACE (python paper_2602_05367_b200/build.py --trace; run with RABIT_LIBRARY=.../librabit_trace.so).
    Three decoder layers (more than L2), one CUDA graph that walks them once, replayed; the stamps of the last
    replay are reported per launch as microseconds after the entry of the cycle's first CTA (median over the CTAs of a
    launch, and the latest CTA for the end stamps)."""
    import ctypes
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding

    torch.cuda.set_device(0)
    device = "cuda:0"
    copies = 3
    shapes, layers, xs, xs_host, ys = build_workload(copies, 1, device, 16)
    lib = binding.raw_lib()
    stream = torch.cuda.Stream(device)
    grouped = not args.no_group
    with torch.cuda.stream(stream):
        for c in range(copies):
            run_step(rabit, shapes, layers[c], xs, ys, c, grouped)
    stream.synchronize()
    buf = torch.zeros(1 << 22, dtype=torch.int64, device=device)
    rc = lib.rabit_trace_begin(ctypes.c_void_p(buf.data_ptr()), buf.numel() * 8)
    if rc != 0:
        raise SystemExit("trace workload: " + rabit.last_error())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for c in range(copies):
            run_step(rabit, shapes, layers[c], xs, ys, c, grouped)
    n = lib.rabit_trace_launches(None, 0)
    ctas = (ctypes.c_int * n)()
    lib.rabit_trace_launches(ctas, n)
    with torch.cuda.stream(stream):
        for _ in range(20):
            g.replay()
    stream.synchronize()
    lib.rabit_trace_begin(None, 0)
    raw = buf.cpu().numpy().astype(np.uint64)
    if args.trace_dump:
        np.save(args.trace_dump, raw[:64 * int(sum(ctas))])
        json.dump([int(c) for c in ctas], open(args.trace_dump + ".ctas.json", "w"))
    names = ["entry", "wait_over", "x_arrived", "table_built", "first_weights", "last_lookup", "end", "first_block_done"]
    mhz = 1965.0
    rows, off, base = [], 0, None
    for i in range(n):
        full = raw[off:off + 64 * ctas[i]].reshape(ctas[i], 64).astype(np.float64)
        rec = full[:, :8]
        off += 64 * ctas[i]
        if base is None:
            base = rec[:, 0].min()
        entry = (rec[:, 0] - base) / 1e3                                   # us, coarse
        dur = rec[:, 1:] / mhz                                              # us since the CTA's entry (cycles / max SM clock)
        row = {"launch": i, "ctas": int(ctas[i]), "entry_first": round(float(entry.min()), 2), "entry_med": round(float(np.median(entry)), 2),
               "end_abs_max": round(float((entry + dur[:, 5]).max()), 2)}
        for j, nm in enumerate(names[1:]):
            row[nm + "_med"] = round(float(np.median(dur[:, j])), 3)
            row[nm + "_max"] = round(float(dur[:, j].max()), 3)
        rows.append(row)
    sys.stderr.write("times in us; per launch: entry on the global timer (first CTA / median), the rest since each CTA's own entry (median / max over CTAs)\n")
    sys.stderr.write("launch ctas | entry first   med | wait_over     | x_arrived     | table_built   | first_weights | first_blk_done| last_lookup   | end           | end(abs,max)\n")
    for r in rows:
        sys.stderr.write("%3d %4d | %7.2f %7.2f |" % (r["launch"], r["ctas"], r["entry_first"], r["entry_med"]))
        for nm in ("wait_over", "x_arrived", "table_built", "first_weights", "first_block_done", "last_lookup", "end"):
            sys.stderr.write(" %6.2f %6.2f |" % (r[nm + "_med"], r[nm + "_max"]))
        sys.stderr.write(" %7.2f\n" % r["end_abs_max"])
    for row in layers:
        for L in row:
            L.free()
    return {"metric": "phase stamps of the decode GEMV launches (us after the first entry of the cycle)", "value": rows[-1]["end_abs_max"] / copies,
            "unit": "us/step", "n_gpus": 1, "steps": copies, "warmup": 3, "ms_per_step": rows[-1]["end_abs_max"] / copies / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "trace7b", "copies": copies, "grouped": grouped}, "launches": rows, "gpu_launches": n}


def bench_reference(args) -> dict:
    """The reference arm: the CPU oracle as it stands, timed on the host cores.  A step is one decoder layer (seven
    projections); when K steps of the whole layer would not end within a couple of minutes, every step runs the oracle
    on the first R rows of each projection (rows are independent dot products) and the time is scaled by M / R."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    from oracle import rabit_oracle as orc
    from synth import llama2_7b_layer_shapes, make_layer, make_x
    shapes = llama2_7b_layer_shapes()
    inputs = [(make_layer(sh.M, sh.N, K_PATHS, key=(1, 0, p)), make_x(1, sh.N, key=(1, 10_000))) for p, sh in enumerate(shapes)]
    t0 = time.perf_counter()
    L, x = inputs[0]
    orc.linear(L.planes[:, :512], L.g[:, :512], L.h, x)                     # warm-up and a cost estimate: 512 rows of 4096 columns
    est_full_step = (time.perf_counter() - t0) * sum(sh.M * sh.N for sh in shapes) / (512 * 4096)
    steps = max(1, args.steps)
    frac = min(1.0, 120.0 / max(est_full_step * (steps + min(args.warmup, 3)), 1e-9))
    rows = [max(32, int(sh.M * frac) // 32 * 32) for sh in shapes]

    def one_step():
        t = 0.0
        for (L, x), sh, R in zip(inputs, shapes, rows):
            t0 = time.perf_counter()
            orc.linear(L.planes[:, :R], L.g[:, :R], L.h, x)
            t += (time.perf_counter() - t0) * sh.M / R
        return t
    for _ in range(min(args.warmup, 3)):
        one_step()
    per_step = [one_step() for _ in range(steps)]
    value = float(np.mean(per_step)) * 1e6 / len(shapes)
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    sample = ("every step: the oracle on the first %s rows of the seven projections of decoder-layer copy 0 (of %s), time scaled to all rows"
              % ([int(r) for r in rows], [sh.M for sh in shapes]))
    base = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": steps, "warmup": args.warmup, "ms_per_step": float(np.mean(per_step)) * 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "copies": 1, "batch": 1, "K": K_PATHS},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3200)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--repeats", type=int, default=5, help="timed repeats of the K-step region; value is their median")
    ap.add_argument("--no-extras", action="store_true", help="only the contract's line: no other configurations, no warm-L2 / read-probe figures")
    ap.add_argument("--impl", default="rabit", choices=["rabit", "reference"])
    ap.add_argument("--copies", type=int, default=32)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--e2e-steps", type=int, default=2000)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-group", action="store_true", help="one rabit_linear launch per projection (7 per step instead of 4)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-shape", default="", help="extra workloads: keep only the layer shape MxN (e.g. 28672x8192)")
    ap.add_argument("--trace-dump", default="", help="trace7b: also save the raw stamps (numpy file) here")
    ap.add_argument("--workload", default="decoder7b", choices=["decoder7b", "gemm70b", "gemm7b", "gemv70b", "sweep8b", "derive7b", "trace7b"],
                    help="decoder7b is the contract's line; the others are extra single-GPU measurements")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        res = bench_reference(args)
    elif args.workload == "derive7b":
        res = bench_derive(args)
    elif args.workload == "trace7b":
        res = bench_trace(args)
    elif args.workload != "decoder7b":
        res = bench_cases(args)
    else:
        res = bench_rabit(args)
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
