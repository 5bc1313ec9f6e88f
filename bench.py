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

# DRAM bytes (read + write) of the four launches of one grouped step, from the ncu capture summarised in
# profiles/gemv_mma_llama2_7b_decoder_layer.md (12.759 + 4.296 + 22.771 + 11.417 MB); valid for the
# default grouped batch-1 workload only.
NCU_DRAM_BYTES_PER_GROUPED_STEP = 51_272_192

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
def build_workload(copies: int, batch: int, device: str, tokens: int, seed_cfg: int = 1, hints: bool = True):
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
    if hints:
        # the order a decoder runs them in: q|k|v -> o -> gate|up -> down -> the next decoder layer's q|k|v
        for c in range(copies):
            nxt = layers[(c + 1) % copies]
            row = layers[c]
            for p in (0, 1, 2):
                row[p].set_next([row[3]])
            row[3].set_next([row[4], row[5]])
            row[4].set_next([row[6]])
            row[5].set_next([row[6]])
            row[6].set_next([nxt[0], nxt[1], nxt[2]])
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

    copies, batch, tokens = args.copies, args.batch, 16
    shapes, layers, xs, xs_host, ys = build_workload(copies, batch, device, tokens, hints=not args.no_hints)
    step_bytes = sum(layer_bytes(sh.M, sh.N, batch) for sh in shapes)
    n_proj = len(shapes)
    stream = torch.cuda.Stream(device)

    # one CUDA graph per decoder-layer copy, and one that walks all copies once
    def capture(copy_ids):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for c in copy_ids:
                run_step(rabit, shapes, layers[c], xs, ys, c % tokens, grouped)
        return g

    grouped = not args.no_group
    launches_per_step = len(GROUPS) if grouped else n_proj
    with torch.cuda.stream(stream):
        for c in range(copies):                      # also the first-call set-up of every kernel variant
            run_step(rabit, shapes, layers[c], xs, ys, c % tokens, grouped)
    stream.synchronize()
    use_graph = not args.no_graph
    if use_graph:
        cycle_graph = capture(list(range(copies)))
        step_graphs = [capture([c]) for c in range(copies)]

    def run_steps(first: int, count: int):
        """Steps first .. first+count-1; step s uses decoder-layer copy s % copies."""
        s, end = first, first + count
        with torch.cuda.stream(stream):
            while s < end:
                if not use_graph:
                    run_step(rabit, shapes, layers[s % copies], xs, ys, (s % copies) % tokens, grouped)
                    s += 1
                elif s % copies == 0 and end - s >= copies:
                    cycle_graph.replay(); s += copies
                else:
                    step_graphs[s % copies].replay(); s += 1

    sampler = ClockSampler(local_rank) if rank == 0 else None
    run_steps(0, args.warmup)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    with torch.cuda.stream(stream):
        ev0.record(stream)
    run_steps(args.warmup, args.steps)
    with torch.cuda.stream(stream):
        ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms = max_over_ranks(ev0.elapsed_time(ev1), dist, device)
    clocks = sampler.summary(t_wall0, t_wall1) if sampler else None
    if sampler and clocks["samples"] < 3:
        # the timed region was shorter than the sampling period: repeat the same work, untimed,
        # for about a second under the sampler and report the clocks seen there
        reps = max(1, int(1.0 / max(ms * 1e-3, 1e-4)))
        t0 = time.time()
        for _ in range(reps):
            run_steps(args.warmup, args.steps)
        torch.cuda.synchronize()
        clocks = sampler.summary(t0, time.time())
        clocks["note"] = "sampled over an untimed repeat of the timed region (region shorter than the sampler period)"
    if sampler:
        sampler.stop()

    ms_per_step = ms / args.steps
    us_per_layer = ms_per_step * 1e3 / n_proj
    gbs = step_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if rank == 0 or dist is not None:
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
        t0 = time.perf_counter()
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

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback"
    result = {
        "metric": METRIC, "value": whole_job_us_per_layer(ms_per_step, n_proj, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 tensor-core products of exact fixed-point activations, int32/fp32 accumulate, fp16 in/out",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "copies": copies, "batch": batch, "K": K_PATHS,
                   "packed_bytes_total": int(step_bytes * copies),
                   "l2": "inputs larger than L2: rotation over %d distinct decoder layers (%.0f MB)" % (copies, step_bytes * copies / 1e6),
                   "launch": "CUDA graph replay" if use_graph else "stream launches",
                   "launches_per_step": launches_per_step,
                   "grouping": "q|k|v and gate|up (projections that share their input) each go through one rabit_linear_group launch; "
                               "o and down through rabit_linear" if grouped else "one rabit_linear launch per projection",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "achieved_hbm_gbs": gbs * world,
        "tokens_per_s_32_layer_stack": world * 1.0 / (32 * ms_per_step * 1e-3),
        "gpu_launches": args.steps * launches_per_step,
        "clocks": clocks,
        "e2e": e2e,
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                     "traffic": (NCU_DRAM_BYTES_PER_GROUPED_STEP / launches_per_step) if (grouped and batch == 1) else None,
                     "algorithmic_bytes_per_launch": step_bytes / launches_per_step,
                     "peak_source": peak_src,
                     "note": "per launch of rabit_gemv_mma_kernel, averaged over the launches of a step: algorithmic bytes of the "
                             "step / device time of the step (launch gaps included); traffic = ncu dram bytes of the same launches"},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(sample_projections=n_proj)
    for row in layers:
        for L in row:
            L.free()
    if dist is not None:
        dist.destroy_process_group()
    return result if rank == 0 else None


# ---------------------------------------------------------------------------------------
# the oracle, timed as it stands on the host cores
# ---------------------------------------------------------------------------------------
def cpu_baseline(sample_projections: int = 7, repeats: int = 1) -> dict:
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
    return {"value": dt * 1e6 / len(shapes), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "decoder-layer copy 0, its %d projections once each, batch 1 (float64: unpack signs, dense W, product)" % len(shapes)}


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
            "dtype": "f16 tensor-core products, fp32 accumulate" if gemm else "int8 tensor-core products of exact fixed-point activations",
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
                              "upload of header and scales and two fills per call"})
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
    shapes, layers, xs, xs_host, ys = build_workload(copies, 1, device, 16, hints=not args.no_hints)
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
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    per_layer = []
    base = None
    for _ in range(max(1, min(args.warmup, 1))):
        cpu_baseline(sample_projections=1)
    t0 = time.perf_counter()
    steps = max(1, min(args.steps, 4))
    for _ in range(steps):
        base = cpu_baseline()
        per_layer.append(base["value"])
    dt = time.perf_counter() - t0
    value = float(np.mean(per_layer))
    base["value"] = value
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 / steps, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch": 1, "K": K_PATHS},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32000)
    ap.add_argument("--warmup", type=int, default=640)
    ap.add_argument("--impl", default="rabit", choices=["rabit", "reference"])
    ap.add_argument("--copies", type=int, default=32)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--e2e-steps", type=int, default=2000)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-group", action="store_true", help="one rabit_linear launch per projection (7 per step instead of 4)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-shape", default="", help="extra workloads: keep only the layer shape MxN (e.g. 28672x8192)")
    ap.add_argument("--no-hints", action="store_true", help="do not tell the layers which layer runs next (no weight prefetch across launches)")
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
