#!/usr/bin/env python
"""Benchmark of the W4A16 g128 linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = the seven linear layers of one Llama-2-7B-shaped decoder layer at M = 1 (decode)
on packed INT4 weights resident in HBM, issued as four C-ABI calls (fused q/k/v, o, fused
gate/up, down) and replayed as a CUDA graph; the step's weights
rotate over several independently seeded layers so that consecutive steps never find their
weights in L2.  The headline value is the algorithmic GB/s of that step (packed codes +
scales + zero points + activations in and out, each moved once).  The same JSON line also
carries the prefill GEMM at M = 2048 on the Llama-2-13B MLP shapes (TFLOP/s), the offline
quantize+pack kernel, the roofline fraction of the dominant kernel, the end-to-end figure
with host buffers, and the CPU oracle timed on a bounded sample.

With N > 1 (torchrun) every rank runs an independent replica; the reported value is all
ranks' bytes over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2306_00978_b200 import replicas, synth  # noqa: E402

METRIC = "W4A16 g128 GEMV GB/s at M=1 (Llama-2-7B decoder-layer linears)"
UNIT = "GB/s"
GROUP = 128
ALPHA = 0.5
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
NOMINAL_HBM_GBS = 8000.0
NOMINAL_FP16_TFLOPS = 2250.0
# DRAM bytes per launch of the dominant kernel from the ncu capture summarised under
# profiles/ (None until a capture of the current kernel exists).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {(11008, 4096): 23470000, (4096, 4096): 8760000}


def algorithmic_bytes(N: int, K: int, M: int, group: int = GROUP) -> int:
    """codes + fp16 scales + 4-bit zero points + x in + y out, each moved once."""
    return N * K // 2 + 2 * N * K // group + N * K // (2 * group) + 2 * M * K + 2 * M * N


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
                "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append((time.time(), parts))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()          # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)

    def summary(self, t0: float, t1: float):
        rows = [r for (t, r) in self.rows if t0 <= t <= t1] or [r for (_, r) in self.rows]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        mhz, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            try:
                mhz.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(mhz)}


# --------------------------------------------------------------------------- workload
def build_layers(n_layers: int, seed0: int = 2000):
    """Quantizes n_layers x 7 seeded Llama-2-7B-shaped matrices on the GPU (setup, untimed)."""
    import torch
    from paper_2306_00978_b200 import binding
    layers = []
    for li in range(n_layers):
        lin = []
        for idx, (name, K, N) in enumerate(synth.LLAMA2_7B_LAYER):
            seed = seed0 + 16 * li + idx
            # q/k/v and gate/up read one activation each, so they share its calibration statistic
            # and scale s (seeded by the first matrix of the group)
            xseed = seed0 + 16 * li + {1: 0, 2: 0, 5: 4}.get(idx, idx)
            W = torch.from_numpy(synth.weight(seed, N, K)).cuda()
            a = torch.from_numpy(synth.act_mean_abs(xseed, K)).cuda()
            qw, sc, zp = binding.quantize_pack(W, a, ALPHA, GROUP)
            s = binding.channel_scale(a, ALPHA, K)
            x = torch.from_numpy(synth.activations(xseed, 1, K)).cuda()
            xs = (x.float() / s[None, :]).half().contiguous()     # the caller's x / s
            lin.append(dict(name=name, N=N, K=K, qw=qw, sc=sc, zp=zp, x=xs))
            del W
        # host-side view of a step (the e2e leg): the step's four activations in one pinned buffer,
        # its seven outputs in another, one copy each way per step; the device tensors the calls
        # read and write are views into the device-side images of the two buffers
        firsts = [idxs[0] for idxs in STEP_CALLS]
        x_host = torch.cat([lin[i]["x"].reshape(-1) for i in firsts]).cpu().pin_memory()
        x_dev = torch.empty(x_host.numel(), dtype=torch.float16, device="cuda")
        y_dev = torch.empty(sum(l["N"] for l in lin), dtype=torch.float16, device="cuda")
        y_host = torch.empty(y_dev.numel(), dtype=torch.float16).pin_memory()
        off = 0
        for i in firsts:
            lin[i]["x_dev_in"] = x_dev[off:off + lin[i]["K"]].view(1, -1)
            off += lin[i]["K"]
        off = 0
        for l in lin:
            l["y"] = y_dev[off:off + l["N"]].view(1, -1)
            off += l["N"]
        lin[0].update(x_host=x_host, x_dev=x_dev, y_dev=y_dev, y_host=y_host)
        layers.append(lin)
    torch.cuda.synchronize()
    return layers


# The step's calls: layers that read the same activation go through awq_linear_multi (fused
# q/k/v and gate/up, as the paper's Sec. 4.2 fuses QKV); o_proj and down_proj are single calls.
STEP_CALLS = ((0, 1, 2), (3,), (4, 5), (6,))


def run_step(layer, e2e=False):
    from paper_2306_00978_b200 import binding
    if e2e:                                            # the step's inputs from pinned host memory
        layer[0]["x_dev"].copy_(layer[0]["x_host"], non_blocking=True)
    for idxs in STEP_CALLS:
        first = layer[idxs[0]]
        xin = first["x_dev_in"] if e2e else first["x"]
        if len(idxs) == 1:
            binding.linear(xin, first["qw"], first["sc"], first["zp"], first["N"], first["K"], GROUP,
                           out=first["y"])
        else:
            binding.linear_multi(xin, [(layer[i]["qw"], layer[i]["sc"], layer[i]["zp"], layer[i]["N"]) for i in idxs],
                                 first["K"], GROUP, outs=[layer[i]["y"] for i in idxs])
    if e2e:                                            # the step's outputs back to the host
        layer[0]["y_host"].copy_(layer[0]["y_dev"], non_blocking=True)


def run_step_e2e(layer):
    """The same step through host buffers: the step's x from pinned memory in (one copy), its y
    back out (one copy)."""
    run_step(layer, e2e=True)


def capture_steps(fn, layers):
    """One CUDA graph per layer, captured from the C-ABI calls of one step (the launch-bound
    inner loop of decode is replayed as a graph, as a serving stack would).  Returns the
    graphs and the number of library kernels in one step."""
    import torch
    from paper_2306_00978_b200 import binding
    graphs = []
    side = torch.cuda.Stream()
    per_step = 0
    for layer in layers:
        fn(layer)                                    # warm: attributes set, workspace registered
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for layer in layers:
            g = torch.cuda.CUDAGraph()
            n0 = binding.launch_count()
            with torch.cuda.graph(g, stream=side):
                fn(layer)
            per_step = binding.launch_count() - n0
            graphs.append(g)
        # the whole rotation as one graph (a decoder stack is replayed as one graph, layer after
        # layer): len(layers) steps per replay
        stack = torch.cuda.CUDAGraph()
        with torch.cuda.graph(stack, stream=side):
            for layer in layers:
                fn(layer)
    torch.cuda.synchronize()
    return graphs, per_step, stack


def timed_region(graphs, stack, steps: int, warmup: int, device: str):
    """W warm-up steps, then exactly `steps` steps between barrier+synchronize, CUDA events on
    the launching stream; returns (seconds = max over ranks, wall-clock window).  Whole rotations
    of the layers are replayed as the stack graph (len(graphs) steps each), the remainder as
    single-layer graphs."""
    import torch
    L = len(graphs)
    for i in range(warmup // L):
        stack.replay()
    for i in range(warmup % L):
        graphs[i].replay()
    torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    start.record()
    for i in range(steps // L):
        stack.replay()
    for i in range(steps % L):
        graphs[i].replay()
    end.record()
    torch.cuda.synchronize()
    t1 = time.time()
    replicas.barrier()
    sec = start.elapsed_time(end) * 1e-3
    return replicas.max_over_ranks(sec, device), (t0, t1)


def gemm_section(peaks, reps: int = 20):
    """Prefill GEMM, M = 2048, Llama-2-13B MLP shapes: best-of-reps and mean TFLOP/s (the binding
    registers the optional stream-K workspace)."""
    import torch
    from paper_2306_00978_b200 import binding
    out = []
    M = 2048
    for idx, (name, K, N) in enumerate(synth.LLAMA2_13B_MLP):
        seed = 3000 + idx
        W = torch.from_numpy(synth.weight(seed, N, K)).cuda()
        a = torch.from_numpy(synth.act_mean_abs(seed, K)).cuda()
        qw, sc, zp = binding.quantize_pack(W, a, ALPHA, GROUP)
        s = binding.channel_scale(a, ALPHA, K)
        x = torch.from_numpy(synth.activations(seed, M, K)).cuda()
        xs = (x.float() / s[None, :]).half().contiguous()
        y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        del W
        for _ in range(3):
            binding.linear(xs, qw, sc, zp, N, K, GROUP, out=y)
        torch.cuda.synchronize()
        # four calls per timed interval: the host prepares the next launch (tensor maps, argument
        # checks) while the GPU runs the previous one, so the interval is device time
        inner = 4
        times = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(inner):
                binding.linear(xs, qw, sc, zp, N, K, GROUP, out=y)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) * 1e-3 / inner)
        binding.poll_status()
        flops = 2.0 * M * N * K
        best, mean = min(times), sum(times) / len(times)
        out.append({"shape": f"{K}->{N}", "M": M, "tflops_best": flops / best / 1e12,
                    "tflops_mean": flops / mean / 1e12, "ms_best": best * 1e3,
                    "frac_of_measured_bf16_burst": flops / best / 1e12 / peaks["bf16_tflops"],
                    "frac_of_nominal_2250": flops / best / 1e12 / NOMINAL_FP16_TFLOPS})
    return out


def quantize_section(peaks, reps: int = 10):
    import torch
    from paper_2306_00978_b200 import binding
    N, K = 11008, 4096
    W = torch.from_numpy(synth.weight(2004, N, K)).cuda()
    a = torch.from_numpy(synth.act_mean_abs(2004, K)).cuda()
    # the C entry point on preallocated outputs (the Python wrapper would add its allocations)
    qw, sc, zp = binding.quantize_pack(W, a, ALPHA, GROUP)
    L = binding.lib()
    stream = torch.cuda.current_stream().cuda_stream
    args = (W.data_ptr(), a.data_ptr(), ALPHA, GROUP, qw.data_ptr(), sc.data_ptr(), zp.data_ptr(), N, K, stream)
    for _ in range(3):
        assert L.awq_quantize_pack(*args) == 0
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        assert L.awq_quantize_pack(*args) == 0
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) * 1e-3)
    nbytes = 2 * N * K + 4 * K + N * K // 2 + 2 * N * K // GROUP + N * K // (2 * GROUP)
    return {"shape": f"{K}->{N}", "gbs": nbytes / best / 1e9, "ms": best * 1e3,
            "frac_of_hbm_peak": nbytes / best / 1e9 / peaks["hbm_gbs"],
            "note": "awq_quantize_pack on preallocated outputs, best of %d single launches" % reps}


def search_section():
    """Scale search (Sec. 3.2) on one 4096 -> 4096 layer: 20 grid points, 512 synthetic calibration
    tokens with outlier channels; wall-clock of the call (it returns its result on the host)."""
    import time
    import torch
    from paper_2306_00978_b200 import binding
    N, K, M = 4096, 4096, 512
    W = torch.from_numpy(synth.weight(2000, N, K)).cuda()
    X = torch.from_numpy(synth.calibration(2000, K, M)).cuda()
    a = X.float().abs().mean(dim=0).contiguous()
    alphas = [i / 20 for i in range(20)]
    binding.search_alpha(W, a, X, GROUP, alphas)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    losses, best = binding.search_alpha(W, a, X, GROUP, alphas)
    dt = time.perf_counter() - t0
    return {"shape": f"{K}->{N}", "calibration_tokens": M, "grid": len(alphas), "ms": dt * 1e3,
            "best_alpha": alphas[best], "loss_best_over_loss_alpha0": losses[best] / losses[0]}


def clip_section():
    """Weight clipping (Sec. 3.2) on one 4096 -> 4096 layer: 20 range ratios per group, then the
    clipped quantizer; CUDA events, best of 5."""
    import torch
    from paper_2306_00978_b200 import binding
    N, K = 4096, 4096
    W = torch.from_numpy(synth.weight(2000, N, K)).cuda()
    a = torch.from_numpy(synth.act_mean_abs(2000, K)).cuda()
    ratios = [1.0 - 0.5 * i / 19 for i in range(20)]
    times = {"search": [], "quantize": []}
    for _ in range(6):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        r = binding.search_clip(W, a, ALPHA, GROUP, ratios)
        e[1].record()
        binding.quantize_pack(W, a, ALPHA, GROUP, clip_ratio=r)
        e[2].record()
        torch.cuda.synchronize()
        times["search"].append(e[0].elapsed_time(e[1]))
        times["quantize"].append(e[1].elapsed_time(e[2]))
    return {"shape": f"{K}->{N}", "ratios": len(ratios), "search_ms": min(times["search"][1:]),
            "clipped_quantize_ms": min(times["quantize"][1:]),
            "groups_clipped_frac": float((r < 1.0).float().mean().item())}


# ------------------------------------------------------------------- oracle (CPU) arm
def _oracle_layer_inputs(max_rows=None, col_div=1):
    """Quantizes one decoder layer's matrices with the oracle; optionally only the first
    `max_rows` output rows (whole 128-row slabs) and the first K / col_div input channels (whole
    128-column blocks) of each, to bound the work."""
    from oracle import awq_oracle as orc
    items = []
    for idx, (name, K, N) in enumerate(synth.LLAMA2_7B_LAYER):
        seed = 2000 + idx
        n = N if max_rows is None else min(N, max_rows)
        kc = max(128, (K // col_div) // 128 * 128)
        W = np.ascontiguousarray(synth.weight(seed, N, K)[:n, :kc])
        a = synth.act_mean_abs(seed, K)[:kc]
        s = orc.channel_scale(a, ALPHA)
        x = synth.activations(seed, 1, K)[:, :kc]
        xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
        qw, sc, zp = orc.quantize_pack(W, a, ALPHA, GROUP)
        items.append((n, kc, xs, qw, sc, zp))
    return items


def _oracle_step(items):
    from oracle import awq_oracle as orc
    for (n, K, xs, qw, sc, zp) in items:
        orc.linear_from_packed(xs, qw, sc, zp, n, K, GROUP)


def cpu_baseline(budget_s: float = 20.0):
    """The oracle as it stands on the host cores, on a bounded sample of the same step."""
    rows = 1024
    items = _oracle_layer_inputs(max_rows=rows)
    nbytes = sum(algorithmic_bytes(n, K, 1) for (n, K, *_rest) in items)
    t0 = time.time()
    reps = 0
    while True:
        _oracle_step(items)
        reps += 1
        if time.time() - t0 > budget_s * 0.5 or reps >= 3:
            break
    sec = (time.time() - t0) / reps
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return {"value": nbytes / sec / 1e9, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"first {rows} output rows of each of the 7 linears of one layer at M=1 "
                      f"(unpack + fp64 dequantize + fp64 product), {reps} repetitions"}


def reference_arm(args):
    rank, world, _ = replicas.env_world()
    if rank != 0:
        return 0
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # size the per-step sample so that the whole run stays within a few minutes: rows first (down
    # to one 128-row slab of each matrix), then input channels; about 50 ns per weight on 8 cores
    budget = 150.0 / (steps + warmup)
    rows, col_div = 1024, 1
    weights_per_row = sum(K for (_name, K, _N) in synth.LLAMA2_7B_LAYER)
    cost = lambda r, c: r * weights_per_row / c * 50e-9
    while rows > 128 and cost(rows, col_div) > budget:
        rows //= 2
    while col_div < 32 and cost(rows, col_div) > budget:
        col_div *= 2
    items = _oracle_layer_inputs(max_rows=rows, col_div=col_div)
    nbytes = sum(algorithmic_bytes(n, K, 1) for (n, K, *_rest) in items)
    for _ in range(warmup):
        _oracle_step(items)
    t0 = time.time()
    for _ in range(steps):
        _oracle_step(items)
    sec = (time.time() - t0) / steps
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    value = nbytes / sec / 1e9
    sample = (f"each step = first {rows} output rows" + (f" x first 1/{col_div} of the input channels" if col_div > 1 else "") +
              " of each of the 7 linears of one layer at M=1 through the CPU oracle")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "llama2-7b decoder-layer linears, M=1, g128, alpha=0.5 (bounded sample)",
                       "rows_per_linear": rows, "input_channel_fraction": 1.0 / col_div},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


def one_shape(args):
    """A small, self-contained run of one shape for ncu captures (random packed bytes: the
    kernels' work does not depend on the values)."""
    import torch
    from paper_2306_00978_b200 import binding
    N, K, M = args.one
    copies = []
    for _ in range(3):
        qw = torch.randint(0, 256, (N * K // 2,), dtype=torch.uint8, device="cuda")
        sc = (torch.rand((N // 16, K // GROUP, 16), device="cuda") * 0.01 + 0.001).half()
        zp = torch.randint(0, 256, (N // 32, K // GROUP, 16), dtype=torch.uint8, device="cuda")
        copies.append((qw, sc, zp))
    x = torch.randn((M, K), device="cuda").half()
    y = torch.empty((M, N), device="cuda", dtype=torch.float16)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(args.reps):
        if r == args.reps - 1:
            e0.record()
        for (qw, sc, zp) in copies:
            binding.linear(x, qw, sc, zp, N, K, GROUP, out=y, path=args.path)
    e1.record()
    torch.cuda.synchronize()
    binding.poll_status()
    us = e0.elapsed_time(e1) * 1e3 / len(copies)
    print(json.dumps({"one": [N, K, M], "path": args.path, "us_per_launch_last_pass": us,
                      "algorithmic_bytes": algorithmic_bytes(N, K, M), "flops": 2 * M * N * K}))
    return 0


def sweep(args):
    """The full-shape sweep over the 7B layer's three distinct shapes: token counts 1 .. 8192 and
    both group sizes through awq_linear (random packed weights, three rotating copies so that
    small shapes do not sit in L2, eight calls per CUDA-graph replay, best of five replays).
    One JSON object per line: microseconds, algorithmic GB/s, TFLOP/s."""
    import torch
    from paper_2306_00978_b200 import binding
    shapes = [("q/k/v/o", 4096, 4096), ("gate/up", 4096, 11008), ("down", 11008, 4096)]
    for group in (128, 64):
        for name, K, N in shapes:
            copies = []
            for _ in range(3):
                qw = torch.randint(0, 256, (N * K // 2,), dtype=torch.uint8, device="cuda")
                sc = (torch.rand((N // 16, K // group, 16), device="cuda") * 0.01 + 0.001).half()
                zp = torch.randint(0, 256, (N // 32, K // group, 16), dtype=torch.uint8, device="cuda")
                copies.append((qw, sc, zp))
            for M in (1, 2, 4, 8, 16, 32, 64, 128, 512, 2048, 8192):
                x = torch.randn((M, K), device="cuda").half()
                y = torch.empty((M, N), device="cuda", dtype=torch.float16)
                calls = 8 if M <= 512 else 2
                for i in range(3):
                    binding.linear(x, *copies[i], N, K, group, out=y)
                torch.cuda.synchronize()
                graph, stream = torch.cuda.CUDAGraph(), torch.cuda.Stream()
                with torch.cuda.stream(stream):
                    with torch.cuda.graph(graph, stream=stream):
                        for i in range(calls):
                            binding.linear(x, *copies[i % 3], N, K, group, out=y)
                torch.cuda.synchronize()
                graph.replay()
                torch.cuda.synchronize()
                best = float("inf")
                for _ in range(5):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    graph.replay()
                    e1.record()
                    torch.cuda.synchronize()
                    best = min(best, e0.elapsed_time(e1) * 1e3 / calls)
                binding.poll_status()
                nbytes = N * K // 2 + (N * K // group) * 2 + (N * K // group) // 2 + M * K * 2 + M * N * 2
                print(json.dumps({"shape": name, "K": K, "N": N, "group": group, "M": M, "us": round(best, 2),
                                  "GBps": round(nbytes / best / 1e3, 1),
                                  "TFLOPs": round(2 * M * N * K / best / 1e6, 1)}), flush=True)
    return 0


# --------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=8, help="independently seeded layers to rotate over (one CUDA graph replays them back to back)")
    ap.add_argument("--skip-extras", action="store_true", help="only the headline step (for profiling)")
    ap.add_argument("--one", nargs=3, type=int, metavar=("N", "K", "M"),
                    help="profiling aid: a few awq_linear launches of one shape on random packed "
                         "weights (three rotating copies), then exit")
    ap.add_argument("--path", type=int, default=0, help="with --one: 0 auto, 1 GEMV, 2 GEMM, 3 split-K GEMV, 4 single-SM GEMM")
    ap.add_argument("--reps", type=int, default=3, help="with --one: passes over the three copies")
    ap.add_argument("--sweep", action="store_true",
                    help="per-shape table over the 7B layer shapes, M = 1 .. 8192, both group sizes; then exit")
    args = ap.parse_args()
    if args.one:
        return one_shape(args)
    if args.sweep:
        return sweep(args)

    if args.impl == "reference":
        return reference_arm(args)

    import torch
    from paper_2306_00978_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    rank, world, local_rank = replicas.env_world()
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    replicas.init("nccl")
    binding.lib()                                     # fail now if the library is missing
    peaks = load_peaks()
    warmup = max(3, args.warmup)
    steps = max(1, args.steps)

    layers = build_layers(args.layers)
    step_bytes = sum(algorithmic_bytes(l["N"], l["K"], 1) for l in layers[0])
    packed_bytes = sum(l["qw"].numel() + l["sc"].numel() * 2 + l["zp"].numel() for l in layers[0])

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    graphs, launches_per_step, stack = capture_steps(run_step, layers)
    e2e_graphs, _, e2e_stack = capture_steps(run_step_e2e, layers)
    sec, (w0, w1) = timed_region(graphs, stack, steps, warmup, device)
    e2e_sec, _ = timed_region(e2e_graphs, e2e_stack, steps, warmup, device)
    launches = launches_per_step * steps
    clocks = None
    if rank == 0:
        if w1 - w0 < 1.0:
            # the timed region is too short for 100 ms clock samples: keep the same load
            # running (untimed) for about a second and sample that instead
            w0 = time.time()
            while time.time() - w0 < 1.2:
                for i in range(50):
                    stack.replay()
                torch.cuda.synchronize()
            w1 = time.time()
            clocks_note = "sampled over ~1.2 s of the same steps run right after the timed region"
        else:
            clocks_note = "sampled during the timed region"
        time.sleep(0.15)
        sampler.stop()
        clocks = sampler.summary(w0, w1)
        clocks["note"] = clocks_note
    binding.poll_status()

    value = replicas.aggregate_throughput(step_bytes * steps, sec) / 1e9
    e2e_value = replicas.aggregate_throughput(step_bytes * steps, e2e_sec) / 1e9
    per_launch_s = sec / max(1, launches)
    achieved = step_bytes * steps / sec / 1e9         # one GPU's algorithmic GB/s over the region
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": sec / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 x int4 -> f32", "data": "synthetic",
        "config": {"workload": "llama2-7b decoder-layer linears (q,k,v,o 4096->4096; gate,up 4096->11008; "
                               "down 11008->4096), M=1, g128, alpha=0.5",
                   "layers_rotated": args.layers, "packed_bytes_per_layer": packed_bytes,
                   "l2_policy": f"weights rotate over {args.layers} layers "
                                f"({args.layers * packed_bytes / 1e6:.0f} MB > 2 x 126 MB L2)",
                   "algorithmic_bytes_per_step": step_bytes, "parallelism": f"replicas x{world}",
                   "launch": "each step is 4 C-ABI calls: awq_linear_multi(q,k,v), awq_linear(o), "
                             "awq_linear_multi(gate,up), awq_linear(down); the rotating layers are replayed "
                             "back to back as one CUDA graph (layers_rotated steps per replay), a remainder of "
                             "steps as single-layer graphs"},
        "roofline": {"bound": "hbm", "kernel": "gemv_band_kernel<128,4,true,true,5>", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                     "avg_launch_us": per_launch_s * 1e6,
                     # per launch, averaged over the step's launches, from the per-matrix captures
                     # in profiles/gemv_band_kernel_llama2_7b_M1.md (4x 4096^2, 3x 4096x11008)
                     "traffic": (4 * NCU_TRAFFIC_BYTES_PER_LAUNCH[(4096, 4096)] +
                                 3 * NCU_TRAFFIC_BYTES_PER_LAUNCH[(11008, 4096)]) / max(1, launches_per_step),
                     "algorithmic_bytes_per_launch": step_bytes / max(1, launches_per_step)},
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": sum(2 * layers[0][idxs[0]]["K"] for idxs in STEP_CALLS),
                "d2h_bytes_per_step": sum(2 * l["N"] for l in layers[0])},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if rank == 0 and not args.skip_extras:
        line["gemm_m2048"] = gemm_section(peaks)
        line["quantize_pack"] = quantize_section(peaks)
        line["alpha_search"] = search_section()
        line["clip_search"] = clip_section()
        if world == 1:
            del graphs, e2e_graphs, layers
            torch.cuda.empty_cache()
            line["cpu_baseline"] = cpu_baseline()
    if rank == 0:
        print(json.dumps(line), flush=True)
    replicas.barrier()
    replicas.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
