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
# DRAM traffic of the dominant kernel: ncu's dram__bytes_read.sum + dram__bytes_write.sum over the
# algorithmic bytes of the captured launch (profiles/gemv_band_kernel_llama2_7b_M1.md: per-matrix
# captures of 4096 -> 11008 and 4096 -> 4096; traffic grows in proportion to the packed bytes).
NCU_TRAFFIC_RATIO = 1.0005
DOMINANT_KERNEL = "gemv_band_kernel<128,4,true,true,5>"
NCU_TRAFFIC_NOTE = ("scaled from the ncu captures of single-matrix launches in "
                    "profiles/gemv_band_kernel_llama2_7b_M1.md: dram bytes / algorithmic bytes = 1.0002 .. 1.001")


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
            # the raw activation: the step's calls scale it by 1 / s themselves (awq_linear*_scaled,
            # step S6 folded into the matrix-vector kernel)
            x = torch.from_numpy(synth.activations(xseed, 1, K)).cuda()
            lin.append(dict(name=name, N=N, K=K, qw=qw, sc=sc, zp=zp, x=x, s=binding.inverse_channel_scale(a, ALPHA, K)))
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


def run_calls(layer, calls, e2e=False):
    from paper_2306_00978_b200 import binding
    for idxs in calls:
        first = layer[idxs[0]]
        xin = first["x_dev_in"] if e2e else first["x"]
        binding.linear_multi_scaled(xin, first["s"],
                                    [(layer[i]["qw"], layer[i]["sc"], layer[i]["zp"], layer[i]["N"]) for i in idxs],
                                    first["K"], GROUP, outs=[layer[i]["y"] for i in idxs])


def run_step(layer, e2e=False):
    if e2e:                                            # the step's inputs from pinned host memory
        layer[0]["x_dev"].copy_(layer[0]["x_host"], non_blocking=True)
    run_calls(layer, STEP_CALLS, e2e)
    if e2e:                                            # the step's outputs back to the host
        layer[0]["y_host"].copy_(layer[0]["y_dev"], non_blocking=True)


def run_step_e2e(layer):
    """The same step through host buffers: the step's x from pinned memory in (one copy), its y
    back out (one copy)."""
    run_step(layer, e2e=True)


def capture_chain(fn, layers, steps: int):
    """ONE CUDA graph of exactly `steps` steps, the layers rotating (step i uses layer i mod L), so
    that every launch of the region is chained to the one before it by programmatic dependent launch
    - a decoder stack is replayed as one graph.  Returns (graph, library kernels per step)."""
    import torch
    from paper_2306_00978_b200 import binding
    for layer in layers:
        fn(layer)                                    # warm: attributes set, workspace registered
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        n0 = binding.launch_count()
        with torch.cuda.graph(g, stream=side):
            for i in range(steps):
                fn(layers[i % len(layers)])
        per_step = (binding.launch_count() - n0) // steps
    torch.cuda.synchronize()
    return g, per_step


def capture_chain_e2e(layers, steps: int):
    """The same `steps` steps with, per step, the host -> device copy of the step's activations (one
    pinned buffer) and the device -> host copy of its outputs, as ONE CUDA graph over three streams:
    the copies of a step overlap the kernels of its neighbours, as a serving loop with asynchronous
    copies does.  Dependencies: a step's kernels wait for its own input copy; its output copy waits
    for its kernels; a layer's buffers are reused len(layers) steps later, after the kernels that
    read them and the copy that drained them."""
    import torch
    for layer in layers:
        run_step_e2e(layer)
    torch.cuda.synchronize()
    n = len(layers)
    side, s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            start = torch.cuda.Event()
            start.record(side)
            s_in.wait_event(start)
            s_out.wait_event(start)
            done_c, done_o = {}, {}
            for i in range(steps):
                layer = layers[i % n]
                head = layer[0]
                if i >= n:
                    s_in.wait_event(done_c[i - n])          # the kernels that read this x_dev are through
                with torch.cuda.stream(s_in):
                    head["x_dev"].copy_(head["x_host"], non_blocking=True)
                    ev_in = torch.cuda.Event()
                    ev_in.record(s_in)
                side.wait_event(ev_in)
                if i >= n:
                    side.wait_event(done_o[i - n])          # this y_dev has been copied out
                run_calls(layer, STEP_CALLS, e2e=True)
                done_c[i] = torch.cuda.Event()
                done_c[i].record(side)
                s_out.wait_event(done_c[i])
                with torch.cuda.stream(s_out):
                    head["y_host"].copy_(head["y_dev"], non_blocking=True)
                    done_o[i] = torch.cuda.Event()
                    done_o[i].record(s_out)
            for s2 in (s_in, s_out):
                ev = torch.cuda.Event()
                ev.record(s2)
                side.wait_event(ev)
    torch.cuda.synchronize()
    return g


def timed_region(graph, steps: int, warmup: int, device: str, min_seconds: float = 0.6, min_replays: int = 50):
    """Warm-up (at least `warmup` steps, as whole replays of the same graph), then R replays of the
    `steps`-step graph between barrier + synchronize, one CUDA event between consecutive replays on
    the launching stream.  R is chosen so that the region lasts at least `min_seconds` (clock samples
    are 100 ms apart) and at least `min_replays`.  Returns (median seconds per replay = max over
    ranks, dict of the spread, wall-clock window, R)."""
    import torch
    for _ in range(max(1, -(-warmup // steps))):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    est = max(1e-6, e0.elapsed_time(e1) * 1e-3 / 3)
    R = int(min(20000, max(min_replays, min_seconds / est)))
    replicas.barrier()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(R + 1)]
    t0 = time.time()
    ev[0].record()
    for r in range(R):
        graph.replay()
        ev[r + 1].record()
    torch.cuda.synchronize()
    t1 = time.time()
    replicas.barrier()
    per = sorted(ev[r].elapsed_time(ev[r + 1]) * 1e-3 for r in range(R))
    med = statistics.median(per)
    spread = {"replays": R, "min": per[0], "p10": per[R // 10], "median": med, "p90": per[(9 * R) // 10],
              "max": per[-1], "mean": sum(per) / R}
    return replicas.max_over_ranks(med, device), spread, (t0, t1), R


def per_position_times(layers, reps: int = 15):
    """Device time of each of the step's four launch positions on its own: a graph that holds only
    that position's call, once per rotating layer, eight times over (chained by programmatic
    dependent launch like the step itself); median over `reps` replays.  Seconds per launch."""
    import torch
    from paper_2306_00978_b200 import binding
    out = []
    side = torch.cuda.Stream()
    for idxs in STEP_CALLS:
        g = torch.cuda.CUDAGraph()
        n = 8 * len(layers)
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(n):
                    run_calls(layers[i % len(layers)], (idxs,))
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e-3 / n)
        out.append(statistics.median(ts))
    binding.poll_status()
    return out


def gemm_section(peaks, sampler=None, reps: int = 20, sustained_s: float = 2.0):
    """Prefill GEMM, M = 2048, Llama-2-13B MLP shapes (the binding registers the optional stream-K
    workspace).  Burst: best and mean of `reps` timings of four back-to-back calls.  Sustained: the
    same call back to back for at least `sustained_s` seconds between two events, SM clock and
    throttle reasons sampled inside that window."""
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
        flops = 2.0 * M * N * K
        best, mean = min(times), sum(times) / len(times)
        row = {"shape": f"{K}->{N}", "M": M, "tflops_best": flops / best / 1e12,
               "tflops_mean": flops / mean / 1e12, "ms_best": best * 1e3,
               "frac_of_measured_bf16_burst": flops / best / 1e12 / peaks["bf16_tflops"],
               "frac_of_nominal_2250": flops / best / 1e12 / NOMINAL_FP16_TFLOPS}
        # sustained: one graph of 64 calls replayed until the window is long enough
        n = 64
        g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(n):
                    binding.linear(xs, qw, sc, zp, N, K, GROUP, out=y)
        torch.cuda.synchronize()
        replays = max(2, int(sustained_s / (n * best)) + 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for _ in range(replays):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        t1 = time.time()
        sec = e0.elapsed_time(e1) * 1e-3
        sus = flops * n * replays / sec / 1e12
        row["sustained"] = {"tflops": sus, "seconds": sec, "calls": n * replays,
                            "frac_of_measured_bf16_sustained": sus / peaks["bf16_tflops_sustained"],
                            "frac_of_nominal_2250": sus / NOMINAL_FP16_TFLOPS,
                            "clocks": sampler.summary(t0 + 0.2, t1) if sampler is not None else None}
        binding.poll_status()
        out.append(row)
        del g
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


def _host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] or [1]))
    except Exception:
        return int(os.cpu_count() or 1)


def cpu_baseline(rows: int = 1024):
    """The oracle as it stands on the host cores, on a bounded sample of the same step: the first
    `rows` output rows of each of the layer's seven matrices.  Its three phases are timed apart:
    quantize + pack (Eq. 2 - Eq. 5), unpack + dequantize to fp64, and the fp64 product."""
    from oracle import awq_oracle as orc
    mats = []
    t_quant = 0.0
    weights = 0
    for idx, (name, K, N) in enumerate(synth.LLAMA2_7B_LAYER):
        seed = 2000 + idx
        n = min(N, rows)
        W = np.ascontiguousarray(synth.weight(seed, N, K)[:n])
        a = synth.act_mean_abs(seed, K)
        x = synth.activations(seed, 1, K)
        t0 = time.time()
        s = orc.channel_scale(a, ALPHA)
        qw, sc, zp = orc.quantize_pack(W, a, ALPHA, GROUP)
        t_quant += time.time() - t0
        xs = (x.astype(np.float32) / s[None, :]).astype(np.float16)
        mats.append((n, K, xs, qw, sc, zp))
        weights += n * K
    nbytes = sum(algorithmic_bytes(n, K, 1) for (n, K, *_r) in mats)
    t_deq = t_mul = 0.0
    reps = 3
    for _ in range(reps):
        for (n, K, xs, qw, sc, zp) in mats:
            t0 = time.time()
            Wdq = orc.dequantize(orc.unpack_qweight(qw, n, K), orc.unpack_zeros(zp, n, K // GROUP),
                                 orc.unpack_scales(sc, n, K // GROUP), GROUP)
            t1 = time.time()
            orc.linear(xs, Wdq)
            t2 = time.time()
            t_deq += t1 - t0
            t_mul += t2 - t1
    t_deq /= reps
    t_mul /= reps
    return {"value": nbytes / (t_deq + t_mul) / 1e9, "unit": UNIT, "cores": _host_threads(), "kind": "oracle",
            "sample": f"first {rows} output rows of each of the 7 linears of one layer at M=1 "
                      f"({weights / 1e6:.1f} M weights); value = algorithmic bytes / (dequantize + multiply)",
            "phases": {"quantize_pack_s": t_quant, "quantize_pack_Mweights_per_s": weights / t_quant / 1e6,
                       "unpack_dequantize_s": t_deq, "unpack_dequantize_Mweights_per_s": weights / t_deq / 1e6,
                       "multiply_fp64_s": t_mul, "multiply_fp64_GFLOPs": 2.0 * weights / t_mul / 1e9,
                       "repetitions_of_layer_phases": reps}}


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
    cores = _host_threads()
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


class RandomPacked:
    """Rotating copies of random packed arrays of one shape (the kernels' work does not depend on the
    values).  cold = True: enough copies that a pass over them moves more than twice the L2 size, so
    that no call finds its weights in L2."""

    def __init__(self, N: int, K: int, group: int, cold: bool = True, max_copies: int = 40):
        import torch
        self.N, self.K, self.group = N, K, group
        packed = N * K // 2 + (N * K // group) * 2 + (N * K // group) // 2
        l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
        n = 3
        if cold:
            n = max(3, min(max_copies, -(-2 * l2 // packed) + 1))
        self.cold = cold and n * packed >= 2 * l2
        self.copies = []
        for _ in range(n):
            qw = torch.randint(0, 256, (N * K // 2,), dtype=torch.uint8, device="cuda")
            sc = (torch.rand((N // 16, K // group, 16), device="cuda") * 0.01 + 0.001).half()
            zp = torch.randint(0, 256, (N // 32, K // group, 16), dtype=torch.uint8, device="cuda")
            self.copies.append((qw, sc, zp))

    def time_chained(self, M: int, path: int = 0, reps: int = 5, calls: int = 0):
        """Microseconds per call inside a CUDA graph of back-to-back calls over the rotating copies
        (launches chained by programmatic dependent launch where the kernel uses it): (best, median)."""
        import torch
        from paper_2306_00978_b200 import binding
        N, K, group = self.N, self.K, self.group
        x = torch.randn((M, K), device="cuda").half()
        y = torch.empty((M, N), device="cuda", dtype=torch.float16)
        n = len(self.copies)
        if calls <= 0:
            calls = max(8, n) if M <= 128 else 2
        for i in range(min(3, n)):
            binding.linear(x, *self.copies[i], N, K, group, out=y, path=path)
        torch.cuda.synchronize()
        graph, stream = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                for i in range(calls):
                    binding.linear(x, *self.copies[i % n], N, K, group, out=y, path=path)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3 / calls)
        binding.poll_status()
        return min(ts), statistics.median(ts)

    def time_isolated(self, M: int, path: int = 0):
        """Microseconds of a single call with nothing in front of it on the device: the stream is
        kept busy by a sleep kernel while the host enqueues event, call, event, so the interval is
        device time of one cold launch (its start-up included, nothing to overlap with).  Median
        over the rotating copies."""
        import torch
        from paper_2306_00978_b200 import binding
        N, K, group = self.N, self.K, self.group
        x = torch.randn((M, K), device="cuda").half()
        y = torch.empty((M, N), device="cuda", dtype=torch.float16)
        binding.linear(x, *self.copies[0], N, K, group, out=y, path=path)
        torch.cuda.synchronize()
        ts = []
        for i in range(len(self.copies)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(400000)
            e0.record()
            binding.linear(x, *self.copies[i], N, K, group, out=y, path=path)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        binding.poll_status()
        return statistics.median(ts)


def _point(N, K, M, group, us, peaks):
    """One measured call as absolute numbers and fractions of both rooflines."""
    nbytes = algorithmic_bytes(N, K, M, group)
    gbs, tf = nbytes / us / 1e3, 2.0 * M * N * K / us / 1e6
    d = {"us": round(us, 2), "GBps": round(gbs, 1), "TFLOPs": round(tf, 2)}
    if M <= 64:          # HBM-bound side of the ridge (about 70 tokens)
        d["frac_hbm_measured"] = round(gbs / peaks["hbm_gbs"], 4)
        d["frac_hbm_8000"] = round(gbs / NOMINAL_HBM_GBS, 4)
    if M >= 64:
        d["frac_tensor_measured_burst"] = round(tf / peaks["bf16_tflops"], 4)
        d["frac_tensor_2250"] = round(tf / NOMINAL_FP16_TFLOPS, 4)
    return d


def config1_section(peaks):
    """configs[0]: a single 4096 -> 4096 linear at M = 1, as an isolated launch and chained."""
    rp = RandomPacked(4096, 4096, GROUP)
    iso = rp.time_isolated(1)
    best, med = rp.time_chained(1)
    return {"shape": "4096->4096", "M": 1, "group": GROUP, "cold_l2": rp.cold, "copies": len(rp.copies),
            "isolated": _point(4096, 4096, 1, GROUP, iso, peaks),
            "chained": _point(4096, 4096, 1, GROUP, med, peaks), "chained_best_us": round(best, 2)}


def config4_section(peaks):
    """configs[3]: the Llama-2-70B MLP shapes over M = 1, 4, 8, 16 on both forced paths and as
    awq_linear dispatches them (graph of chained calls over rotating copies, median of 5)."""
    from paper_2306_00978_b200 import binding
    rows = []
    for name, K, N in synth.LLAMA2_70B_MLP:
        rp = RandomPacked(N, K, GROUP)
        for M in (1, 4, 8, 16):
            r = {"shape": f"{K}->{N}", "M": M}
            for label, path in (("gemv", binding.PATH_GEMV), ("gemm", binding.PATH_GEMM), ("auto", binding.PATH_AUTO)):
                _, med = rp.time_chained(M, path=path, calls=8)
                r[label] = _point(N, K, M, GROUP, med, peaks)
            rows.append(r)
        del rp
    return rows


def int3_section(peaks):
    """The layer on the 3-bit storage (band matrix-vector kernel, M = 1) next to the same shapes on
    the 4-bit layout: microseconds, algorithmic GB/s of each and the bytes saved."""
    import torch
    from paper_2306_00978_b200 import binding
    out = []
    for (K, N) in ((4096, 11008), (8192, 28672)):
        l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
        b3 = N * K * 3 // 8 + (N * K // GROUP) * 2 + (N * K // GROUP) // 2
        n = max(3, -(-2 * l2 // b3) + 1)
        copies = []
        for _ in range(n):
            q3 = torch.randint(0, 256, (N * K * 3 // 8,), dtype=torch.uint8, device="cuda")
            sc = (torch.rand((N // 16, K // GROUP, 16), device="cuda") * 0.01 + 0.001).half()
            zp = torch.randint(0, 120, (N // 32, K // GROUP, 16), dtype=torch.uint8, device="cuda")
            copies.append((q3, sc, zp))
        x = torch.randn((1, K), device="cuda").half()
        y = torch.empty((1, N), device="cuda", dtype=torch.float16)
        scratch = torch.empty(16, dtype=torch.uint8, device="cuda")
        for i in range(3):
            binding.linear_int3(x, *copies[i], N, K, GROUP, out=y, scratch=scratch)
        torch.cuda.synchronize()
        g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        calls = max(8, n)
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(calls):
                    binding.linear_int3(x, *copies[i % n], N, K, GROUP, out=y, scratch=scratch)
        torch.cuda.synchronize()
        g.replay()
        ts = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3 / calls)
        binding.poll_status()
        us3 = statistics.median(ts)
        del copies, g
        torch.cuda.empty_cache()
        rp = RandomPacked(N, K, GROUP)
        _, us4 = rp.time_chained(1)
        del rp
        torch.cuda.empty_cache()
        bytes3 = b3 + 2 * K + 2 * N
        bytes4 = algorithmic_bytes(N, K, 1)
        out.append({"shape": f"{K}->{N}", "M": 1, "int3_us": round(us3, 2), "int3_GBps": round(bytes3 / us3 / 1e3, 1),
                    "int3_frac_hbm_measured": round(bytes3 / us3 / 1e3 / peaks["hbm_gbs"], 4),
                    "int4_us": round(us4, 2), "int4_GBps": round(bytes4 / us4 / 1e3, 1),
                    "bytes_int3": bytes3, "bytes_int4": bytes4, "bytes_saved_frac": round(1 - bytes3 / bytes4, 4)})
    return out


SWEEP_SHAPES = (("q/k/v/o", 4096, 4096), ("gate/up", 4096, 11008), ("down", 11008, 4096))
SWEEP_M = (1, 2, 4, 8, 16, 32, 64, 128, 512, 2048, 8192)


def sweep_rows(peaks, groups=(128, 64), reps: int = 5):
    """configs[4]: the 7B layer's three distinct shapes x token counts 1 .. 8192 x both group sizes
    through awq_linear (alpha only changes the values of the packed arrays, not the run time: the
    sweep's parity over alpha in {0, 0.5, 1} is a test).  Cold-L2 rotation for M <= 128."""
    import torch
    for group in groups:
        for name, K, N in SWEEP_SHAPES:
            rp = RandomPacked(N, K, group)
            for M in SWEEP_M:
                best, med = rp.time_chained(M, reps=reps)
                row = {"shape": name, "K": K, "N": N, "group": group, "M": M}
                row.update(_point(N, K, M, group, best, peaks))
                row["us_median"] = round(med, 2)
                yield row
            del rp
            torch.cuda.empty_cache()


def quantize_only(args):
    """A small, self-contained run of the quantize+pack kernel for ncu captures."""
    import torch
    from paper_2306_00978_b200 import binding
    N, K = args.quantize_only
    W = torch.from_numpy(synth.weight(2004, N, K)).cuda()
    a = torch.from_numpy(synth.act_mean_abs(2004, K)).cuda()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(args.reps + 1):
        if r == args.reps:
            e0.record()
        binding.quantize_pack(W, a, ALPHA, GROUP)
    e1.record()
    torch.cuda.synchronize()
    nbytes = 2 * N * K + 4 * K + N * K // 2 + 2 * N * K // GROUP + N * K // (2 * GROUP)
    print(json.dumps({"quantize_only": [N, K], "us_last_launch": e0.elapsed_time(e1) * 1e3, "algorithmic_bytes": nbytes}))
    return 0


def sweep(args):
    """The full-shape sweep, one JSON object per line."""
    peaks = load_peaks()
    for row in sweep_rows(peaks):
        print(json.dumps(row), flush=True)
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
    ap.add_argument("--path", type=int, default=0, help="with --one: 0 auto, 1 GEMV, 2 GEMM, 3 split-K GEMV, 4 single-SM GEMM, 5 chunked GEMV, 6 chunked tensor-core")
    ap.add_argument("--reps", type=int, default=3, help="with --one: passes over the three copies")
    ap.add_argument("--quantize-only", nargs=2, type=int, metavar=("N", "K"),
                    help="profiling aid: a few awq_quantize_pack launches on seeded weights of one shape, then exit")
    ap.add_argument("--sweep", action="store_true",
                    help="per-shape table over the 7B layer shapes, M = 1 .. 8192, both group sizes; then exit")
    args = ap.parse_args()
    if args.one:
        return one_shape(args)
    if args.quantize_only:
        return quantize_only(args)
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
    # each operand once per matrix as in the roofline table, plus the inverse channel scales (fp32 [K])
    # that each of the four calls reads
    step_bytes = sum(algorithmic_bytes(l["N"], l["K"], 1) for l in layers[0]) + \
        sum(4 * layers[0][idxs[0]]["K"] for idxs in STEP_CALLS)
    packed_bytes = sum(l["qw"].numel() + l["sc"].numel() * 2 + l["zp"].numel() for l in layers[0])
    l2_bytes = torch.cuda.get_device_properties(local_rank).L2_cache_size

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    graph, launches_per_step = capture_chain(run_step, layers, steps)
    sec, spread, (w0, w1), R = timed_region(graph, steps, warmup, device)
    del graph
    e2e_graph = capture_chain_e2e(layers, steps)
    e2e_sec, e2e_spread, _, _ = timed_region(e2e_graph, steps, warmup, device, min_seconds=0.3, min_replays=20)
    del e2e_graph
    launches = launches_per_step * steps * R
    clocks = None
    if rank == 0:
        time.sleep(0.15)
        clocks = sampler.summary(w0, w1)
        clocks["note"] = f"sampled during the timed region ({w1 - w0:.2f} s)"
    binding.poll_status()
    pos_sec = per_position_times(layers) if rank == 0 else None

    value = replicas.aggregate_throughput(step_bytes, sec / steps) / 1e9
    e2e_value = replicas.aggregate_throughput(step_bytes, e2e_sec / steps) / 1e9
    achieved_step = step_bytes * steps / sec / 1e9      # one GPU's algorithmic GB/s over the region
    rotation = args.layers * packed_bytes
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": sec / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 x int4 -> f32", "data": "synthetic",
        "config": {"workload": "llama2-7b decoder-layer linears (q,k,v,o 4096->4096; gate,up 4096->11008; "
                               "down 11008->4096), M=1, g128, alpha=0.5",
                   "layers_rotated": args.layers, "packed_bytes_per_layer": packed_bytes,
                   "l2_policy": f"weights rotate over {args.layers} layers = {rotation / 1e6:.0f} MB, "
                                + ("more" if rotation > 2 * l2_bytes else "NOT more")
                                + f" than 2 x the {l2_bytes / 1e6:.0f} MB L2"
                                + ("" if rotation > 2 * l2_bytes else " (weights partly L2-resident: not a valid HBM figure)"),
                   "algorithmic_bytes_per_step": step_bytes, "parallelism": f"replicas x{world}",
                   "launch": "each step is 4 C-ABI calls: awq_linear_multi_scaled(q,k,v), awq_linear_scaled(o), "
                             "awq_linear_multi_scaled(gate,up), awq_linear_scaled(down) on the UNDIVIDED activations "
                             "(x / s is folded into the kernels: 4 launches per step); the `steps` steps (layers "
                             "rotating) are ONE CUDA graph, all launches chained by programmatic dependent launch",
                   "timing": f"the {steps}-step graph replayed {R} times, one CUDA event between replays; "
                             "ms_per_step = median replay time / steps"},
        "replay_seconds": spread,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": sum(2 * layers[0][idxs[0]]["K"] for idxs in STEP_CALLS),
                "d2h_bytes_per_step": sum(2 * l["N"] for l in layers[0]),
                "replays": e2e_spread["replays"],
                "note": "every step copies its activations in from pinned host memory and its outputs back inside "
                        "the timed region; the copies run on two copy streams of the same graph and overlap the "
                        "kernels of neighbouring steps"},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if rank == 0:
        # the dominant kernel: the K = 4096 instantiation of the band kernel serves three of the four
        # launch positions (q+k+v, o, gate+up) and most of the step's bytes and time
        pos_bytes = [sum(algorithmic_bytes(layers[0][i]["N"], layers[0][i]["K"], 1) for i in idxs)
                     - 2 * layers[0][idxs[0]]["K"] * (len(idxs) - 1) + 4 * layers[0][idxs[0]]["K"]
                     for idxs in STEP_CALLS]
        dom = [0, 1, 2]
        dom_bytes = sum(pos_bytes[i] for i in dom) / len(dom)
        dom_sec = sum(pos_sec[i] for i in dom) / len(dom)
        achieved = dom_bytes / dom_sec / 1e9
        line["roofline"] = {
            "bound": "hbm", "kernel": DOMINANT_KERNEL, "achieved": achieved,
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
            "peak_source": peaks["source"], "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
            "avg_launch_us": dom_sec * 1e6, "algorithmic_bytes_per_launch": dom_bytes,
            "how": "average over this kernel's three launch positions of the step (q+k+v, o, gate+up), each "
                   "timed with CUDA events on a graph that holds only that position, chained over the "
                   "rotating layers",
            "traffic": dom_bytes * NCU_TRAFFIC_RATIO,
            "traffic_note": NCU_TRAFFIC_NOTE,
            "per_position": [{"calls": "+".join(layers[0][i]["name"] for i in idxs), "us": pos_sec[k] * 1e6,
                              "algorithmic_bytes": pos_bytes[k], "GBps": pos_bytes[k] / pos_sec[k] / 1e9,
                              "frac": pos_bytes[k] / pos_sec[k] / 1e9 / peaks["hbm_gbs"]}
                             for k, idxs in enumerate(STEP_CALLS)],
            "step": {"achieved": achieved_step, "frac": achieved_step / peaks["hbm_gbs"],
                     "frac_of_nominal_8000": achieved_step / NOMINAL_HBM_GBS,
                     "sum_of_positions_us": sum(pos_sec) * 1e6}}
    if rank == 0 and not args.skip_extras:
        del layers
        torch.cuda.empty_cache()
        line["config1_single_linear"] = config1_section(peaks)
        line["config4_70b_mlp"] = config4_section(peaks)
        torch.cuda.empty_cache()
        rows = list(sweep_rows(peaks, reps=3))
        cols = ["shape", "group", "M", "us", "GBps", "TFLOPs"]
        line["config5_sweep"] = {"columns": cols, "rows": [[r[c] for c in cols] for r in rows],
                                 "note": "awq_linear, automatic dispatch, best of 3 graph replays; cold-L2 rotation "
                                         "for M <= 128; alpha does not enter the run time"}
        torch.cuda.empty_cache()
        line["int3_storage"] = int3_section(peaks)
        line["quantize_pack"] = quantize_section(peaks)
        line["alpha_search"] = search_section()
        line["clip_search"] = clip_section()
        # last of the GPU sections: its sustained leg runs the GPU into the power cap, and the SM
        # clock stays low for a while afterwards
        line["gemm_m2048"] = gemm_section(peaks, sampler)
        if world == 1:
            torch.cuda.empty_cache()
            line["cpu_baseline"] = cpu_baseline()
    if rank == 0:
        sampler.stop()
        print(json.dumps(line), flush=True)
    replicas.barrier()
    replicas.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
