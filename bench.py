#!/usr/bin/env python
"""Benchmark of the time-rotated quantized linear path on B200.

A step is one denoising step of the DiT workload: for each of the transformer blocks, each of its
quantized linears runs rotate + quantize and the INT8 GEMM with its epilogue (two kernels per
linear), at the time-step of that sampling step, so the timed run includes the group switches.
The default workload is the largest single-GPU 8-bit one (PixArt-style, M = 32768 plus the cross-attention
projections); the other workloads get short passes in the same run (`per_workload`).
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2503_06564_b200 import workloads as WL

METRIC = "rotated_w8a8_linear_tops"
UNIT = "TOPS"
# DRAM traffic per unit of algorithmic work, from the Nsight Compute captures summarised under profiles/
# (dram__bytes_read.sum + dram__bytes_write.sum of one launch); None once a kernel has changed since its capture.
GEMM_PAIR_DRAM_BYTES_PER_OP = 116.3e6 / 174.0e9     # gemm_w8a8_pair_kernel, M = 16384, K = 1152, N = 4608
RQ_TEAM_DRAM_BYTES_PER_ALG_BYTE = 659.6 / 793.3     # rotate_quantize_team_kernel, M = 32768: three K = 1152 launches and one K = 4608
INT8_OVER_BF16 = 2.0          # nominal dense INT8 : bf16 tensor throughput ratio (4.5 : 2.25 PFLOP/s)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def step_ops(wl: WL.Workload) -> float:
    """Integer operations (2 per multiply-add) of one denoising step."""
    total = 0.0
    for layer in wl.layers:
        total += 2.0 * wl.M * layer.N * layer.K
    for layer in wl.extra_layers:
        total += 2.0 * (layer.M or wl.M) * layer.N * layer.K
    return total * wl.blocks


def step_rq_bytes(wl: WL.Workload) -> float:
    """Algorithmic bytes of the rotate + quantize launches of one step: 3K + 4 per token."""
    total = 0.0
    for layer in wl.layers + wl.extra_layers:
        total += (layer.M or wl.M) * (3.0 * layer.K + 4.0)
    return total * wl.blocks


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.device_index = device_index
        self.proc = None
        self.path = os.path.join(tempfile.gettempdir(), f"trdq_bench_clocks_{os.getpid()}_{device_index}.csv")

    def start(self):
        try:
            os.makedirs(os.path.dirname(self.path), exist_ok=True)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.device_index)], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# device workload
# ------------------------------------------------------------------------------------------
def make_device_x(wl: WL.Workload, M: int, K: int, gen):
    """Activations drawn on the device with the recipe of workloads.make_x: N(0,1) bulk, 1 % of the
    channels heavy tailed (Student-t, nu = 3) or scaled, per the workload."""
    import torch
    x = torch.randn((M, K), generator=gen, device="cuda", dtype=torch.float32)
    n_out = int(np.ceil(0.01 * K))
    ch = torch.randperm(K, generator=gen, device="cuda")[:n_out]
    if wl.outlier == "student_t3":
        z = torch.randn((M, n_out), generator=gen, device="cuda")
        chi2 = (torch.randn((M, n_out, 3), generator=gen, device="cuda") ** 2).sum(-1)
        x[:, ch] = z / torch.sqrt(chi2 / 3.0)
    elif wl.outlier == "scale30":
        x[:, ch] *= 30.0
    elif wl.outlier == "fixed50":
        x[:, ch] *= 50.0
    return x.to(torch.bfloat16)


def build_device_workload(wl: WL.Workload, seed: int, blocks: int, rotation: str = "hadamard"):
    """Distinct weights, activations and outputs for every linear of every block, so that one step
    streams a working set far larger than L2."""
    import torch
    from paper_2503_06564_b200 import trdq
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    layers = trdq.LayerList()
    alphas = WL.group_alphas(wl.num_groups)
    rng = np.random.default_rng(seed)
    dense_blocks = {}
    for b in range(blocks):
        for layer in wl.layers + wl.extra_layers:
            M = layer.M or wl.M
            w = (torch.randn((layer.N, layer.K), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
            x = make_device_x(wl, M, layer.K, gen)
            bias = (torch.randn((layer.N,), generator=gen, device="cuda") * 0.01).to(torch.bfloat16)
            ax = x.abs().amax(dim=0).double().clamp_min(1e-5).cpu().numpy()
            aw = w.abs().amax(dim=0).double().clamp_min(1e-5).cpu().numpy()
            smooth = np.stack([1.0 / (ax ** a / aw ** (1.0 - a)) for a in alphas]).astype(np.float32)
            ws = None
            if rotation == "dense":
                # Eq. 6-8: dense 128 x 128 orthogonal blocks per group (random ones stand in for calibrated products; one set
                # per C_in is reused by every layer of that width, each layer still folds in its own smoothing vector)
                if layer.K not in dense_blocks:
                    blk = np.empty((wl.num_groups, layer.K // 128, 128, 128), np.float32)
                    for g in range(wl.num_groups):
                        for j in range(layer.K // 128):
                            blk[g, j] = np.linalg.qr(rng.standard_normal((128, 128)))[0]
                    dense_blocks[layer.K] = blk
                rot = trdq.DenseRotation(layer.K, wl.t_bounds, dense_blocks[layer.K], smooth)
                ws = torch.empty((trdq.trdq_rotate_dense_workspace(rot, M),), dtype=torch.uint8, device="cuda")
            else:
                signs = (rng.integers(0, 2, (wl.num_groups, layer.K)) * 2 - 1).astype(np.int8)
                rot = trdq.Rotation(layer.K, wl.t_bounds, signs, smooth)
            wts = trdq.trdq_prepare_weights(rot, w, wl.wbits)
            codes = torch.empty((M, layer.K), dtype=torch.int8, device="cuda")
            scales = torch.empty((M,), dtype=torch.float32, device="cuda")
            y = torch.empty((M, layer.N), dtype=torch.bfloat16, device="cuda")
            layers.add(rot, wts, x, codes, scales, bias, y, workspace=ws)
            del w
    torch.cuda.synchronize()
    return layers


def time_region(fn, steps: int):
    """CUDA-event time (ms) of `steps` calls of fn(i) on the current stream, synchronised on both sides."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


class KernelPass:
    """One step's launches of ONE kernel kind (rotate + quantize, or GEMM + epilogue) captured in a CUDA graph, so that
    the launches run back to back on the device."""

    def __init__(self, layers, wl, which: str):
        import torch
        from paper_2503_06564_b200 import trdq
        t = int(wl.timesteps()[0])
        keep = layers._keep

        def issue():
            for (rot, w, x, codes, scales, bias, y), ws in zip(keep, layers._extra):
                if which == "rq" and ws is not None:
                    trdq.trdq_rotate_dense_quantize(rot, t, x, codes, scales, ws)
                elif which == "rq":
                    trdq.trdq_rotate_quantize(rot, t, x, codes, scales)
                else:
                    trdq.trdq_linear(w, t, codes, scales, bias, y)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            issue()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph, capture_error_mode="thread_local"):
            issue()
        for _ in range(3):
            self.graph.replay()
        torch.cuda.synchronize()

    @classmethod
    def per_layer_us(cls, layers, wl, reps: int = 5):
        """Microseconds per launch of each layer of a block, both kernel kinds: the launches of that layer over all blocks
        (distinct buffers) replayed back to back from a graph."""
        import torch
        from paper_2503_06564_b200 import trdq
        t = int(wl.timesteps()[0])
        per_block = len(wl.layers + wl.extra_layers)
        out = []
        for j, layer in enumerate(wl.layers + wl.extra_layers):
            entry = {"layer": layer.name}
            for which in ("rq", "gemm"):
                self = cls.__new__(cls)
                sel = [(k, ws) for i, (k, ws) in enumerate(zip(layers._keep, layers._extra)) if i % per_block == j]

                def issue():
                    for (rot, w, x, codes, scales, bias, y), ws in sel:
                        if which == "rq" and ws is not None:
                            trdq.trdq_rotate_dense_quantize(rot, t, x, codes, scales, ws)
                        elif which == "rq":
                            trdq.trdq_rotate_quantize(rot, t, x, codes, scales)
                        else:
                            trdq.trdq_linear(w, t, codes, scales, bias, y)

                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, capture_error_mode="thread_local"):
                    issue()
                ms, _ = self.ms(reps=reps)
                us = ms * 1e3 / len(sel)
                m = layer.M or wl.M
                if which == "rq":
                    entry["rotate_quantize_us"] = us
                    entry["rotate_quantize_gbs"] = m * (3.0 * layer.K + 4.0) / (us * 1e-6) / 1e9
                else:
                    entry["linear_us"] = us
                    entry["linear_tops"] = 2.0 * m * layer.N * layer.K / (us * 1e-6) / 1e12
            out.append(entry)
        return out

    def ms(self, reps: int = 0, min_seconds: float = 0.0):
        """(ms per pass, seconds timed): `reps` passes, or as many as fill `min_seconds`; a tenth of them untimed first."""
        once = time_region(lambda i: self.graph.replay(), 3) / 3
        if min_seconds > 0.0:
            reps = max(reps, int(np.ceil(1.1 * min_seconds * 1e3 / max(once, 1e-6))))
        reps = max(reps, 3)
        for _ in range(max(3, reps // 10)):
            self.graph.replay()
        total = time_region(lambda i: self.graph.replay(), reps)
        if min_seconds > 0.0 and total * 1e-3 < min_seconds:      # the first estimate was taken at other clocks
            reps = int(np.ceil(reps * 1.2 * min_seconds / (total * 1e-3)))
            total = time_region(lambda i: self.graph.replay(), reps)
        return total / reps, total * 1e-3


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------
def oracle_block_inputs(wl: WL.Workload, rows: int):
    """Inputs of the linears of ONE transformer block, `rows` tokens each, with the oracle's own
    (untimed, offline) weight preparation for the first time-step's group."""
    from oracle import trdq_oracle as O
    t = int(wl.timesteps()[0])
    g = O.group_of(wl.t_bounds, t)
    items = []
    for li, layer in enumerate(wl.layers + wl.extra_layers):
        m = min(rows, layer.M or wl.M)
        inp = WL.make_layer_inputs(wl, li, M=m)
        act, wv = O.fused_vectors(inp.signs[g], None if inp.smooth is None else inp.smooth[g])
        if wl.wbits == 8:
            qw, sw = O.prepare_w8(inp.w, wv)
        else:
            qw, sw = O.prepare_w4(inp.w, wv)
        items.append((inp, act, qw, sw, m))
    return items


def oracle_block_seconds(wl: WL.Workload, items) -> float:
    """Wall time of the oracle's online path (rotate + quantize, integer GEMM, epilogue) on the block."""
    from oracle import trdq_oracle as O
    t0 = time.perf_counter()
    for inp, act, qw, sw, m in items:
        q, sx = O.rotate_quantize(inp.x, act)
        rows = np.arange(m)
        if wl.wbits == 8:
            O.linear_w8_rows(q, sx, qw, sw, inp.bias, rows)
        else:
            O.linear_w4_rows(q, sx, qw, sw, inp.bias, rows)
    return time.perf_counter() - t0


def block_ops(wl: WL.Workload, rows: int) -> float:
    return sum(2.0 * min(rows, l.M or wl.M) * l.N * l.K for l in wl.layers + wl.extra_layers)


def run_reference(args, wl: WL.Workload):
    """`--impl reference`: the CPU oracle on this host, each step a bounded sample of the workload."""
    from oracle import trdq_oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total_steps = args.steps + args.warmup
    cal_rows = 16
    cal = oracle_block_inputs(wl, cal_rows)
    oracle_block_seconds(wl, cal)
    per_row = oracle_block_seconds(wl, cal) / cal_rows
    budget = 120.0 / max(total_steps, 1)
    rows = int(max(8, min(wl.M, budget / max(per_row, 1e-9))))
    items = oracle_block_inputs(wl, rows)
    for _ in range(args.warmup):
        oracle_block_seconds(wl, items)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_block_seconds(wl, items)
    sec = time.perf_counter() - t0
    tops = block_ops(wl, rows) * args.steps / sec / 1e12
    sample = f"each step = 1 of {wl.blocks} blocks, first {rows} of {wl.M} token rows, on host cores"
    line = {"impl": "reference", "metric": METRIC, "value": tops, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec / max(args.steps, 1) * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": wl.name, "M": wl.M, "blocks": wl.blocks, "sample": sample},
            "cpu_baseline": {"value": tops, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": tops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------
NOMINAL_INT8_TOPS = 4500.0     # dense INT8, public figure for the part
NOMINAL_HBM_GBS = 8000.0


def peak_for(peaks, seconds: float):
    """Tensor-core denominator by the length of the timed region: the burst figure for a region under a second, the
    sustained (power-capped) one for a region of two seconds or more; in between, the burst figure (the harder one)."""
    if seconds >= 2.0:
        return peaks["bf16_tflops_sustained"] * INT8_OVER_BF16, "sustained"
    return peaks["bf16_tflops"] * INT8_OVER_BF16, "burst"


def kernel_names(wl: WL.Workload):
    """Kernel the library runs per layer (asked from the library itself), and for each stage the kernel that does
    most of the work of a step."""
    from paper_2503_06564_b200 import trdq
    rq, gemm, per_layer = {}, {}, []
    for layer in wl.layers + wl.extra_layers:
        m = layer.M or wl.M
        a = trdq.trdq_kernel_choice(0, m, layer.K)
        b = trdq.trdq_kernel_choice(1, m, layer.K, layer.N, wl.wbits)
        per_layer.append({"layer": layer.name, "M": m, "K": layer.K, "N": layer.N, "rotate_quantize": a, "linear": b})
        rq[a] = rq.get(a, 0.0) + m * (3.0 * layer.K + 4.0)
        b0 = b.split("<")[0]
        gemm[b0] = gemm.get(b0, 0.0) + 2.0 * m * layer.N * layer.K
    return max(rq, key=rq.get), max(gemm, key=gemm.get), per_layer


def roofline_entries(wl, peaks, ops, ms_gemm, sec_gemm, ms_rq, sec_rq, dense=False):
    rq_kernel, gemm_kernel, per_layer = kernel_names(wl)
    if dense:
        rq_kernel = "rotate_dense_amax_kernel+rotate_dense_quantize_kernel"
    int8_peak, which = peak_for(peaks, sec_gemm)
    gemm_tops = ops / (ms_gemm * 1e-3) / 1e12
    rq_gbs = step_rq_bytes(wl) / (ms_rq * 1e-3) / 1e9
    n_ops = len(wl.layers + wl.extra_layers) * wl.blocks
    gemm = {"kernel": gemm_kernel, "bound": "tensor", "achieved": gemm_tops, "peak": int8_peak, "unit": "TOPS",
            "frac": gemm_tops / int8_peak, "frac_nominal": gemm_tops / NOMINAL_INT8_TOPS, "seconds_timed": sec_gemm,
            "peak_source": f"{peaks['_source']} {which} bf16 {int8_peak / INT8_OVER_BF16:.1f} TFLOP/s x {INT8_OVER_BF16:g} (nominal int8:bf16); "
                           f"nominal {NOMINAL_INT8_TOPS:g} TOPS",
            "traffic": (GEMM_PAIR_DRAM_BYTES_PER_OP * ops / n_ops) if gemm_kernel == "gemm_w8a8_pair_kernel" else None,
            "traffic_note": "bytes per launch, scaled by operations from the capture in profiles/gemm_w8a8_pair_*.txt to an average launch of this workload"}
    rq = {"kernel": rq_kernel, "bound": "hbm", "achieved": rq_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
          "frac": rq_gbs / peaks["hbm_gbs"], "frac_nominal": rq_gbs / NOMINAL_HBM_GBS, "seconds_timed": sec_rq,
          "peak_source": f"{peaks['_source']} copy rate; nominal {NOMINAL_HBM_GBS:g} GB/s",
          "traffic": RQ_TEAM_DRAM_BYTES_PER_ALG_BYTE * step_rq_bytes(wl) / n_ops
          if (rq_kernel == "rotate_quantize_team_kernel" and RQ_TEAM_DRAM_BYTES_PER_ALG_BYTE) else None,
          "traffic_note": "bytes per launch, scaled by algorithmic bytes from the capture in profiles/rotate_quantize_team_*.txt"}
    return gemm, rq, per_layer


class DeviceRun:
    """A workload resident on the device with its per-group CUDA graphs."""

    def __init__(self, wl, args, rank):
        import torch
        from paper_2503_06564_b200 import trdq
        self.wl = wl
        self.layers = build_device_workload(wl, seed=1234 + rank, blocks=wl.blocks, rotation=args.rotation)
        self.ts = wl.timesteps()
        layers, ts = self.layers, self.ts
        for i in range(3):
            trdq.trdq_run_layers(layers, int(ts[i % len(ts)]))
        torch.cuda.synchronize()
        assert trdq.trdq_device_status() == 0
        # One CUDA graph per time-step group (the kernels of a step depend on t only through its group: a group switch
        # is a switch of graph); the step of the sampling loop replays the graph of its group.
        self.graphs = {}
        if not args.no_graph:
            side = torch.cuda.Stream()
            for t in ts:
                g = trdq.trdq_find_group(wl.t_bounds, int(t))
                if g in self.graphs:
                    continue
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    trdq.trdq_run_layers(layers, int(t))
                torch.cuda.current_stream().wait_stream(side)
                torch.cuda.synchronize()
                self.graphs[g] = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graphs[g], capture_error_mode="thread_local"):
                    trdq.trdq_run_layers(layers, int(t))
            self.groups_of_steps = [trdq.trdq_find_group(wl.t_bounds, int(t)) for t in ts]

    def step(self, i):
        from paper_2503_06564_b200 import trdq
        if self.graphs:
            self.graphs[self.groups_of_steps[i % len(self.ts)]].replay()
        else:
            trdq.trdq_run_layers(self.layers, int(self.ts[i % len(self.ts)]))


def measure_side_workload(wl, args, rank, peaks):
    """Short passes of a workload other than the headline one: step time, both kernel classes, clocks."""
    import torch
    from paper_2503_06564_b200 import trdq
    run = DeviceRun(wl, args, rank)
    for i in range(3):
        run.step(i)
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    steps = max(5, min(args.steps, 20)) if wl.index != 0 else 200
    ms = time_region(run.step, steps) / steps
    ms_rq, sec_rq = KernelPass(run.layers, wl, "rq").ms(reps=steps)
    gemm_pass = KernelPass(run.layers, wl, "gemm")
    ms_gemm, sec_gemm = gemm_pass.ms(reps=steps)
    clocks = sampler.stop()
    long_gemm = None
    if wl.M >= 16384 and wl.wbits == 8 and not args.quick:
        # the large launches are power-limited: also a two-second pass against the sustained peak
        ms_l, sec_l = gemm_pass.ms(min_seconds=2.0)
        long_gemm = roofline_entries(wl, peaks, step_ops(wl), ms_l, sec_l, ms_rq, sec_rq)[0]
    assert trdq.trdq_device_status() == 0
    ops = step_ops(wl)
    gemm, rq, _ = roofline_entries(wl, peaks, ops, ms_gemm, sec_gemm, ms_rq, sec_rq)
    for d in (gemm, rq):
        for k in ("traffic", "traffic_note", "peak_source", "bound", "unit"):
            d.pop(k, None)
    out = {"workload": wl.name, "M": wl.M, "wbits": wl.wbits, "steps": steps, "ms_per_step": ms, "us_per_dit_step": ms * 1e3,
           "tops": ops / (ms * 1e-3) / 1e12, "kernel_ms_per_step": {"rotate_quantize": ms_rq, "gemm_epilogue": ms_gemm},
           "gemm": gemm, "rotate_quantize": rq, "clocks": clocks}
    if long_gemm is not None:
        out["gemm_sustained"] = {k: long_gemm[k] for k in ("achieved", "peak", "frac", "frac_nominal", "seconds_timed")}
    del run
    torch.cuda.empty_cache()
    return out


def gpu_parity_and_cpu_baseline(wl: WL.Workload, budget_s: float = 20.0):
    """The cpu_baseline leg: the oracle as it stands, timed on this host's cores on a bounded sample of the workload's
    own seeded inputs (whole blocks of the step, or one block with as many token rows as fit the budget) - and, since it
    has then computed those rows, the same inputs are run through the library in the launch configuration the benchmark
    times (trdq_run_layers) and compared: activation codes and scales bit for bit, outputs in bf16 steps."""
    import torch
    from oracle import trdq_oracle as O
    from paper_2503_06564_b200 import trdq
    cal_rows = 32
    cal = oracle_block_inputs(wl, cal_rows)
    oracle_block_seconds(wl, cal)                                  # warm the thread pool
    per_row = oracle_block_seconds(wl, cal) / cal_rows
    rows = int(max(cal_rows, min(wl.M, budget_s / max(per_row, 1e-9))))
    items = oracle_block_inputs(wl, rows)
    t = int(wl.timesteps()[0])
    t0 = time.perf_counter()
    refs = []
    for inp, act, qw, sw, m in items:
        q, sx = O.rotate_quantize(inp.x, act)
        idx = np.arange(m)
        y = O.linear_w8_rows(q, sx, qw, sw, inp.bias, idx) if wl.wbits == 8 else O.linear_w4_rows(q, sx, qw, sw, inp.bias, idx)
        refs.append((q, sx, y))
    sec = time.perf_counter() - t0
    blocks_done = 1
    while sec < 10.0 and blocks_done < wl.blocks:
        sec += oracle_block_seconds(wl, items)
        blocks_done += 1
    tops = blocks_done * block_ops(wl, rows) / sec / 1e12
    baseline = {"value": tops, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                "sample": f"{blocks_done} of {wl.blocks} blocks ({len(items)} linears each), first {rows} of {wl.M} token rows, {sec:.2f} s"}

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()

    layers, outs = trdq.LayerList(), []
    for inp, act, qw, sw, m in items:
        rot = trdq.Rotation(inp.layer.K, inp.t_bounds, inp.signs, inp.smooth)
        wts = trdq.trdq_prepare_weights(rot, dev(inp.w), wl.wbits)
        codes = torch.empty((m, inp.layer.K), dtype=torch.int8, device="cuda")
        scales = torch.empty((m,), dtype=torch.float32, device="cuda")
        y = torch.empty((m, inp.layer.N), dtype=torch.bfloat16, device="cuda")
        layers.add(rot, wts, dev(inp.x), codes, scales, dev(inp.bias), y)
        outs.append((codes, scales, y))
    trdq.trdq_run_layers(layers, t)
    torch.cuda.synchronize()
    codes_equal, scales_equal, max_steps, worst_l2, n_out = True, True, 0.0, 0.0, 0
    for (q, sx, y_ref), (codes, scales, y) in zip(refs, outs):
        codes_equal &= bool(np.array_equal(codes.cpu().numpy(), q))
        scales_equal &= bool(np.array_equal(scales.cpu().numpy(), sx))
        y_gpu = WL.bf16_bits_to_f32(y.view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
        err = np.abs(y_gpu - y_ref)
        _, e = np.frexp(np.abs(y_ref).astype(np.float64))
        max_steps = max(max_steps, float((err / np.ldexp(1.0, np.maximum(e - 8, -133))).max()))
        worst_l2 = max(worst_l2, float(np.sqrt((err ** 2).sum() / max((y_ref.astype(np.float64) ** 2).sum(), 1e-300))))
        n_out += y_ref.size
    parity = {"against": "oracle", "launch": "trdq_run_layers", "linears": len(items), "rows": rows, "outputs": n_out,
              "codes_bit_exact": codes_equal, "scales_bit_exact": scales_equal, "max_bf16_steps": max_steps, "rel_l2": worst_l2,
              "ok": bool(codes_equal and scales_equal and max_steps <= 2.0 and worst_l2 <= 2e-3)}
    return baseline, parity


def run_ours(args, wl: WL.Workload):
    import torch
    import torch.distributed as dist
    from paper_2503_06564_b200 import build as lib_build, microbench, multirank, trdq

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()
    trdq.lib()                                   # fails loudly if the CUDA library is missing
    peaks = load_peaks()

    # weak scaling: every rank runs the whole workload on its own batch (rows are independent; no collective)
    run = DeviceRun(wl, args, rank)
    layers, ts, n_ops = run.layers, run.ts, len(run.layers)
    step = run.step
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    if world > 1:
        dist.barrier()
    ms = time_region(step, args.steps)
    ms = multirank.max_over_ranks(ms, device="cuda")
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ops = step_ops(wl)
    ms_per_step = ms / args.steps
    value = world * ops / (ms_per_step * 1e-3) / 1e12

    # Per-kernel passes on the same buffers, launches back to back from a CUDA graph: once for at least two seconds (the
    # part settles under its power cap: compared with the sustained peak) and once briefly (compared with the burst peak).
    dense = args.rotation == "dense"
    long_s = 0.0 if args.quick else 2.0
    sampler2 = ClockSampler(local_rank)
    sampler2.start()
    gemm_pass, rq_pass = KernelPass(layers, wl, "gemm"), KernelPass(layers, wl, "rq")
    ms_gemm, sec_gemm = gemm_pass.ms(reps=3, min_seconds=long_s)
    ms_rq, sec_rq = rq_pass.ms(reps=3, min_seconds=long_s)
    reps_long = max(args.steps, int(np.ceil(long_s * 1e3 / ms_per_step)))
    ms_sustained = time_region(step, reps_long) / reps_long
    clocks_sustained = sampler2.stop()
    # brief passes (a few tenths of a second each, after a pause): compared with the burst peak
    time.sleep(0.0 if args.quick else 1.0)
    ms_gemm_b, sec_gemm_b = gemm_pass.ms(min_seconds=0.25)
    time.sleep(0.0 if args.quick else 1.0)
    ms_rq_b, sec_rq_b = rq_pass.ms(min_seconds=0.25)
    assert trdq.trdq_device_status() == 0, "a bounded device-side wait expired during the benchmark"
    # GEMM: the two-second pass against the sustained tensor peak is the headline, the brief pass against the burst peak
    # beside it.  Rotate + quantize: the one measured copy rate is a best-of-ten of millisecond copies, i.e. a burst
    # figure, so the brief pass is the like-for-like headline and the two-second pass is reported beside it.
    roof_gemm, rq_long, per_layer = roofline_entries(wl, peaks, ops, ms_gemm, sec_gemm, ms_rq, sec_rq, dense)
    burst_gemm, roof_rq, _ = roofline_entries(wl, peaks, ops, ms_gemm_b, sec_gemm_b, ms_rq_b, sec_rq_b, dense)
    roof_gemm["brief"] = {k: burst_gemm[k] for k in ("achieved", "peak", "frac", "frac_nominal", "seconds_timed", "peak_source")}
    roof_rq["sustained"] = {k: rq_long[k] for k in ("achieved", "frac", "frac_nominal", "seconds_timed")}
    roof_rq["peak_source"] += " (best of ten 4 GB copies: a burst figure, compared with the brief pass)"
    per_layer_clocks = None
    if rank == 0:   # per-layer passes: microseconds per launch of every layer shape, in the state the long passes left the part in
        sampler3 = ClockSampler(local_rank)
        sampler3.start()
        for entry, timing in zip(per_layer, KernelPass.per_layer_us(layers, wl, reps=10)):
            entry.update({k: v for k, v in timing.items() if k != "layer"})
        per_layer_clocks = sampler3.stop()
    ceiling = None
    if rank == 0 and wl.wbits == 8:
        c = microbench.mma_ceiling(65536, 5)
        ceiling = {"kernel": c["kernel"], "tops": c["rate_best"], "what": "back-to-back 256x256x32 int8 MMAs per CTA pair on resident operands"}
        roof_gemm["frac_of_mma_ceiling"] = roof_gemm["achieved"] / c["rate_best"]

    # end to end through the public call with host buffers: H2D of every X, the step, D2H of every Y.  The pinned host
    # buffers hold ONE transformer block's tensors and serve every block (the bytes moved are those of the whole step).
    e2e_steps = max(1, min(args.steps, 3))
    per_block = len(wl.layers + wl.extra_layers)
    host_x = [torch.empty(k[2].shape, dtype=k[2].dtype).pin_memory() for k in layers._keep[:per_block]]
    host_y = [torch.empty(k[6].shape, dtype=k[6].dtype).pin_memory() for k in layers._keep[:per_block]]
    for hx, k in zip(host_x, layers._keep):
        hx.copy_(k[2])
    h2d = sum(k[2].numel() * k[2].element_size() for k in layers._keep)
    d2h = sum(k[6].numel() * k[6].element_size() for k in layers._keep)

    # Copies and kernels are pipelined layer by layer over three streams (PCIe carries both directions at once): layer i's
    # kernels wait for its input copy, its output copy waits for its kernels; across steps a buffer is not overwritten before
    # its reader of the step before has finished.
    s_main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(n_ops)]
    ev_done = [torch.cuda.Event() for _ in range(n_ops)]
    ev_out = [torch.cuda.Event() for _ in range(n_ops)]
    first_e2e = [True]

    def e2e_step(i):
        t = int(ts[i % len(ts)])
        s_in.wait_stream(s_main)        # buffers written before this step (warm-up, the step before) are complete
        s_out.wait_stream(s_main)
        for j, k in enumerate(layers._keep):
            hx, hy = host_x[j % per_block], host_y[j % per_block]
            with torch.cuda.stream(s_in):
                if not first_e2e[0]:
                    s_in.wait_event(ev_done[j])       # the step before has read X_j
                k[2].copy_(hx, non_blocking=True)
                ev_in[j].record(s_in)
            s_main.wait_event(ev_in[j])
            if not first_e2e[0]:
                s_main.wait_event(ev_out[j])          # the step before has copied Y_j out
            trdq.trdq_run_layers(layers, t, first=j, count=1)
            ev_done[j].record(s_main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[j])
                hy.copy_(k[6], non_blocking=True)
                ev_out[j].record(s_out)
        first_e2e[0] = False
        s_main.wait_stream(s_in)
        s_main.wait_stream(s_out)       # the step's results are on the host when the timed region ends

    e2e_step(0)
    ms_e2e = time_region(e2e_step, e2e_steps) / e2e_steps
    ms_e2e = multirank.max_over_ranks(ms_e2e, device="cuda")
    assert trdq.trdq_device_status() == 0

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8" if wl.wbits == 8 else "int8xint4", "data": "synthetic",
        "config": {"workload": wl.name, "M": wl.M, "blocks": wl.blocks, "linears_per_step": n_ops, "groups": wl.num_groups,
                   "sampling_steps": wl.steps, "wbits": wl.wbits, "parallelism": f"replicas x{world} (rows independent)",
                   "rotation": args.rotation, "launch": "host" if args.no_graph else "one CUDA graph per time-step group",
                   "l2": "inputs larger than L2: every linear has its own X, codes, Y and weights"},
        "us_per_dit_step": ms_per_step * 1e3,
        "rotate_quantize_gbs": roof_rq["achieved"],
        "gemm_tops": roof_gemm["achieved"],
        "kernel_ms_per_step": {"rotate_quantize": ms_rq, "gemm_epilogue": ms_gemm, "what": "two-second passes of one kernel kind",
                               "brief": {"rotate_quantize": ms_rq_b, "gemm_epilogue": ms_gemm_b}},
        "sustained": {"ms_per_step": ms_sustained, "steps": reps_long, "tops": ops / (ms_sustained * 1e-3) / 1e12,
                      "clocks": clocks_sustained, "what": "the same step loop run for at least two seconds, after the per-kernel passes"},
        "roofline": roof_gemm,
        "roofline_rotate_quantize": roof_rq,
        "mma_ceiling": ceiling,
        "kernels_per_layer": per_layer,
        "kernels_per_layer_note": "us per launch: that layer's launches over all blocks replayed from a graph, ten times, right after the "
                                  "two-second passes (the part is still at its power-capped clocks)",
        "kernels_per_layer_clocks": per_layer_clocks,
        "e2e": {"value": world * ops / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": e2e_steps},
        "gpu_launches": (3 if dense else 2) * n_ops * args.steps,
        "clocks": clocks,
    }
    del run, layers, gemm_pass, rq_pass, host_x, host_y, step
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not dense:
        if not args.no_per_workload:
            line["per_workload"] = [measure_side_workload(w2, args, rank, peaks) for w2 in WL.WORKLOADS if w2.index != wl.index]
        if not args.no_cpu_baseline:
            line["cpu_baseline"], line["parity"] = gpu_parity_and_cpu_baseline(wl)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3,
                    help="index into the workload list; default 3 = PixArt-style 1024 px, M = 32768 plus cross-attention, the largest "
                         "single-GPU 8-bit configuration (1 = DiT-XL/2 256 px, 2 = 512 px, 4 = video DiT W4A8, 0 = single layer)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle leg (CPU baseline and the parity check that rides on it)")
    ap.add_argument("--no-per-workload", action="store_true", help="skip the short passes over the other workloads")
    ap.add_argument("--quick", action="store_true", help="no two-second passes (development runs)")
    ap.add_argument("--no-graph", action="store_true", help="issue every step's launches from the host instead of replaying one CUDA graph per time-step group")
    ap.add_argument("--rotation", default="hadamard", choices=["hadamard", "dense"],
                    help="hadamard: the headline path; dense: dense 128 x 128 blocks on the tensor cores (Eq. 6-8), no CPU baseline")
    args = ap.parse_args()
    wl = WL.WORKLOADS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for several GPUs outside a launcher: start one process per GPU here (rank 0 prints the line)
        from paper_2503_06564_b200 import multirank
        rc, out = multirank.spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:])
        sys.stdout.write(out)
        sys.stdout.flush()
        sys.exit(rc)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
