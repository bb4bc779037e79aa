#!/usr/bin/env python
"""Benchmark of the time-rotated quantized linear path on B200.

A step is one denoising step of the DiT workload: for each of the transformer blocks, each of its
quantized linears runs rotate + quantize and the INT8 GEMM with its epilogue (two kernels per
linear), at the time-step of that sampling step, so the timed run includes the group switches.
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
GEMM_PAIR_DRAM_BYTES_PER_OP = 123.3e6 / 174.0e9     # gemm_w8a8_pair_kernel, M = 16384, K = 1152, N = 4608
RQ_TMA_DRAM_BYTES_PER_ALG_BYTE = 191.7 / 226.6      # rotate_quantize_tma_kernel, M = 65536, K = 1152
RQ_ROWS_DRAM_BYTES_PER_ALG_BYTE = 20.8 / 31.1       # rotate_quantize_rows_kernel, M = 9000, K = 1152
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


def kernel_pass_ms(layers, wl, which: str, reps: int):
    """Average time (ms) of one step's launches of ONE kernel kind, replayed from a CUDA graph so the
    launches are back to back.  which = 'rq' (rotate + quantize) or 'gemm' (GEMM + epilogue)."""
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
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, capture_error_mode="thread_local"):
        issue()
    for _ in range(3):
        graph.replay()
    ms = time_region(lambda i: graph.replay(), reps)
    return ms / reps


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


def cpu_baseline(wl: WL.Workload, budget_s: float = 20.0):
    """The oracle as it stands on this host's cores, on a bounded sample: whole blocks of the step (or, for the large
    workloads, one block with as many token rows as fit the time budget, calibrated on 32 rows first)."""
    from oracle import trdq_oracle as O
    cal_rows = 32
    cal = oracle_block_inputs(wl, cal_rows)
    oracle_block_seconds(wl, cal)                                  # warm the thread pool
    per_row = oracle_block_seconds(wl, cal) / cal_rows
    rows = int(max(cal_rows, min(wl.M, budget_s / max(per_row, 1e-9))))
    items = oracle_block_inputs(wl, rows)
    sec = oracle_block_seconds(wl, items)
    # when a whole block takes only a second or two, go through more of the step's (identically shaped) blocks: 10 - 30 s in all
    blocks_done = 1
    while sec < 10.0 and blocks_done < wl.blocks:
        sec += oracle_block_seconds(wl, items)
        blocks_done += 1
    tops = blocks_done * block_ops(wl, rows) / sec / 1e12
    return {"value": tops, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": f"{blocks_done} of {wl.blocks} blocks ({len(items)} linears each), first {rows} of {wl.M} token rows, {sec:.2f} s"}


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
def run_ours(args, wl: WL.Workload):
    import torch
    import torch.distributed as dist
    from paper_2503_06564_b200 import build as lib_build, multirank, trdq

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

    # weak scaling: every rank runs the whole workload on its own batch (rows are independent; no collective)
    layers = build_device_workload(wl, seed=1234 + rank, blocks=wl.blocks, rotation=args.rotation)
    ts = wl.timesteps()
    n_ops = len(layers)

    def step_direct(i):
        trdq.trdq_run_layers(layers, int(ts[i % len(ts)]))

    for i in range(max(args.warmup, 3)):
        step_direct(i)
    torch.cuda.synchronize()
    assert trdq.trdq_device_status() == 0

    # One CUDA graph per time-step group (the kernels of a step depend on t only through its group: a group switch is a
    # switch of graph); the step of the sampling loop replays the graph of its group.
    graphs = {}
    if not args.no_graph:
        side = torch.cuda.Stream()
        for t in ts:
            g = trdq.trdq_find_group(wl.t_bounds, int(t))
            if g in graphs:
                continue
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                trdq.trdq_run_layers(layers, int(t))
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graphs[g] = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graphs[g], capture_error_mode="thread_local"):
                trdq.trdq_run_layers(layers, int(t))
        groups_of_steps = [trdq.trdq_find_group(wl.t_bounds, int(t)) for t in ts]

    def step(i):
        if graphs:
            graphs[groups_of_steps[i % len(ts)]].replay()
        else:
            step_direct(i)

    for i in range(3):
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
    # per-kernel passes (same buffers, launches back to back from a CUDA graph)
    reps = max(3, min(args.steps, 20))
    ms_rq = kernel_pass_ms(layers, wl, "rq", reps)
    ms_gemm = kernel_pass_ms(layers, wl, "gemm", reps)
    clocks = sampler.stop()
    assert trdq.trdq_device_status() == 0, "a bounded device-side wait expired during the benchmark"

    ops = step_ops(wl)
    ms_per_step = ms / args.steps
    value = world * ops / (ms_per_step * 1e-3) / 1e12

    # end to end through the public call with host buffers: H2D of every X, the step, D2H of every Y
    e2e_steps = max(1, min(args.steps, 3))
    host_x = [torch.empty(k[2].shape, dtype=k[2].dtype).pin_memory() for k in layers._keep]
    host_y = [torch.empty(k[6].shape, dtype=k[6].dtype).pin_memory() for k in layers._keep]
    for hx, k in zip(host_x, layers._keep):
        hx.copy_(k[2])
    h2d = sum(h.numel() * h.element_size() for h in host_x)
    d2h = sum(h.numel() * h.element_size() for h in host_y)

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
        for j, (hx, hy, k) in enumerate(zip(host_x, host_y, layers._keep)):
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

    peaks = load_peaks()
    in_long_step = True
    bf16_peak = peaks["bf16_tflops_sustained"] if in_long_step else peaks["bf16_tflops"]
    int8_peak = bf16_peak * INT8_OVER_BF16
    gemm_kernel = "gemm_w4a8_kernel" if wl.wbits == 4 else ("gemm_w8a8_pair_kernel" if wl.M >= 2048 else "gemm_w8a8_kernel")
    # which rotate + quantize kernel the library picks per layer (rows of <= 36 blocks and >= 6 rounds of one tile per SM
    # go to the TMA-staged kernel), and the kernel that moves most of the step's bytes
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rq_bytes = {"rotate_quantize_tma_kernel": 0.0, "rotate_quantize_rows_kernel": 0.0}
    for layer in wl.layers + wl.extra_layers:
        m, nb = (layer.M or wl.M), layer.K // 128
        r = (288 // nb) // 8 * 8 if nb <= 36 else 0
        tma = r > 0 and (m + r - 1) // r >= 6 * sms
        rq_bytes["rotate_quantize_tma_kernel" if tma else "rotate_quantize_rows_kernel"] += m * (3.0 * layer.K + 4.0)
    rq_kernel = max(rq_bytes, key=rq_bytes.get)
    rq_traffic_ratio = RQ_TMA_DRAM_BYTES_PER_ALG_BYTE if rq_kernel == "rotate_quantize_tma_kernel" else RQ_ROWS_DRAM_BYTES_PER_ALG_BYTE
    dense = args.rotation == "dense"
    if dense:
        rq_kernel, rq_traffic_ratio = "rotate_dense_amax_kernel+rotate_dense_quantize_kernel", None
    gemm_tops = ops / (ms_gemm * 1e-3) / 1e12
    rq_gbs = step_rq_bytes(wl) / (ms_rq * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8" if wl.wbits == 8 else "int8xint4", "data": "synthetic",
        "config": {"workload": wl.name, "M": wl.M, "blocks": wl.blocks, "linears_per_step": n_ops, "groups": wl.num_groups,
                   "sampling_steps": wl.steps, "wbits": wl.wbits, "parallelism": f"replicas x{world} (rows independent)",
                   "rotation": args.rotation, "launch": "host" if args.no_graph else "one CUDA graph per time-step group",

                   "l2": "inputs larger than L2: every linear has its own X, codes, Y and weights"},
        "us_per_dit_step": ms_per_step * 1e3,
        "rotate_quantize_gbs": rq_gbs,
        "gemm_tops": gemm_tops,
        "kernel_ms_per_step": {"rotate_quantize": ms_rq, "gemm_epilogue": ms_gemm},
        "roofline": {"kernel": gemm_kernel, "bound": "tensor", "achieved": gemm_tops, "peak": int8_peak,
                     "unit": "TOPS", "frac": gemm_tops / int8_peak,
                     "traffic": (GEMM_PAIR_DRAM_BYTES_PER_OP * ops / n_ops) if gemm_kernel == "gemm_w8a8_pair_kernel" else None,
                     "traffic_note": "bytes per launch: capture at M=16384,K=1152,N=4608 scaled by the ops of an average launch of this workload",
                     "peak_source": f"{peaks['_source']} sustained bf16 {bf16_peak:.1f} TFLOP/s x {INT8_OVER_BF16:g} (nominal int8:bf16)"},
        "roofline_rotate_quantize": {"kernel": rq_kernel, "bound": "hbm", "achieved": rq_gbs,
                                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": rq_gbs / peaks["hbm_gbs"],
                                     "traffic": None if rq_traffic_ratio is None else rq_traffic_ratio * step_rq_bytes(wl) / n_ops,
                                     "traffic_note": "bytes per launch: capture of this kernel (TMA: M=65536,K=1152; rows: M=9000,K=1152) scaled by algorithmic bytes",
                                     "peak_source": peaks["_source"]},
        "e2e": {"value": world * ops / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": e2e_steps},
        "gpu_launches": (3 if dense else 2) * n_ops * args.steps,
        "clocks": clocks,
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline and not dense:
            line["cpu_baseline"] = cpu_baseline(wl)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, help="index into the workload list (1 = DiT-XL/2 256px, M = 4096)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="issue every step's launches from the host instead of replaying one CUDA graph per time-step group")
    ap.add_argument("--rotation", default="hadamard", choices=["hadamard", "dense"],
                    help="hadamard: the headline path; dense: dense 128 x 128 blocks on the tensor cores (Eq. 6-8), no CPU baseline")
    args = ap.parse_args()
    wl = WL.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
