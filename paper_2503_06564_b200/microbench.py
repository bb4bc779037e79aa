"""Single-kernel micro-benchmark: times one kernel of the library on one shape with CUDA events.

    python -m paper_2503_06564_b200.microbench rq   --M 65536 --K 1152
    python -m paper_2503_06564_b200.microbench gemm --M 16384 --K 1152 --N 4608
    python -m paper_2503_06564_b200.microbench rqd  --M 16384 --K 1152      (dense block rotation, Eq. 6-8)
    python -m paper_2503_06564_b200.microbench nrq  --M 16384 --K 1152      (LayerNorm + modulation folded in front)
    python -m paper_2503_06564_b200.microbench ceiling --mmas 65536         (tensor pipe alone: back-to-back MMAs on resident operands)

Also the small, self-ending command to put under a profiler (few launches, a few hundred MB).
Buffers are rotated through `--sets` distinct copies so that consecutive launches do not find
their inputs in L2.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def mma_ceiling(mmas: int = 65536, iters: int = 10):
    """Rate of the tensor pipe alone (TOPS): the best and the median of `iters` launches of the library's MMA-only kernel
    (the rate scales with the SM clock the device runs at)."""
    import torch
    from paper_2503_06564_b200 import trdq
    ops = trdq.trdq_measure_mma_ceiling(mmas)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record()
    for i in range(iters):
        trdq.trdq_measure_mma_ceiling(mmas)
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(iters))
    assert trdq.trdq_device_status() == 0
    return {"kernel": "mma_ceiling_kernel", "mmas_per_cluster": mmas, "ops_per_launch": ops, "ms_median": ms[len(ms) // 2], "ms_min": ms[0],
            "rate_median": ops / (ms[len(ms) // 2] * 1e-3) / 1e12, "rate_best": ops / (ms[0] * 1e-3) / 1e12, "unit": "TOPS"}


def main():
    import torch
    from paper_2503_06564_b200 import build, trdq
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["rq", "rqd", "nrq", "gemm", "ceiling"])
    ap.add_argument("--M", type=int, default=16384)
    ap.add_argument("--K", type=int, default=1152)
    ap.add_argument("--N", type=int, default=4608)
    ap.add_argument("--wbits", type=int, default=8)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--sets", type=int, default=4)
    ap.add_argument("--mmas", type=int, default=65536, help="ceiling: MMAs (256 x 256 x 32, int8) per CTA pair and launch")
    ap.add_argument("--full-transform", action="store_true", help="rq: rotation, zigzag permutation, second rotation (Eq. 9)")
    ap.add_argument("--splitk", action="store_true", help="gemm: use trdq_linear_splitk with a preallocated workspace")
    ap.add_argument("--no-graph", action="store_true", help="time individual launches issued from Python (profiler runs)")
    args = ap.parse_args()
    build.build()
    if args.kernel == "ceiling":
        print(json.dumps(mma_ceiling(args.mmas, args.iters)))
        return
    torch.manual_seed(0)
    M, K, N = args.M, args.K, args.N
    rng = np.random.default_rng(0)
    signs = (rng.integers(0, 2, (1, K)) * 2 - 1).astype(np.int8)
    perm = rng.permutation(K).astype(np.int32)[None, :] if args.full_transform else None
    rot = trdq.Rotation(K, [0, 1000], signs, None, perm=perm)
    xs = [torch.randn((M, K), device="cuda").to(torch.bfloat16) for _ in range(args.sets)]
    codes = [torch.empty((M, K), dtype=torch.int8, device="cuda") for _ in range(args.sets)]
    scales = [torch.empty((M,), dtype=torch.float32, device="cuda") for _ in range(args.sets)]
    if args.kernel == "rqd":
        blocks = np.empty((1, K // 128, 128, 128), np.float32)
        for b in range(K // 128):
            q, _ = np.linalg.qr(rng.standard_normal((128, 128)))
            blocks[0, b] = q
        drot = trdq.DenseRotation(K, [0, 1000], blocks, None)
        ws = torch.empty((trdq.trdq_rotate_dense_workspace(drot, M),), dtype=torch.uint8, device="cuda")

        def run(i):
            s = i % args.sets
            trdq.trdq_rotate_dense_quantize(drot, 0, xs[s], codes[s], scales[s], ws)
        work, unit = M * (3.0 * K + 4.0) / 1e9, "GB/s"
    elif args.kernel == "nrq":
        rps = 256
        shift = (torch.randn(((M + rps - 1) // rps, K), device="cuda") * 0.2).to(torch.bfloat16)
        scale = (torch.randn(((M + rps - 1) // rps, K), device="cuda") * 0.2).to(torch.bfloat16)

        def run(i):
            s = i % args.sets
            trdq.trdq_norm_rotate_quantize(rot, 0, xs[s], shift, scale, rps, 1e-6, codes[s], scales[s])
        work, unit = M * (3.0 * K + 4.0) / 1e9, "GB/s"
    elif args.kernel == "rq":
        def run(i):
            s = i % args.sets
            trdq.trdq_rotate_quantize(rot, 0, xs[s], codes[s], scales[s])
        work, unit = M * (3.0 * K + 4.0) / 1e9, "GB/s"
    else:
        w = (torch.randn((N, K), device="cuda") * 0.02).to(torch.bfloat16)
        wts = trdq.trdq_prepare_weights(rot, w, args.wbits)
        bias = torch.zeros((N,), dtype=torch.bfloat16, device="cuda")
        ys = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(args.sets)]
        for s in range(args.sets):
            trdq.trdq_rotate_quantize(rot, 0, xs[s], codes[s], scales[s])

        splits, nbytes = trdq.trdq_linear_splitk_workspace(wts, M)
        ws = torch.empty((max(nbytes, 16),), dtype=torch.uint8, device="cuda")

        def run(i):
            s = i % args.sets
            if args.splitk:
                trdq.trdq_linear_splitk(wts, 0, codes[s], scales[s], bias, ys[s], ws)
            else:
                trdq.trdq_linear(wts, 0, codes[s], scales[s], bias, ys[s])
        work, unit = 2.0 * M * N * K / 1e12, "TOPS"
    for i in range(args.warmup):
        run(i)
    torch.cuda.synchronize()
    if args.no_graph:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.iters + 1)]
        ev[0].record()
        for i in range(args.iters):
            run(i)
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(args.iters))
    else:
        # one pass over all buffer sets captured in a CUDA graph: launches are back to back on the
        # device, so small shapes are not limited by the host's launch rate
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for i in range(args.sets):
                run(i)
        graph.replay()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.iters + 1)]
        ev[0].record()
        for i in range(args.iters):
            graph.replay()
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = sorted(ev[i].elapsed_time(ev[i + 1]) / args.sets for i in range(args.iters))
    med = ms[len(ms) // 2]
    assert trdq.trdq_device_status() == 0
    print(json.dumps({"kernel": args.kernel, "M": M, "K": K, "N": N if args.kernel == "gemm" else None, "wbits": args.wbits,
                      "ms_median": med, "ms_min": ms[0], "rate_median": work / (med * 1e-3), "rate_best": work / (ms[0] * 1e-3),
                      "unit": unit}))


if __name__ == "__main__":
    main()
