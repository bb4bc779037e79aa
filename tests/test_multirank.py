"""World-size-2 (gloo, CPU) checks of the multi-GPU host logic: rows shard with no collective."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_06564_b200 import multirank, workloads as WL


def test_row_shard_partitions_exactly():
    for M in (0, 1, 5, 256, 4096, 4097, 32768 + 960):
        for world in (1, 2, 3, 4, 8):
            for align in (1, 128):
                pieces = [multirank.row_shard(M, r, world, align) for r in range(world)]
                assert pieces[0][0] == 0 and pieces[-1][1] == M
                for (a0, a1), (b0, b1) in zip(pieces, pieces[1:]):
                    assert a1 == b0 and a0 <= a1
                sizes = [e - b for b, e in pieces]
                assert max(sizes) - min(sizes) <= 2 * align - 1
    with pytest.raises(ValueError):
        multirank.row_shard(10, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    from oracle import trdq_oracle as O
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = WL.WORKLOADS[0]
        inp = WL.make_layer_inputs(wl, 0, M=70)                 # every rank draws the same seeded inputs
        act, wv = O.fused_vectors(inp.signs[1], None)
        qw, sw = O.prepare_w8(inp.w, wv)
        b, e = multirank.row_shard(inp.M, rank, world)
        q, sx = O.rotate_quantize(inp.x[b:e], act)              # this rank's rows only
        y = O.linear_w8_rows(q, sx, qw, sw, inp.bias, np.arange(e - b))
        np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
        # timing agreement: the slowest rank defines the step time
        t = multirank.max_over_ranks(10.0 + rank)
        assert t == 10.0 + world - 1
        assert abs(multirank.aggregate_rate(100.0, world, t) - world * 100.0 / (t * 1e-3)) < 1e-9
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_without_collective(tmp_path):
    from oracle import trdq_oracle as O
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = WL.WORKLOADS[0]
    inp = WL.make_layer_inputs(wl, 0, M=70)
    act, wv = O.fused_vectors(inp.signs[1], None)
    qw, sw = O.prepare_w8(inp.w, wv)
    q, sx = O.rotate_quantize(inp.x, act)
    y_full = O.linear_w8_rows(q, sx, qw, sw, inp.bias, np.arange(inp.M))
    y_cat = np.concatenate([np.load(tmp_path / f"y{r}.npy") for r in range(world)])
    assert np.array_equal(y_cat, y_full)                        # sharding over rows is exact


def test_max_over_ranks_without_process_group():
    assert multirank.max_over_ranks(3.5) == 3.5


def test_spawn_ranks_gives_every_rank_its_environment(tmp_path):
    """The launcher bench.py uses when it is asked for N GPUs outside torchrun: N processes with RANK / WORLD_SIZE /
    MASTER_* set, which can form a process group (gloo here) and agree on a maximum; rank 0's output is returned."""
    import sys
    script = tmp_path / "rank.py"
    script.write_text(
        "import os, sys\n"
        f"sys.path.insert(0, {repr(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))})\n"
        "import torch.distributed as dist\n"
        "from paper_2503_06564_b200 import multirank\n"
        "rank, world = int(os.environ['RANK']), int(os.environ['WORLD_SIZE'])\n"
        "assert os.environ['MASTER_ADDR'] == '127.0.0.1' and int(os.environ['LOCAL_RANK']) == rank\n"
        "dist.init_process_group('gloo', rank=rank, world_size=world)\n"
        "t = multirank.max_over_ranks(1.0 + rank)\n"
        "dist.barrier()\n"
        "dist.destroy_process_group()\n"
        "if rank == 0: print('world', world, 'max', t)\n")
    rc, out = multirank.spawn_ranks(2, [sys.executable, str(script)], timeout=120)
    assert rc == 0 and out.strip() == "world 2 max 2.0"
    bad = tmp_path / "bad.py"
    bad.write_text("import os, sys\nsys.exit(3 if os.environ['RANK'] == '1' else 0)\n")
    rc, _ = multirank.spawn_ranks(2, [sys.executable, str(bad)], timeout=60)
    assert rc == 3
    # a rank that never finishes is ended when another one fails (no waiting for a collective that cannot complete)
    hang = tmp_path / "hang.py"
    hang.write_text("import os, sys, time\nif os.environ['RANK'] == '0': time.sleep(600)\nsys.exit(5)\n")
    import time
    t0 = time.monotonic()
    rc, _ = multirank.spawn_ranks(2, [sys.executable, str(hang)], timeout=120)
    assert rc == 5 and time.monotonic() - t0 < 60
    with pytest.raises(ValueError):
        multirank.spawn_ranks(0, [sys.executable, str(bad)])
