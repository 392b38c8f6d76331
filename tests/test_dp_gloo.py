"""The N > 1 host logic on CPU: two gloo ranks shard a matrix by rows, each encodes its shard (with the
oracle, standing in for the GPU kernel), and the pieces equal the single-process result; the timing
reduction takes the slowest rank; the reference arm of bench.py prints one line under torchrun."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import hif4_workloads as wl
    import oracle
    from paper_2602_11287_b200 import dp
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    x = wl.llama_activations(37, 512, seed=5)                       # same seeded matrix on every rank
    lo, hi = dp.shard_rows(x.shape[0], world, rank)
    mine = oracle.quantize(wl.bf16_to_u16_numpy(x[lo:hi]))
    pieces = [None] * world
    dist.all_gather_object(pieces, (lo, hi, mine))
    slowest = dp.max_over_ranks(10.0 + rank)                         # rank 1 is "slower"
    dp.barrier()
    if rank == 0:
        whole = oracle.quantize(wl.bf16_to_u16_numpy(x))
        pieces.sort(key=lambda p: p[0])
        assert pieces[0][0] == 0 and pieces[-1][1] == x.shape[0]
        assert all(pieces[i][1] == pieces[i + 1][0] for i in range(world - 1)), "shards must tile the rows"
        assert np.array_equal(np.concatenate([p[2] for p in pieces]), whole)
        assert slowest == 10.0 + world - 1
        assert dp.job_throughput(100.0, world, slowest) == world * 100.0 / slowest
        open(os.path.join(out_dir, "ok"), "w").write("ok")
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_and_reduce_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "ok").exists()


def test_shard_rows_tiles_any_size():
    from paper_2602_11287_b200 import dp
    for total in (0, 1, 7, 8, 1000, 32768):
        for world in (1, 2, 3, 8):
            spans = [dp.shard_rows(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        dp.shard_rows(10, 2, 2)
    assert dp.rank_seed(1002, 0) == 1002 and dp.rank_seed(1002, 1) != dp.rank_seed(1002, 2)
    assert dp.max_over_ranks(3.5) == 3.5                             # no process group: identity


def test_reference_arm_prints_one_line_under_torchrun():
    env = dict(os.environ, OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, "rank 0 alone prints the reference line"
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
