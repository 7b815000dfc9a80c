"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, no GPU.

The path shards by sequence with no data-path collective, so what there is to test is the host logic: every
rank draws its own batch, and the timing / unit counts are reduced over ranks as MAX / SUM.
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    from paper_2505_02351_b200 import workloads as W

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        # each rank times its own step; the job's time is the slowest rank's, its units the sum
        t = bench.max_over_ranks(10.0 + rank, "cpu")
        units = bench.sum_over_ranks(float(8 * (rank + 1)), "cpu")
        bench.barrier()
        # ranks draw different batches of the same shape (weak scaling, sharded by sequence)
        wl = W.make_config(1, seed_offset=1000 * rank)
        np.save(os.path.join(out_dir, f"q{rank}.npy"), wl.q.numpy())
        np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([t, units, wl.B, wl.Hq]))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_time_as_max_and_units_as_sum(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    assert r0[0] == r1[0] == 11.0          # MAX over ranks
    assert r0[1] == r1[1] == 24.0          # SUM over ranks
    assert (r0[2:] == r1[2:]).all()        # same shape on every rank
    q0, q1 = np.load(tmp_path / "q0.npy"), np.load(tmp_path / "q1.npy")
    assert q0.shape == q1.shape and not np.array_equal(q0, q1)   # but different values


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    """Under a multi-rank launch only rank 0 runs the oracle and prints the line; other ranks exit without work."""
    import json
    import subprocess

    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = env["LOCAL_RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--config", "2"], env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
