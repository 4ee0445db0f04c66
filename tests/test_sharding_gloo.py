"""The multi-GPU path of the benchmark shards by request with no data-path
collective: every rank scores its own seeded requests, the only exchanges are
the barrier around the timed region and the MAX-reduce of the per-rank times.
These tests run that host logic as two `gloo` ranks on CPU (no GPU, no kernel
call): seeds differ per rank, the reduced time is the slowest rank's, and the
aggregate value counts every rank's tokens."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    from paper_2601_07667_b200 import inputs as I
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        r, w, local = bench.dist_env()
        assert (r, w, local) == (rank, world, rank)
        wl = I.workload("C1", seqlens=(600,), budgets=(64,))
        x = I.layer_inputs(wl, 0, bench.rank_seed(0, rank))            # every rank draws its own requests
        digest = int(np.bitwise_xor.reduce(x["k"].astype(np.uint64).ravel() * np.uint64(2654435761)))
        ms_local = 1.0 + rank                                            # rank 1 is the slow one
        ms = bench.max_over_ranks(ms_local, world, device="cpu")
        value = bench.aggregate_tokens_per_s(wl.total_tokens, world, ms)
        gathered = [None] * world
        dist.all_gather_object(gathered, (digest, ms, value))
        if rank == 0:
            np.save(os.path.join(out_dir, "result.npy"), np.array(gathered, dtype=np.float64))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_requests_and_reduce_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = np.load(os.path.join(str(tmp_path), "result.npy"))
    digests, ms, value = res[:, 0], res[:, 1], res[:, 2]
    assert digests[0] != digests[1], "ranks must score different requests"
    assert (ms == 2.0).all(), "the reduced time is the slowest rank's on every rank"
    assert value[0] == pytest.approx(2 * 600 / 2.0e-3)                   # whole-job tokens / slowest time


def test_bench_started_without_a_launcher_spawns_its_own_ranks():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment: the script starts the two
    replicas itself; rank 0 prints one line for the whole job (here without kernels, gloo on CPU)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--seed", "5"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, "one line for the whole job, from rank 0"
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 2.0          # slowest rank's time
    assert lines[0]["seed_of_last_rank"] == 6                                    # ranks draw their own requests
    assert lines[0]["value"] == pytest.approx(2 * 1000 / 2.0e-3)


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    import subprocess
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--dry-run"], env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "WORLD_SIZE" in r.stderr


def test_single_rank_helpers_need_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, device="cpu") == 3.5
    assert bench.rank_seed(7, 0) == 7 and bench.rank_seed(7, 3) == 10
    assert bench.aggregate_tokens_per_s(1000, 4, 2.0) == pytest.approx(4 * 1000 / 2.0e-3)
