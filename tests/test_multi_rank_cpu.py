"""The multi-GPU path of the benchmark on CPU: two gloo ranks.  The hot path shards by sequence with no data-path
collective, so what needs testing is the plumbing: per-rank seeds give disjoint batches, the slowest rank's time
is what every rank sees, and the aggregate counts the units of all ranks."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2508_04257_b200 import dist_util, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ri = dist_util.rank_info()
    assert (ri.rank, ri.world) == (rank, world)
    wl = synth.WORKLOADS["tiny"].scaled(seed=dist_util.rank_seed(synth.WORKLOADS["tiny"].seed, rank))
    K, _ = synth.make_kv(wl)
    my_ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    dist.barrier()
    ms = dist_util.max_over_ranks(my_ms, "cpu")
    value = dist_util.aggregate_throughput(1000.0, world, ms * 1e-3)
    digest = torch.tensor([float(K.float().sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    out.put((rank, ms, value, [float(g) for g in gathered]))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_sequence_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, sums in res:
        assert ms == 20.0                            # max over ranks, seen by both
        assert np.isclose(value, 2 * 1000.0 / 0.020)
        assert sums[0] != sums[1]                    # per-rank seeds: different batches
    assert res[0][3] == res[1][3]


def test_single_process_is_the_identity():
    assert dist_util.max_over_ranks(3.5, "cpu") == 3.5
    assert dist_util.aggregate_throughput(10.0, 1, 2.0) == 5.0


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself; here only the plumbing runs (gloo, no kernels)."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plumbing-only"], capture_output=True, text=True,
                       env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 2.0 and lines[0]["scaling"] == "weak"
