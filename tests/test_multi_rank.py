"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path has no exchange step
(every (sequence, KV head) unit is independent), so N GPUs run N replicas and only the
timing is reduced: these tests cover exactly that host logic."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2512_09238_b200 import inputs as I


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank-dependent timings: the job reports the slowest rank, stage by stage
        local = [10.0 + rank, 5.0 - rank, 1.0]
        red = bench.reduce_max(local, world)
        wl = bench.replica_workload(I.WORKLOADS["config1"].scaled(L=256), rank)
        k = I.generate(wl)["k"]
        out.put((rank, red, wl.seed, float(np.abs(k).sum())))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_timing_and_draw_independent_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, seed, checksum in got:
        assert red == [11.0, 5.0, 1.0]                  # element-wise max over ranks
    assert got[0][2] != got[1][2] and got[0][3] != got[1][3]   # different seeds, different data


def test_single_rank_paths_need_no_process_group():
    assert bench.reduce_max([3.0, 4.0], 1) == [3.0, 4.0]
    # value is the aggregate over all replicas: N ranks x batch x tokens in the slowest rank's time
    assert bench.job_throughput(8, 1, 131072, 100.0) == 8 * 131072 / 0.1
    assert bench.replica_workload(I.WORKLOADS["config4"], 0).seed == I.WORKLOADS["config4"].seed
