"""The multi-rank benchmark logic on CPU: two gloo ranks, each with its own batch, exchange
nothing but their timing; the job's throughput uses the slowest rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2002_12418_b200 import replicas as R
from paper_2002_12418_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        layer = W.config0()[0].with_batch(2, seed_offset=R.rank_seed_offset(rank))
        x, _, _ = W.make_inputs(layer)
        local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        dist.barrier()
        slowest = R.max_over_ranks(dist, local_ms)
        value = R.whole_job_throughput(layer.direct_flops, 4, world, slowest)
        out.put((rank, float(x.ravel()[0]), slowest, value))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_own_batches():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, x0, s0, v0), (r1, x1, s1, v1) = got
    assert (r0, r1) == (0, 1)
    assert x0 != x1                                        # every rank drew its own batch
    assert s0 == s1 == 15.0                                # max over ranks, identical everywhere
    layer = W.config0()[0].with_batch(2)
    expect = 2 * layer.direct_flops * 4 / 15e-3 / 1e12
    assert v0 == v1 and abs(v0 - expect) <= 1e-12 * expect


def test_single_rank_needs_no_process_group():
    assert R.max_over_ranks(None, 3.5) == 3.5
    assert R.rank_seed_offset(0) == 0 and R.rank_seed_offset(3) == 30000
    assert np.isclose(R.whole_job_throughput(1e12, 10, 1, 1000.0), 10.0)


def test_launch_plan_spawns_ranks_only_on_a_plain_command_line():
    assert R.launch_plan(1, {}) == "single"
    assert R.launch_plan(8, {}) == "spawn"
    assert R.launch_plan(8, {"WORLD_SIZE": "8", "RANK": "3"}) == "env"
    assert R.launch_plan(1, {"WORLD_SIZE": "1", "RANK": "0"}) == "env"
    env = R.rank_environment(2, 4, 29512)
    assert env == {"RANK": "2", "LOCAL_RANK": "2", "WORLD_SIZE": "4", "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "29512"}
