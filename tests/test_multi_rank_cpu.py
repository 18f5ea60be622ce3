"""World-size-2 run of the multi-GPU host logic on CPU (gloo): layers are dealt to ranks without
overlap or gaps, and the job rate is (sum of units) / (max of times)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_22370_b200 import inputs, shard


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
        mine = shard.layers_for_rank(len(inputs.LLAMA32_1B_BLOCK), rank, world)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        rate, ms = shard.job_rate(units_local=100.0 * (rank + 1), ms_local=50.0 + 25.0 * rank)
        if rank == 0:
            out.put((gathered, rate, ms))
    finally:
        dist.destroy_process_group()


def test_two_ranks_partition_the_layers_and_reduce_the_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, rate, ms = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(gathered[0] + gathered[1]) == list(range(7))
    assert not set(gathered[0]) & set(gathered[1])
    assert ms == 75.0                                  # max over ranks
    assert abs(rate - (100.0 + 200.0) / 0.075) < 1e-9  # all units over the slowest rank's time


def test_single_process_rate_needs_no_group():
    rate, ms = shard.job_rate(10.0, 20.0)
    assert rate == 500.0 and ms == 20.0
    assert shard.layers_for_rank(7, 0, 1) == list(range(7))
