"""World-size-2 run of the multi-GPU host logic on CPU (gloo): layers are dealt to ranks without
overlap or gaps, the job rate is (sum of units) / (max of times), and for a layer split by output rows
the ranks agree on the largest tensor scale and add their loss shares."""
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
        # a 300-row layer split by rows: rank 0 holds the larger weights
        rows = shard.rows_for_rank(301, rank, world)
        scale = shard.global_tensor_scale(torch.tensor([0.25 if rank == 0 else 0.125]))
        losses = shard.combine_losses(torch.tensor([10.0 + rank, 0.5 + 0.25 * rank]), rows[1] - rows[0], 301)
        if rank == 0:
            out.put((gathered, rate, ms, rows, float(scale), losses.tolist()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_partition_the_layers_and_reduce_the_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, rate, ms, rows0, scale, losses = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(gathered[0] + gathered[1]) == list(range(7))
    assert not set(gathered[0]) & set(gathered[1])
    assert ms == 75.0                                  # max over ranks
    assert abs(rate - (100.0 + 200.0) / 0.075) < 1e-9  # all units over the slowest rank's time
    assert rows0 == (0, 151)
    assert scale == 0.25                               # the largest of the ranks' scales
    assert abs(losses[0] - 21.0) < 1e-12               # squared errors add up
    assert abs(losses[1] - (0.5 * 151 + 0.75 * 150) / 301) < 1e-12   # Round Loss: mean over all weights


def test_single_process_rate_needs_no_group():
    rate, ms = shard.job_rate(10.0, 20.0)
    assert rate == 500.0 and ms == 20.0
    assert shard.layers_for_rank(7, 0, 1) == list(range(7))


def test_row_ranges_tile_the_layer():
    for rows, world in ((2048, 2), (301, 2), (7, 3), (5, 8), (1, 1)):
        ranges = [shard.rows_for_rank(rows, r, world) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == rows
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        sizes = [e - b for b, e in ranges]
        assert max(sizes) - min(sizes) <= 1
    # without a process group the collectives are the identity
    t = torch.tensor([0.5])
    assert shard.global_tensor_scale(t) is t and float(t) == 0.5
    assert shard.combine_losses(torch.tensor([3.0, 0.5]), 10, 40).tolist() == [3.0, 0.125]
