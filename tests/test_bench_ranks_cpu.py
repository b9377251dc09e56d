"""The N > 1 plumbing of bench.py (replicas only: barrier, max over ranks, whole-job value) with two gloo
ranks on CPU.  No GPU and no data-path collective is involved."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        dist.barrier()
        slowest = bench.max_over_ranks(mine, world, torch.device("cpu"))
        out[rank] = (slowest, bench.ms_per_layer(slowest, world, 1), bench.replica_seed(100, rank))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_rank_and_aggregate_value():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    assert res[0][1] == 7.5                        # two layers (one per rank) per 15 ms step
    assert {res[0][2], res[1][2]} == {100, 101}    # independent replicas


def test_single_rank_is_identity():
    assert bench.max_over_ranks(3.0, 1, torch.device("cpu")) == 3.0
    assert bench.ms_per_layer(8.0, 1, 2) == 4.0
