"""The N > 1 path is N independent replicas: only the timing bookkeeping crosses ranks.
Covered here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_25405_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    step_ms, e2e_ms, units = [(10.0, 12.0, 4096.0), (14.0, 11.0, 4000.0)][rank]
    got = replicas.aggregate(dist, "cpu", step_ms, e2e_ms, units)
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_two_ranks_gloo():
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (14.0, 12.0, 8096.0)      # slowest rank's times, summed units


def test_single_process_passthrough_and_assignment():
    assert replicas.aggregate(None, "cpu", 3.0, 4.0, 5.0) == (3.0, 4.0, 5.0)
    assert replicas.assign_round_robin(7, 3) == [[0, 3, 6], [1, 4], [2, 5]]
    assert replicas.rank_seed(1003, 0) == 1003 and replicas.rank_seed(1003, 2) != replicas.rank_seed(1003, 1)
