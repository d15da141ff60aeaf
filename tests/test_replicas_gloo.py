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


def test_spawned_ranks_rendezvous_and_rank0_reports_the_job():
    """The launcher `bench.py --gpus N` uses when no external launcher set the environment: N child
    processes, each with RANK / LOCAL_RANK / WORLD_SIZE and the rendezvous address, here as two gloo
    ranks on CPU.  Rank 0's line reports the whole job: n_gpus = 2, slowest rank's times, summed
    units."""
    import json
    import sys
    codes, text = replicas.spawn_ranks([sys.executable, "-m", "paper_2609_25405_b200.replicas", "--gloo-selftest"],
                                       2, capture_rank0=True)
    assert codes == [0, 0]
    line = json.loads(text.strip().splitlines()[-1])
    assert line == {"n_gpus": 2, "ms": 11.0, "e2e_ms": 12.0, "units": 300.0, "seed": 5}


def test_spawn_stops_the_other_ranks_when_one_fails():
    import sys
    prog = "import os, sys, time\nsys.exit(3) if os.environ['RANK'] == '1' else time.sleep(60)"
    codes = replicas.spawn_ranks([sys.executable, "-c", prog], 2)
    assert codes[1] == 3 and codes[0] not in (0, None)
