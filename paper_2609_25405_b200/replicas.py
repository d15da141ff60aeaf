"""Multi-GPU = independent replicas (the method scales by one full replica per GPU with requests
distributed round-robin; a step has no exchange between replicas).  The only cross-rank work is
bookkeeping: a barrier around the timed region and the reduction of each rank's numbers into the
whole-job figure (slowest rank's time, summed units).  Works on any torch.distributed backend."""
import os
import socket
import subprocess
import time

import torch


def rank_seed(base_seed, rank):
    """Each replica draws its own batch stream."""
    return int(base_seed) + 7919 * int(rank)


def assign_round_robin(n_requests, world):
    """Request i goes to replica i % world; returns the per-rank index lists."""
    return [list(range(r, n_requests, world)) for r in range(world)]


def aggregate(dist, device, step_ms, e2e_ms, units):
    """(max step_ms over ranks, max e2e_ms over ranks, sum of units over ranks)."""
    t = torch.tensor([float(step_ms), float(e2e_ms), float(units)], dtype=torch.float64, device=device)
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(t[0]), float(t[1]), float(t[2])
    mx = t.clone()
    dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    sm = t.clone()
    dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return float(mx[0]), float(mx[1]), float(sm[2])


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(argv, n, capture_rank0=False, poll_s=0.2):
    """Start `argv` n times as ranks 0..n-1 of one job on this node (one replica per GPU: rank r gets
    LOCAL_RANK r) and wait for all of them.  Each child finds RANK, LOCAL_RANK, WORLD_SIZE and the
    rendezvous address in its environment, exactly as under an external launcher.  The communicator
    log of the collective library stays on (to stderr), so the N ranks of the job are visible.  If a
    rank fails, the others are stopped (by their own process ids).  Returns the list of exit codes,
    or (codes, rank 0's stdout) with capture_rank0."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        out = subprocess.PIPE if (capture_rank0 and r == 0) else None
        procs.append(subprocess.Popen(argv, env=env, stdout=out, text=True if out else None))
    codes = [None] * n
    text = None
    while any(c is None for c in codes):
        for r, p in enumerate(procs):
            if codes[r] is None and p.poll() is not None:
                codes[r] = p.returncode
        if any(c not in (None, 0) for c in codes):
            for r, p in enumerate(procs):
                if codes[r] is None:
                    p.terminate()
            for r, p in enumerate(procs):
                if codes[r] is None:
                    try:
                        codes[r] = p.wait(timeout=10)
                    except subprocess.TimeoutExpired:
                        p.kill()
                        codes[r] = p.wait()
            break
        if capture_rank0 and procs[0].stdout is not None and codes[0] is not None and text is None:
            text = procs[0].stdout.read()
        time.sleep(poll_s)
    if capture_rank0:
        if text is None and procs[0].stdout is not None:
            text = procs[0].stdout.read()
        return codes, text
    return codes


def _gloo_selftest():
    """One rank of a CPU-only job (backend gloo): what a replica rank of the benchmark does around its
    timed region, without a GPU.  Rank 0 prints one JSON line."""
    import json

    import torch.distributed as dist
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms, e2e, units = aggregate(dist, "cpu", 10.0 + rank, 12.0 - rank, 100.0 * (rank + 1))
    dist.barrier()
    dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ms": ms, "e2e_ms": e2e, "units": units, "seed": rank_seed(5, rank)}))


if __name__ == "__main__":
    import sys
    if "--gloo-selftest" in sys.argv:
        _gloo_selftest()
