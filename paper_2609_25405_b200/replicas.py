"""Multi-GPU = independent replicas (the method scales by one full replica per GPU with requests
distributed round-robin; a step has no exchange between replicas).  The only cross-rank work is
bookkeeping: a barrier around the timed region and the reduction of each rank's numbers into the
whole-job figure (slowest rank's time, summed units).  Works on any torch.distributed backend."""
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
