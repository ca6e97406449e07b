"""Several GPUs: independent replicas.

The round loop does not shard (one simulated server, one version ring), so N GPUs run N
independent ABS runs with different seeds and no data-path collective.  The only exchange is
the benchmark bookkeeping below: whole-job throughput = units of all ranks / slowest rank's time.
"""
import torch
import torch.distributed as dist


def replica_seed(base_seed, rank):
    """Run (Philox) seed of a replica: distinct per rank, reproducible."""
    return int(base_seed) + int(rank)


def aggregate_replicas(seconds, units, device="cpu", group=None):
    """(max over ranks of seconds, sum over ranks of units) per column.

    seconds, units: equal-length lists of floats of this rank.  Works with any initialised
    process group (nccl with a CUDA device, gloo with "cpu"); without one it returns its inputs."""
    if not (dist.is_available() and dist.is_initialized()):
        return list(seconds), list(units)
    t = torch.tensor(seconds, dtype=torch.float64, device=device)
    u = torch.tensor(units, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    return [float(x) for x in t], [float(x) for x in u]
