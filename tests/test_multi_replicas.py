"""The N > 1 path of the benchmark: independent replicas, aggregated over a process group
(gloo, world size 2, on CPU)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2301_08895_b200 import multi


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seed = multi.replica_seed(2004, rank)
    secs, units = multi.aggregate_replicas([1.0 + rank, 0.5], [100.0 * (rank + 1), 7.0])
    out.put((rank, seed, secs, units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2004, 2005]            # distinct seeds, one run per rank
    for _, _, secs, units in res:
        assert secs == [2.0, 0.5]                          # slowest rank decides the time
        assert units == [300.0, 14.0]                      # work of all ranks counts


def test_single_process_passthrough():
    assert multi.aggregate_replicas([1.5], [3.0]) == ([1.5], [3.0])
