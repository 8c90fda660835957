"""The N>1 path is "replicas only": independent cubes per rank, max-over-ranks timing.  Exercised here with
two CPU processes over gloo (127.0.0.1): the replica logic needs no GPU."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2002_03260_b200 import inputs, replicas
    seed = replicas.rank_seed(1003, rank)
    x = inputs.cube((4, 4, 8), "uniform", seed, device="cpu")
    # each rank reports a different local time; the job's time is the slowest rank's
    local_ms = 10.0 * (rank + 1)
    value, ms = replicas.aggregate_throughput(1000.0, local_ms)
    gathered = [None] * world
    dist.all_gather_object(gathered, (seed, float(x.real.sum()), ms, value))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    seeds = [g[0] for g in got]
    assert seeds == [1003, 1004]
    assert got[0][1] != got[1][1]                       # different cubes per replica
    assert all(abs(g[2] - 20.0) < 1e-12 for g in got)   # max over ranks of the local times
    assert all(abs(g[3] - 2 * 1000.0 / 0.020) < 1e-6 for g in got)   # all ranks' units over the slowest time
