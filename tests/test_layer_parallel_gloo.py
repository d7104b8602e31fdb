"""The N > 1 path on CPU: two gloo ranks shard a list of layers (layer l -> rank l mod world, no
data-path collective) and form the whole-job throughput as total units over the slowest rank's time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_14929_b200 import pipeline


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, n_layers: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = pipeline.layers_for_rank(n_layers, rank, world)
    # every rank "sweeps" its layers: units = elements, time grows with the rank so that the max matters
    units = float(sum(1000 + l for l in mine))
    secs = 1.0 + rank
    tp = pipeline.job_throughput(units, secs)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    if rank == 0:
        out.put((gathered, tp))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_layers_and_reduce_times():
    world, n_layers = 2, 7
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_layers, q)) for r in range(world)]
    for p in procs:
        p.start()
    gathered, tp = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert sorted(gathered[0] + gathered[1]) == list(range(n_layers))     # every layer exactly once
    assert not set(gathered[0]) & set(gathered[1])
    total = float(sum(1000 + l for l in range(n_layers)))
    assert abs(tp - total / 2.0) < 1e-9                                   # slowest rank took 2 s


def test_single_process_and_bad_ranks():
    assert pipeline.layers_for_rank(5, 0, 1) == [0, 1, 2, 3, 4]
    assert pipeline.job_throughput(10.0, 2.0) == 5.0
    try:
        pipeline.layers_for_rank(5, 2, 2)
        assert False
    except ValueError:
        pass


def _bench_worker(rank: int, world: int, port: int, out):
    # the N > 1 bookkeeping of bench.py with the device work replaced by made-up times: which block a rank
    # takes, the slowest rank's time for every named timer, whole-job throughput over that time
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    block = bench.block_for_rank(rank)
    units = 1000.0                                            # every rank sweeps a block of the same size (weak scaling)
    times = dict(_ms=10.0 + 5.0 * rank, _e2e_ms=30.0 - 4.0 * rank, sweep1=1.0 + rank, sweep2=2.0)
    red = bench.reduce_times(times, torch.device("cpu"), world)
    tp = pipeline.job_throughput(units, red["_ms"] * 1e-3)
    blocks = [None] * world
    dist.all_gather_object(blocks, block)
    out.put((rank, blocks, red, tp))
    dist.barrier()
    dist.destroy_process_group()


def test_bench_bookkeeping_with_two_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_bench_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, blocks, red, tp in got:
        assert blocks == [0, 1]                                  # every rank its own transformer block
        assert red == dict(_ms=15.0, _e2e_ms=30.0, sweep1=2.0, sweep2=2.0)     # the slowest rank's, timer by timer
        assert abs(tp - 2 * 1000.0 / 15e-3) < 1e-6               # all ranks' units over the slowest rank's time
