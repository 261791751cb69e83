"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on CPU with gloo."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_05957_b200.replicas import aggregate_throughput, max_over_ranks


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (10 + r) ms for the device-resident loop and (100 - r) ms end to end
    got = max_over_ranks([10.0 + rank, 100.0 - rank])
    dist.barrier()
    out.put((rank, got))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(world):
        assert results[r] == [11.0, 100.0]          # every rank ends with the same maxima
    # two replicas of 8 x 1000 entries, 5 steps in 11 ms
    assert aggregate_throughput(8000, 5, 11.0, world) == 2 * 8000 * 5 / 11e-3


def test_single_process_is_identity():
    assert max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert aggregate_throughput(100, 2, 1.0, 1) == 200 / 1e-3
