"""The N > 1 path is replicas only: two gloo ranks on CPU check the seed split and the
max-over-ranks / sum-over-ranks bookkeeping that bench.py uses."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_14075_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = [246, 250][rank]                   # verify steps this rank ran
    ms = [62.5, 71.0][rank]                    # its device time
    total, slowest = replicas.combine(units, ms)
    value = replicas.throughput(units, ms)
    dist.barrier()
    out.put((rank, total, slowest, value, replicas.replica_streams(rank, 4)))
    dist.destroy_process_group()


def test_two_ranks_sum_work_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total, slowest, value, streams in res:
        assert total == 496 and slowest == 71.0
        assert abs(value - 496 / 0.071) < 1e-6
    assert res[0][4] == [100, 101, 102, 103] and res[1][4] == [104, 105, 106, 107]   # disjoint replicas


def test_single_process_is_identity():
    assert replicas.combine(10, 2.0) == (10.0, 2.0)
    assert replicas.throughput(10, 2.0) == 5000.0
