"""The N > 1 bookkeeping of the benchmark (replicas only: no data-path collective), run as two
gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_15750_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" 5 + r ms per step and committed 2 + r tokens
    times, counts = replicas.combine(dist, [5.0 + rank, 7.0 - rank], [2 + rank, 10 * (rank + 1)])
    dist.barrier()
    q.put((rank, times, counts, replicas.replica_seed(100, rank)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, counts, seed in res:
        assert times == [6.0, 7.0]            # max over ranks
        assert counts == [5, 30]              # sum over ranks
        assert seed == 100 + 1000 * rank      # disjoint sequences per replica
    assert replicas.aggregate_throughput(5, 6.0) == 5 / 6e-3


def test_single_process_passes_values_through():
    assert replicas.combine(None, [1.5], [3]) == ([1.5], [3])
