"""The multi-GPU mode runs independent replicas; what the ranks share is the timing barrier and the
max over ranks.  Exercised here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_21215_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, r, lr = replicas.world_info(os.environ)
    assert (w, r, lr) == (world, rank, rank)
    replicas.barrier()
    # rank 1 is the slow replica for the first quantity, rank 0 for the second
    total_ms, e2e_ms = replicas.max_over_ranks([10.0 + 5.0 * rank, 30.0 - 4.0 * rank])
    value = replicas.aggregate_tokens_per_s(tokens_per_rank_step=8192, steps=5, world=w, slowest_total_ms=total_ms)
    replicas.barrier()
    out.put((rank, total_ms, e2e_ms, value))
    dist.destroy_process_group()


def test_two_replicas_report_all_tokens_over_the_slowest_rank():
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
    for rank, total_ms, e2e_ms, value in res:
        assert total_ms == 15.0 and e2e_ms == 30.0                      # max over the two ranks, on every rank
        assert abs(value - 2 * 8192 * 5 / 15e-3) < 1e-6


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.aggregate_tokens_per_s(100, 2, 1, 50.0) == 4000.0
