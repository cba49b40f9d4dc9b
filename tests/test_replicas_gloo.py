"""The multi-process protocol of the benchmark (replicas only, no data-path collective) on CPU with
the gloo backend, world size 2: barrier, maximum over ranks, whole-job throughput."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_1711_01348_b200 import replicas
    assert replicas.rank_info() == (rank, rank, world)
    distributed = replicas.init("gloo")
    assert distributed
    replicas.barrier(distributed)
    slowest = replicas.max_over_ranks(10.0 + rank, distributed, torch.device("cpu"))
    out[rank] = (slowest, replicas.aggregate_throughput(100.0, slowest, world))
    replicas.finish(distributed)


def test_two_replicas_agree_on_the_slowest_rank():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1] == (11.0, 2 * 100.0 / 11.0)


def test_single_process_needs_no_group():
    from paper_1711_01348_b200 import replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.rank_info() == (0, 0, 1)
    assert replicas.init("gloo") is False
    assert replicas.max_over_ranks(3.5, False, torch.device("cpu")) == 3.5
