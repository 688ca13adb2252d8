"""Two gloo ranks on CPU: the replica bookkeeping used by bench.py at N > 1 (slowest rank's
time, total tokens, distinct seeds per rank)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_08721_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, tok = replicas.aggregate(10.0 + 5.0 * rank, 1000.0 + rank, device="cpu")
    out[rank] = (ms, tok, replicas.rank_seed(2, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_all_tokens():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == res[1][:2] == (15.0, 2001.0)
    assert res[0][2] != res[1][2]
    assert replicas.throughput(15.0, 2001.0, 3) == 2001.0 * 3 / 0.015


def test_single_process_is_the_identity():
    assert replicas.aggregate(7.0, 9.0) == (7.0, 9.0)
