"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_24082_b200 import multi
from paper_2602_24082_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.config1(seed=multi.rank_seed(1, rank))
    f, b = w.useful_flops()
    ms = 10.0 + 5.0 * rank              # rank 1 is the slow one
    total_ms, flops, tokens = multi.aggregate(ms, float(f + b), float(w.total_tokens))
    out.put((rank, total_ms, flops, tokens, w.total_tokens, f + b))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_max_time_and_summed_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, t0, f0, k0, tok0, fl0), (_, t1, f1, k1, tok1, fl1) = res
    assert t0 == t1 == 15.0                          # slowest rank decides
    assert f0 == f1 == float(fl0 + fl1)              # all ranks' useful FLOPs
    assert k0 == k1 == float(tok0 + tok1)
    assert tok0 != tok1                              # the ranks really drew different batches
    assert multi.whole_job_throughput(15.0, 3, f0) == pytest.approx(f0 / 5e-3 / 1e12)


def test_single_process_passthrough():
    assert multi.aggregate(3.0, 7.0, 9.0) == (3.0, 7.0, 9.0)
    assert multi.rank_seed(1, 0) == 1 and multi.rank_seed(3, 2, stride=10) == 23
