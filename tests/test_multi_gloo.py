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


def _dp_worker(rank, world, port, out):
    """The data-parallel path of the benchmark on CPU: every rank pools the same batches,
    takes the same assignment (here from the row oracle; on GPUs from pp_assign_rows) and
    keeps its own rows; the aggregate is the pool's work over the slowest rank's time."""
    from oracle import rows as R
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    batches = [W.config3(seed=multi.rank_seed(3, r, 10)) for r in range(world)]
    pool, costs = multi.pool_rows(batches)
    _, rank_of_row, rank_cost = R.assign_rows(costs, world)
    w = multi.rank_batch(batches, pool, rank_of_row.tolist(), rank)
    f, b = w.useful_flops()
    total_ms, flops, tokens = multi.aggregate(float(w.useful_pairs()) * 1e-6, float(f + b), float(w.total_tokens))
    out.put((rank, total_ms, flops, tokens, w.total_tokens, w.useful_pairs(), int(rank_cost[rank]),
             sum(costs), sum(bw.total_tokens for bw in batches)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_a_pool_of_rows_by_cost():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, t0, f0, k0, tok0, u0, c0, all_cost, all_tok), (_, t1, f1, k1, tok1, u1, c1, _, _) = res
    assert u0 == c0 and u1 == c1                      # a rank's batch is exactly its assigned rows
    assert u0 + u1 == all_cost and tok0 + tok1 == all_tok == k0 == k1   # the pool is partitioned
    assert t0 == t1 == max(u0, u1) * 1e-6
    assert max(u0, u1) <= all_cost / 2 + max(u0, u1, 1)


def test_rank_batch_keeps_low_variance_ranges_and_gives_every_rank_work():
    batches = [W.config2(seed=multi.rank_seed(2, r, 10)) for r in range(2)]
    pool, costs = multi.pool_rows(batches)
    assert len(pool) == 8 and all(c > 0 for c in costs)
    w = multi.rank_batch(batches, pool, [0] * 8, 0)
    assert w.total_tokens == sum(b.total_tokens for b in batches)
    assert len(w.low_var_ranges) == 8 and all(0 <= lo < hi <= w.total_tokens for lo, hi in w.low_var_ranges)
    idle = multi.rank_batch(batches, pool, [0] * 8, 1)      # nothing assigned: the shortest row
    assert len(idle.rows) == 1
    assert idle.total_tokens == min(l for b in batches for l in b.row_lengths())
