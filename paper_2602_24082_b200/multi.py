"""Host-side logic for running on several GPUs.

The path shards with no exchange step: every (row, KV-head group) is independent, so each
rank processes its own batch of rows (data parallel, as in the paper's FSDP run, Sec. 5.2)
and nothing crosses ranks inside the hot path.  The only collectives are the benchmark's
own: a MAX over ranks of the timed region and a SUM of the work done.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int, stride: int = 1) -> int:
    """Seed of the batch a rank draws (rank 0 keeps the recipe's own seed)."""
    return base_seed + stride * rank


def aggregate(total_ms: float, flops: float, tokens: float, device="cpu") -> Tuple[float, float, float]:
    """(max over ranks of the timed milliseconds, sum of FLOPs, sum of tokens).

    Works on any initialised process group (NCCL with a CUDA device, gloo on CPU); without a
    process group it returns its arguments."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return total_ms, flops, tokens
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    s = torch.tensor([flops, tokens], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(t.item()), float(s[0].item()), float(s[1].item())


def whole_job_throughput(total_ms: float, steps: int, flops_per_step_all_ranks: float) -> float:
    """Useful TFLOP/s of the whole job: all ranks' FLOPs per step over the slowest rank's
    time per step."""
    return flops_per_step_all_ranks / (total_ms / steps * 1e-3) / 1e12


def pool_rows(batches: Sequence) -> Tuple[List[Tuple[int, int]], List[int]]:
    """All rows of the ranks' batches as (batch, row) pairs, with each row's attention cost
    (visible query-key pairs, paper Sec. 3.2.1) -- the input of the row assignment."""
    pool = [(b, r) for b, w in enumerate(batches) for r in range(len(w.rows))]
    costs = [int(batches[b].select_rows([r]).useful_pairs()) for (b, r) in pool]
    return pool, costs


def rank_batch(batches: Sequence, pool: Sequence[Tuple[int, int]], rank_of_row: Sequence[int], rank: int):
    """The workload of one rank: the pooled rows assigned to it, in pool order (paper Sec. 2.2:
    rows are dealt out so that no rank waits for the one with the longest sequences).  A rank
    that got no row keeps the shortest row of the pool, so that every rank has work to time."""
    mine = [i for i, k in enumerate(rank_of_row) if k == rank]
    if not mine:
        mine = [min(range(len(pool)), key=lambda i: batches[pool[i][0]].row_lengths()[pool[i][1]])]
    rows, lv, off = [], [], 0
    for i in mine:
        b, r = pool[i]
        sub = batches[b].select_rows([r])
        rows.extend(sub.rows)
        lv.extend((lo + off, hi + off) for (lo, hi) in sub.low_var_ranges)
        off += sub.total_tokens
    t = batches[0]
    return dataclasses.replace(t, name=f"{t.name}/rank{rank}", rows=rows, low_var_ranges=lv,
                               seed=t.seed + 1000 * rank)
