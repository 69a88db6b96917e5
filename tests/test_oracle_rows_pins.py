"""Pins for the row-builder oracle (oracle/rows.py): properties fixed by the definitions, a
hand-worked example, and the pair count against the dense mask of the attention oracle."""
import os

import numpy as np
import pytest

import oracle
from oracle import rows as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "rows_example.txt")


def _random_groups(rng, G, max_len):
    P = rng.integers(1, max_len, size=G)
    n = rng.integers(1, 5, size=G)
    off = np.concatenate([[0], np.cumsum(n)])
    rl = rng.integers(1, max_len, size=off[-1])
    return P.astype(np.int32), off.astype(np.int32), rl.astype(np.int32)


def test_worked_example():
    kv = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        kv[k] = [int(x) for x in v]
    out = R.build_rows(kv["prompts"], kv["resp_off"], kv["resp_len"], kv["capacity"][0])
    assert out["order"].tolist() == kv["order"]
    assert out["row_group_off"].tolist() == kv["row_group_off"]
    assert out["row_tokens"].tolist() == kv["row_tokens"]
    assert out["row_cost"].tolist() == kv["row_cost"]


@pytest.mark.parametrize("seed", range(5))
def test_order_and_next_fit_properties(seed):
    rng = np.random.default_rng(seed)
    P, off, rl = _random_groups(rng, 200, 300)
    tok = np.array([P[g] + rl[off[g]:off[g + 1]].sum() for g in range(len(P))])
    cap = int(tok.max() * 2.5)
    out = R.build_rows(P, off, rl, cap)
    order = out["order"]
    assert sorted(order.tolist()) == list(range(len(P)))               # a permutation
    st = tok[order]
    assert (np.diff(st) <= 0).all()                                     # longest first
    for a, b in zip(order[:-1], order[1:]):                             # ties keep their order
        if tok[a] == tok[b]:
            assert a < b
    rgo = out["row_group_off"]
    assert rgo[0] == 0 and rgo[-1] == len(P) and (np.diff(rgo) >= 1).all()
    for r in range(len(rgo) - 1):
        t = st[rgo[r]:rgo[r + 1]].sum()
        assert t == out["row_tokens"][r] and t <= cap                   # within capacity
        if r + 1 < len(rgo) - 1:
            assert t + st[rgo[r + 1]] > cap                             # next fit: it was full
    # the reordered descriptors describe the same groups
    nP, noff, nrl = out["grp_prompt_len"], out["grp_resp_off"], out["resp_len"]
    for pos, g in enumerate(order):
        assert nP[pos] == P[g]
        assert nrl[noff[pos]:noff[pos + 1]].tolist() == rl[off[g]:off[g + 1]].tolist()
    assert out["row_tokens"].sum() == tok.sum()


def test_equal_lengths_closed_form():
    G, ell, cap = 37, 10, 45
    P = np.full(G, 4, dtype=np.int32)
    off = np.arange(G + 1, dtype=np.int32) * 2
    rl = np.full(2 * G, 3, dtype=np.int32)
    out = R.build_rows(P, off, rl, cap)
    per = cap // ell
    assert out["order"].tolist() == list(range(G))                      # all ties: original order
    assert np.diff(out["row_group_off"]).tolist() == [per] * (G // per) + ([G % per] if G % per else [])


def test_group_longer_than_capacity_is_rejected():
    with pytest.raises(ValueError):
        R.build_rows([5, 50], [0, 1, 2], [3, 60], 100)


def test_pair_count_matches_dense_mask():
    """The cost formula against a brute-force count over the attention oracle's dense mask."""
    rng = np.random.default_rng(3)
    P, off, rl = _random_groups(rng, 12, 20)
    want = R.group_pairs(P, off, rl)
    for g in range(len(P)):
        desc = (np.array([0, 1], dtype=np.int32), P[g:g + 1], np.array([0, off[g + 1] - off[g]], dtype=np.int32),
                rl[off[g]:off[g + 1]])
        m = oracle.dense_mask(desc, 0)
        assert int(m.sum()) == int(want[g])
    assert int(R.group_tokens(P, off, rl).sum()) == int(P.sum() + rl.sum())


# ---------------------------------------------------------------- rows -> ranks
ASSIGN_GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "assign_example.txt")


def test_assign_worked_example():
    kv = {}
    for line in open(ASSIGN_GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        kv[k] = [int(x) for x in v]
    order, rank_of_row, rank_cost = R.assign_rows(kv["row_cost"], kv["ranks"][0])
    assert order.tolist() == kv["order"]
    assert rank_of_row.tolist() == kv["rank_of_row"]
    assert rank_cost.tolist() == kv["rank_cost"]


def _best_makespan(cost, m):
    """Brute force over all m^n assignments (tiny n only)."""
    import itertools
    best = None
    for assign in itertools.product(range(m), repeat=len(cost)):
        load = [0] * m
        for c, k in zip(cost, assign):
            load[k] += c
        best = max(load) if best is None else min(best, max(load))
    return best


@pytest.mark.parametrize("seed", range(8))
def test_assign_properties_and_bound_against_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n, m = int(rng.integers(1, 9)), int(rng.integers(1, 4))
    cost = rng.integers(0, 50, size=n).tolist()
    order, rank_of_row, rank_cost = R.assign_rows(cost, m)
    assert sorted(order.tolist()) == list(range(n))                       # a permutation
    assert all(cost[order[i]] >= cost[order[i + 1]] for i in range(n - 1))  # decreasing cost
    load = [sum(c for c, k in zip(cost, rank_of_row) if k == r) for r in range(m)]
    assert load == rank_cost.tolist() and sum(load) == sum(cost)
    # list scheduling: the fullest rank got its last row while it was the emptiest
    assert max(load) <= sum(cost) / m + max(cost)
    # longest-processing-time rule: within (4/3 - 1/(3m)) of the optimum (Graham 1969)
    opt = _best_makespan(cost, m)
    assert max(load) <= (4.0 / 3.0 - 1.0 / (3 * m)) * opt + 1e-9


def test_assign_ties_and_more_ranks_than_rows():
    order, rank_of_row, rank_cost = R.assign_rows([5, 5, 5], 5)
    assert order.tolist() == [0, 1, 2] and rank_of_row.tolist() == [0, 1, 2]
    assert rank_cost.tolist() == [5, 5, 5, 0, 0]
    order, rank_of_row, rank_cost = R.assign_rows([0, 0, 7], 2)
    assert order.tolist() == [2, 0, 1] and rank_of_row.tolist() == [1, 1, 0]
