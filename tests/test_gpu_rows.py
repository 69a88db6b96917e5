"""GPU parity for the row builder (bit-exact: integer work) against oracle/rows.py, and the
hand-over of its output to the plan builder."""
import numpy as np
import pytest
import torch

from oracle import rows as R

pytestmark = pytest.mark.gpu


def _random_groups(rng, G, max_len, max_resp=5):
    P = rng.integers(1, max_len, size=G)
    n = rng.integers(1, max_resp, size=G)
    off = np.concatenate([[0], np.cumsum(n)])
    rl = rng.integers(1, max_len, size=off[-1])
    return P.astype(np.int32), off.astype(np.int32), rl.astype(np.int32)


def _gpu(P, off, rl, cap):
    from paper_2602_24082_b200 import binding as B
    d = lambda a: torch.from_numpy(np.ascontiguousarray(np.asarray(a, dtype=np.int32))).cuda()
    return B.pp_build_rows(d(P), d(off), d(rl), cap)


def _compare(P, off, rl, cap):
    want = R.build_rows(P, off, rl, cap)
    got = _gpu(P, off, rl, cap)
    assert got["status"] == (0, 0)
    for k in ("order", "row_group_off", "row_tokens", "row_cost", "grp_prompt_len", "grp_resp_off",
              "resp_len"):
        assert np.array_equal(got[k].cpu().numpy(), want[k]), k
    return want, got


def test_worked_example():
    want, _ = _compare([2, 4, 1, 5, 3], [0, 2, 4, 6, 7, 9], [2, 1, 3, 2, 1, 1, 4, 2, 2], 16)
    assert want["row_group_off"].tolist() == [0, 1, 3, 5]


@pytest.mark.parametrize("G,max_len,cap_factor,seed", [(1, 50, 1.0, 0), (7, 30, 1.0, 1), (300, 400, 2.5, 2),
                                                       (1500, 2000, 4.0, 3), (5000, 64, 30.0, 4)])
def test_random_batches(G, max_len, cap_factor, seed):
    rng = np.random.default_rng(seed)
    P, off, rl = _random_groups(rng, G, max_len)
    tok = R.group_tokens(P, off, rl)
    _compare(P, off, rl, int(tok.max() * cap_factor))


def test_many_equal_lengths_keep_original_order():
    G = 2000
    P = np.full(G, 100, dtype=np.int32)
    off = np.arange(G + 1, dtype=np.int32)
    rl = np.full(G, 28, dtype=np.int32)
    want, _ = _compare(P, off, rl, 1024)
    assert want["order"].tolist() == list(range(G))
    assert (np.diff(want["row_group_off"]) == 8).all()


def test_errors_reported_in_status():
    got = _gpu(np.array([5, 50], dtype=np.int32), np.array([0, 1, 2], dtype=np.int32),
               np.array([3, 60], dtype=np.int32), 100)
    assert got["status"] == (2, 1) and got["row_group_off"].numel() == 1
    got = _gpu(np.array([5, 0], dtype=np.int32), np.array([0, 1, 2], dtype=np.int32),
               np.array([3, 6], dtype=np.int32), 100)
    assert got["status"] == (1, 1)


def test_output_feeds_the_plan_builder():
    """The reordered descriptors + row offsets are a valid problem for pp_build_plan with
    descriptors on the device; the plan's tiles cover exactly the builder's tokens."""
    from paper_2602_24082_b200 import binding as B
    rng = np.random.default_rng(9)
    P, off, rl = _random_groups(rng, 40, 500)
    tok = R.group_tokens(P, off, rl)
    got = _gpu(P, off, rl, int(tok.max() * 2))
    T = int(got["row_tokens"].sum().item())
    assert T == int(tok.sum())
    desc_dev = [got["row_group_off"].contiguous(), got["grp_prompt_len"], got["grp_resp_off"], got["resp_len"]]
    desc = [x.cpu().numpy() for x in desc_dev]
    plan = B.pp_build_plan(desc, 4, 2, 64, T, "cuda:0", device_arrays=desc_dev)
    assert plan.status() == (0, 0)
    tiles = plan.read()[0]
    assert int(tiles[:, 1].sum()) == T


@pytest.mark.parametrize("rows,ranks,seed", [(1, 1, 0), (6, 3, 1), (3, 8, 2), (100, 8, 3), (777, 64, 4),
                                             (5000, 1024, 5), (4096, 7, 6)])
def test_assign_rows_matches_the_oracle_bit_for_bit(rows, ranks, seed):
    from paper_2602_24082_b200 import binding as B
    rng = np.random.default_rng(seed)
    cost = rng.integers(0, 1 << 40, size=rows).astype(np.int64)
    if seed == 3:
        cost[::3] = cost[0]                      # ties
    order, rank_of_row, rank_cost = B.pp_assign_rows(torch.from_numpy(cost).cuda(), ranks)
    want = R.assign_rows(cost, ranks)
    assert np.array_equal(order.cpu().numpy(), want[0])
    assert np.array_equal(rank_of_row.cpu().numpy(), want[1])
    assert np.array_equal(rank_cost.cpu().numpy(), want[2])


def test_assign_rows_worked_example_and_hand_over_from_the_row_builder():
    from paper_2602_24082_b200 import binding as B
    order, rank_of_row, rank_cost = B.pp_assign_rows(torch.tensor([7, 3, 9, 3, 5, 1], dtype=torch.int64).cuda(), 3)
    assert rank_of_row.tolist() == [1, 2, 0, 1, 2, 2] and rank_cost.tolist() == [9, 10, 9]
    rng = np.random.default_rng(9)
    P, off, rl = _random_groups(rng, 400, 500)
    tok = R.group_tokens(P, off, rl)
    got = _gpu(P, off, rl, int(tok.max() * 3))
    o2, r2, c2 = B.pp_assign_rows(got["row_cost"], 8)           # device to device, no copy back
    want = R.assign_rows(got["row_cost"].cpu().numpy(), 8)
    assert np.array_equal(r2.cpu().numpy(), want[1]) and np.array_equal(c2.cpu().numpy(), want[2])
    cost = got["row_cost"].cpu().numpy()
    assert c2.max().item() <= cost.sum() / 8 + cost.max()


def test_assign_rows_errors():
    from paper_2602_24082_b200 import binding as B
    c = torch.ones(4, dtype=torch.int64).cuda()
    with pytest.raises(B.PPError) as e:
        B.pp_assign_rows(c, 0)
    assert e.value.code == -1
    with pytest.raises(B.PPError) as e:
        B.pp_assign_rows(c, 2000)
    assert e.value.code == -2
