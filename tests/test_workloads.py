"""Host-side checks of the synthetic workload recipes and of the paper's cost model."""
import os

import numpy as np
import pytest

from paper_2602_24082_b200 import cost_model
from paper_2602_24082_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _table(name):
    rows = []
    for line in open(os.path.join(GOLDEN, name)):
        if line.strip() and not line.startswith("#"):
            f = line.split()
            rows.append((f[0], [float(x) for x in f[1:]]))
    return rows


def test_table1_is_self_consistent_and_eq1_holds():
    """Sec. 5.1: effective time = memory ratio x time ratio; Eq. (1) holds for all three
    datasets (the paper says the condition 'is largely satisfied')."""
    for name, (l_in, rmax, rmin, mem, t, eff) in _table("table1.txt"):
        assert abs(mem * t - eff) < 1.5e-3, name
        assert cost_model.packing_wins(l_in, [rmax, rmin]), name
        assert cost_model.attention_cost_ratio(l_in, [rmax, rmin]) < 1
        assert cost_model.memory_ratio(l_in, [rmax, rmin]) <= 1


def test_table2_combined_gain():
    t = dict((k, v[0]) for k, v in _table("table2.txt"))
    assert abs(t["both"] / t["batch_sorting"] - 1.23) < 0.005     # "approximately 23%"


def test_cost_model_closed_forms():
    # equal responses: ratio (l+K r)^2 / (K (l+r)^2); K=1 -> 1
    assert cost_model.attention_cost_ratio(100, [50]) == pytest.approx(1.0)
    assert cost_model.memory_ratio(100, [50]) == pytest.approx(1.0)
    assert cost_model.attention_cost_ratio(0, [10, 10]) == pytest.approx(2.0)
    assert cost_model.memory_ratio(7, [5, 5, 5]) == pytest.approx(22 / 36)
    assert not cost_model.packing_wins(1, [100, 100])          # Limitations: long responses lose


def test_recipes_shapes():
    c0 = W.config0()
    assert c0.rows == [[(64, (32, 48))]] and c0.head_dim == 64 and c0.seed == 0
    c1 = W.config1()
    assert len(c1.rows) == 8 and (c1.num_q_heads, c1.num_kv_heads, c1.head_dim) == (32, 8, 128)
    for (p, rs), in c1.rows:
        assert 64 <= p <= 2048 and len(rs) == 2 and all(64 <= r <= 512 for r in rs)
    c2 = W.config2()
    assert len(c2.rows) == 4 and (c2.num_q_heads, c2.num_kv_heads) == (28, 4)
    for ((p, rs),), (lo, hi) in zip(c2.rows, c2.low_var_ranges):
        assert 1024 <= p <= 4096 and len(rs) == 4 and all(128 <= r <= 1024 for r in rs)
        assert 1024 <= hi - lo <= min(2048, p)
    c3 = W.config3()
    assert c3.row_lengths() == [8192, 8192] and (c3.num_q_heads, c3.num_kv_heads) == (64, 8)
    assert all(len(rs) == 2 and p >= 1 and min(rs) >= 1 for row in c3.rows for p, rs in row)
    for s, (rho, n) in enumerate(W.CONFIG4_POINTS):
        c4 = W.config4(s)
        assert c4.row_lengths() == [32768, 32768]
        tot = [p + sum(rs) for row in c4.rows for p, rs in row]
        # length-sorted within what was poured before the shrunk tail of each row
        assert all(len(rs) == n or len(rs) >= 1 for row in c4.rows for p, rs in row)
        first_row = [p + sum(rs) for p, rs in c4.rows[0][:-1]]
        assert first_row == sorted(first_row, reverse=True)


def test_recipes_are_deterministic_and_descriptors_consistent():
    for w in (W.config1(), W.config3(), W.config4(3)):
        w2 = type(w)(**{f: getattr(w, f) for f in ("name", "rows", "num_q_heads", "num_kv_heads",
                                                     "head_dim", "seed")})
        assert w2.rows == w.rows
        rgo, gpl, gro, rl = w.descriptors()
        assert rgo[-1] == len(gpl) and gro[-1] == len(rl)
        assert int(gpl.sum() + rl.sum()) == w.total_tokens
        segs = w.segments()
        assert segs[0][0] == 0 and all(a[0] + a[1] == b[0] for a, b in zip(segs, segs[1:]))
    assert W.config1().rows == W.config1().rows


def test_tensors_seeded_and_low_variance_prefix():
    w = W.config0()
    a, b = w.tensors(), w.tensors()
    assert all((x.view(dtype=__import__("torch").int16) == y.view(dtype=__import__("torch").int16)).all()
               for x, y in zip(a, b))
    small = W.Workload("s", [[(2000, (40, 30))]], 2, 1, 16, seed=5,
                       low_var_ranges=[(0, 1500)], low_std=0.5 ** 0.5)
    q, k, v, do = small.tensors()
    assert abs(float(q[:1500].float().var()) - 0.5) < 0.03
    assert abs(float(q[1500:].float().var()) - 1.0) < 0.08
    assert abs(float(do[:1500].float().var()) - 1.0) < 0.03


def test_unpacked_baseline_structure():
    w = W.Workload("u", [[(5, (2, 4))], [(3, (1, 1, 2))]], 2, 1, 8, seed=1)
    up, gather = W.unpacked(w, padded=True)
    assert up.rows == [[(5, (4,)), (5, (4,))], [(3, (2,)), (3, (2,)), (3, (2,))]]
    assert len(gather) == up.total_tokens == 18 + 15
    assert gather[:5].tolist() == [0, 1, 2, 3, 4] and gather[5:7].tolist() == [5, 6]
    assert gather[9:14].tolist() == [0, 1, 2, 3, 4] and gather[14:18].tolist() == [7, 8, 9, 10]
    un, g2 = W.unpacked(w, padded=False)
    assert un.rows == [[(5, (2,)), (5, (4,))], [(3, (1,)), (3, (1,)), (3, (2,))]]
    # F4: unpacked-unpadded pairs exceed packed pairs by (K-1) P (P+1) / 2 per group
    extra = sum((len(rs) - 1) * p * (p + 1) // 2 for row in w.rows for p, rs in row)
    assert un.useful_pairs() - w.useful_pairs() == extra


def test_slice_heads_is_an_independent_subproblem():
    w = W.Workload("s", [[(5, (2, 4))], [(3, (1, 2))]], 4, 2, 8, seed=2)
    tens = w.tensors()
    sub, (q, k, v, do), tok, qh = W.slice_heads(w, tens, [1], [1])
    assert sub.rows == [w.rows[1]] and sub.num_q_heads == 2 and sub.num_kv_heads == 1
    assert tok.tolist() == list(range(11, 17)) and qh.tolist() == [2, 3]
    assert (q == tens[0][11:17][:, 2:4]).all() and (k == tens[1][11:17][:, 1:2]).all()
