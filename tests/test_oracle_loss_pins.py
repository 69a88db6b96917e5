"""Pins for the loss-side oracle (oracle/loss.py)."""
import math

import numpy as np
import torch

from oracle import loss as L
from paper_2602_24082_b200 import workloads as W


def _inputs(w, seed):
    rng = np.random.default_rng(seed)
    T = w.total_tokens
    return -rng.gamma(2.0, 1.0, T), -rng.gamma(2.0, 1.0, T)


def test_matches_torch_logsigmoid_and_autograd_on_sliced_sequences():
    w = W.Workload("l", [[(5, (2, 4, 3)), (3, (1, 6))], [(7, (3, 3))]], 1, 1, 8, seed=0)
    lp, ref = _inputs(w, 1)
    beta = 0.3
    s, r, loss, grad = L.preference_loss(w.rows, lp, ref, beta)
    tl = torch.tensor(lp, dtype=torch.float64, requires_grad=True)
    tr = torch.tensor(ref, dtype=torch.float64)
    total, losses, t = 0.0, [], 0
    for row in w.rows:
        for (p, rs) in row:
            off, rew = t + p, []
            for rl in rs:
                rew.append(beta * (tl[off:off + rl].sum() - tr[off:off + rl].sum()))
                off += rl
            pairs = [(a, b) for a in range(len(rs)) for b in range(a)]
            gl = sum(-torch.nn.functional.logsigmoid(rew[a] - rew[b]) for a, b in pairs) / len(pairs)
            losses.append(float(gl.detach()))
            total = total + gl
            t = off
    total.backward()
    assert np.abs(loss - np.array(losses)).max() < 1e-12
    assert np.abs(grad - tl.grad.numpy()).max() < 1e-12


def test_pairwise_closed_form_and_equal_rewards():
    """K = 2: the DPO loss -log sigmoid(beta ((s_w - s_w_ref) - (s_l - s_l_ref))) with the later
    response preferred; equal rewards give log 2."""
    w = W.Workload("l2", [[(4, (3, 2))]], 1, 1, 8, seed=0)
    lp, ref = _inputs(w, 2)
    beta = 0.1
    s, r, loss, _ = L.preference_loss(w.rows, lp, ref, beta)
    s_l, s_w = lp[4:7].sum(), lp[7:9].sum()
    r_l, r_w = ref[4:7].sum(), ref[7:9].sum()
    x = beta * ((s_w - r_w) - (s_l - r_l))
    assert abs(loss[0] - math.log1p(math.exp(-x))) < 1e-12
    assert np.allclose(s, [s_l, s_w])
    same = np.full(9, -0.5)
    _, _, loss2, g2 = L.preference_loss([[(3, (3, 3))]], same, same, 1.0)
    assert abs(loss2[0] - math.log(2)) < 1e-15
    # no reference: rewards are beta * sums; a single response has no pair
    _, r3, loss3, g3 = L.preference_loss([[(2, (3,))]], np.array([0, 0, -1.0, -2.0, -3.0]), None, 2.0)
    assert r3[0] == -12.0 and loss3[0] == 0.0 and not g3.any()


def test_finite_differences_and_prompt_tokens_have_no_gradient():
    w = W.Workload("l3", [[(3, (2, 3, 2))]], 1, 1, 8, seed=0)
    lp, ref = _inputs(w, 3)
    _, _, _, grad = L.preference_loss(w.rows, lp, ref, 0.7)
    assert not grad[:3].any()
    for t in (3, 5, 8):
        e = np.zeros_like(lp); e[t] = 1e-6
        lp_, lm_ = L.preference_loss(w.rows, lp + e, ref, 0.7)[2].sum(), L.preference_loss(w.rows, lp - e, ref, 0.7)[2].sum()
        assert abs((lp_ - lm_) / 2e-6 - grad[t]) < 1e-8
