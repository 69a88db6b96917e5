"""GPU parity of the loss-side consumer against the numpy oracle (fp32 sums vs fp64)."""
import numpy as np
import pytest
import torch

from oracle import loss as L
from paper_2602_24082_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    W.config0(),
    W.Workload("ragged", [[(257, (5, 128, 31))], [(1, (1, 300))]], 4, 2, 128, seed=4),
    W.Workload("single", [[(97, (64,)), (128, (128, 128, 7, 9, 40))], [(700, (1, 1))]], 2, 2, 64, seed=5),
    W.config2(),
    W.config4(3),
] + [W.random_structure(s) for s in range(8)]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("with_ref", [True, False], ids=["dpo", "noref"])
def test_preference_loss_parity(w, with_ref):
    from paper_2602_24082_b200 import binding as B
    rng = np.random.default_rng(7)
    T = w.total_tokens
    lp = (-rng.gamma(2.0, 1.0, T)).astype(np.float32)
    ref = (-rng.gamma(2.0, 1.0, T)).astype(np.float32) if with_ref else None
    beta = 0.1 if with_ref else 0.01
    plan = B.plan_for(w, desc_on_device=True)
    out = B.pp_preference_loss(plan, torch.from_numpy(lp).cuda(),
                               torch.from_numpy(ref).cuda() if with_ref else None, beta)
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    s, r, loss, grad = (x.cpu().numpy().astype(np.float64) for x in out)
    S, Rw, Ls, G = L.preference_loss(w.rows, lp, ref, beta)
    # fp32 sums of up to a few thousand O(1) terms: relative 1e-5 of the magnitude
    assert np.abs(s - S).max() <= 1e-5 * max(1.0, np.abs(S).max())
    assert np.abs(r - Rw).max() <= 2e-5 * max(1.0, np.abs(Rw).max()) + 1e-5
    assert np.abs(loss - Ls).max() <= 1e-4 * max(1.0, np.abs(Ls).max())
    assert np.abs(grad - G).max() <= 1e-4 * max(1e-3, np.abs(G).max())
    # prompt tokens carry no gradient: exactly zero
    prompt = np.zeros(T, dtype=bool)
    for (st, ln, _, _, seg) in w.segments():
        if seg == 0:
            prompt[st:st + ln] = True
    assert not grad[prompt].any()
