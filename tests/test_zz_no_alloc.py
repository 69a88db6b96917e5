"""pp_attn_bwd_noalloc: the backward for callers that cannot allocate device memory.

Such callers (plug-ins inside an application that owns the device heap, code running once
memory is fully committed, loops where cudaMalloc's possible device synchronisation is not
allowed) cannot give the library a scratch buffer, so this entry point uses an array built
into the library instead.  The test calls it through the C ABI twice in a row, on different
inputs, and compares each result with the ordinary pp_attn_bwd on the same inputs: the
second call must not see anything the first one left in the shared array.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.  It passes on its own in a fresh process as well as after the others.
"""
import numpy as np
import pytest
import torch

from paper_2602_24082_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _rel_l2(a, b):
    a, b = a.float(), b.float()
    return float((a - b).norm() / b.norm().clamp_min(1e-30))


def test_noalloc_backward_matches_regular_backward_twice():
    from paper_2602_24082_b200 import binding as B
    # same shapes, different values: call 2 would go wrong if call 1's accumulator survived
    shapes = [[(257, (5, 128, 31))], [(1, (1, 300))]]
    for seed in (21, 22):
        w = W.Workload("noalloc", shapes, 4, 2, 128, seed=seed)
        q, k, v, do = (x.cuda() for x in w.tensors())
        plan = B.plan_for(w)
        assert plan.bwd_scratch_bytes <= B.pp_attn_bwd_noalloc_max_bytes()
        o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
        ref_dq, ref_dk, ref_dv = B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)
        dq, dk, dv = torch.full_like(q, 9.0), torch.full_like(k, 9.0), torch.full_like(v, 9.0)
        B.pp_attn_bwd_noalloc(plan, q, k, v, o, lse, do, w.softmax_scale, dq, dk, dv)
        torch.cuda.synchronize()
        assert plan.status() == (0, 0)
        # dK and dV have a fixed summation order: identical.  dQ is summed by floating-point
        # reductions in arbitrary order: same tolerance as the run-to-run determinism test.
        assert torch.equal(dk, ref_dk) and torch.equal(dv, ref_dv)
        assert _rel_l2(dq, ref_dq) < 1e-3
        assert B.pp_last_launch_count() == 3


def test_noalloc_rejects_problems_beyond_the_builtin_scratch():
    from paper_2602_24082_b200 import binding as B
    limit = B.pp_attn_bwd_noalloc_max_bytes()
    assert limit == 32 << 20
    w = W.Workload("big", [[(1500, (300, 300))]], 32, 8, 128, seed=1)      # 4*T*Hq*D = 34 MB
    plan = B.plan_for(w)
    assert plan.bwd_scratch_bytes > limit
    T = w.total_tokens
    mk = lambda h: torch.zeros(T, h, 128, dtype=torch.bfloat16, device="cuda")
    q, o, do, dq = mk(32), mk(32), mk(32), mk(32)
    k, v, dk, dv = mk(8), mk(8), mk(8), mk(8)
    lse = torch.zeros(32, T, dtype=torch.float32, device="cuda")
    dq.fill_(5.0)
    with pytest.raises(B.PPError) as e:
        B.pp_attn_bwd_noalloc(plan, q, k, v, o, lse, do, w.softmax_scale, dq, dk, dv)
    assert e.value.code == -7 and "32 MiB" in str(e.value)
    torch.cuda.synchronize()
    assert (dq == 5.0).all()          # nothing was launched
