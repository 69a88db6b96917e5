"""GPU parity of the packed position ids and the rotary embedding against the numpy oracle."""
import numpy as np
import pytest
import torch

from oracle import rope as R
from paper_2602_24082_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    W.config0(),
    W.Workload("ragged", [[(257, (5, 128, 31))], [(1, (1, 300))]], 4, 2, 128, seed=4),
    W.Workload("groups", [[(97, (64, 200)), (128, (128, 128)), (3, (2, 1))], [(700, (1,))]], 2, 2, 64, seed=5),
    W.Workload("d96", [[(97, (64, 200)), (3, (2, 1))], [(130, (1, 40))]], 6, 2, 96, seed=6),
] + [W.random_structure(s) for s in range(8)]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_position_ids_bit_exact(w):
    from paper_2602_24082_b200 import binding as B
    plan = B.plan_for(w)
    pos = B.pp_position_ids(plan).cpu().numpy()
    assert plan.status() == (0, 0)
    assert np.array_equal(pos.astype(np.int64), R.position_ids(w.rows))


def test_position_ids_full_size_configs():
    from paper_2602_24082_b200 import binding as B
    for w in (W.config1(), W.config3(), W.config4(1)):
        plan = B.plan_for(w, desc_on_device=True)
        pos = B.pp_position_ids(plan).cpu().numpy()
        assert np.array_equal(pos.astype(np.int64), R.position_ids(w.rows))


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("base", [10000.0, 500000.0])
def test_rope_parity(w, base):
    """bf16 outputs: max-abs within one bf16 half-ulp of the largest value plus slack (2e-2),
    relative L2 within 4e-3 (bf16 rounding alone gives about 2e-3)."""
    from paper_2602_24082_b200 import binding as B
    q, k, _, _ = w.tensors()
    plan = B.plan_for(w)
    qd, kd = q.cuda().clone(), k.cuda().clone()
    B.pp_rope_qk(plan, qd, kd, base)
    torch.cuda.synchronize()
    pos = R.position_ids(w.rows)
    for got, src in ((qd, q), (kd, k)):
        ref = R.rope(src.double().numpy(), pos, base)
        g = got.float().cpu().numpy().astype(np.float64)
        assert np.abs(g - ref).max() <= 2e-2
        assert np.linalg.norm(g - ref) / np.linalg.norm(ref) <= 4e-3


def test_rope_then_attention_equals_unpacked_with_plain_positions():
    """End to end: rotary with packed positions + packed attention == plain positions + plain
    causal attention on every (x, y_k) (compared through the GPU path itself, bit for bit on
    the rotated inputs and within rounding on the outputs)."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("e2e", [[(150, (70, 129))]], 2, 1, 128, seed=11)
    q, k, v, _ = (x.cuda() for x in w.tensors())
    plan = B.plan_for(w)
    B.pp_rope_qk(plan, q, k, 10000.0)
    o, _ = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
    (p, rs), = w.rows[0]
    off = p
    q0, k0, v0, _ = (x.cuda() for x in w.tensors())
    for r in rs:
        idx = torch.tensor(list(range(p)) + list(range(off, off + r)), device="cuda")
        uw = W.Workload("u", [[(p, (r,))]], 2, 1, 128, seed=0)
        uplan = B.plan_for(uw)
        uq, uk, uv = q0[idx].contiguous(), k0[idx].contiguous(), v0[idx].contiguous()
        B.pp_rope_qk(uplan, uq, uk, 10000.0)
        assert torch.equal(uq, q[idx]) and torch.equal(uk, k[idx])
        uo, _ = B.pp_attn_fwd(uplan, uq, uk, uv, w.softmax_scale)
        assert (uo.float() - o[idx].float()).abs().max().item() <= 2e-2
        off += r


def test_rope_with_element_offsets_beyond_32_bits():
    """Q of more than 2^31 elements: the rotation of the last tokens (largest offsets) and of
    the tokens around the 2^31-element mark against the oracle, position ids bit for bit."""
    from paper_2602_24082_b200 import binding as B
    big = (8192, (4096, 4096))
    w = W.Workload("beyond-32-bit", [[big] * 32 + [(520, (300, 200))] + [big] + [(77, (130, 1, 64))]],
                   32, 8, 128, seed=91)
    T = w.total_tokens
    assert T * 32 * 128 > 2 ** 31
    g = torch.Generator().manual_seed(5)
    q = torch.randn(T, 32, 128, generator=g, dtype=torch.float32).to(torch.bfloat16)
    k = torch.randn(T, 8, 128, generator=g, dtype=torch.float32).to(torch.bfloat16)
    plan = B.plan_for(w, desc_on_device=True)
    pos_gpu = B.pp_position_ids(plan).cpu().numpy()
    pos = R.position_ids(w.rows)
    assert np.array_equal(pos_gpu, pos)
    qd, kd = q.cuda(), k.cuda()
    B.pp_rope_qk(plan, qd, kd, 10000.0)
    torch.cuda.synchronize()
    for lo, hi in ((32 * 16384 - 64, 32 * 16384 + 600), (T - 300, T)):
        for got, src in ((qd, q), (kd, k)):
            ref = R.rope(src[lo:hi].double().numpy(), pos[lo:hi], 10000.0)
            out = got[lo:hi].float().cpu().numpy().astype(np.float64)
            assert np.abs(out - ref).max() <= 2e-2
            assert np.linalg.norm(out - ref) / np.linalg.norm(ref) <= 4e-3
