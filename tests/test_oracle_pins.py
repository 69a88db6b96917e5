"""Pins for the CPU oracle: each test checks it against something that is not its own code.

P1  packed == unpacked [x, y_k] plain causal attention (the paper's Sec. 3.2 identity),
    outputs and gradients, the reference being textbook torch fp64 ops + autograd;
P2  torch fp64 masked attention with a mask built here from the segment lengths;
P3  closed forms for Q = 0 (LSE = ln count, O = mean of the visible V rows);
P4  one response per group reduces to ordinary causal attention (torch SDPA);
P5  central finite differences of <dO, O>;
P6  invariants: independence from sibling responses, permutation equivariance;
P7  the bookkeeping count of visible pairs equals the dense mask's popcount.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2602_24082_b200 import workloads as W

torch.set_default_dtype(torch.float32)


def _f64(x):
    return x.to(torch.float64)


def _python_mask(w):
    """Independent re-statement of the mask from the segment lengths (global T x T)."""
    T = w.total_tokens
    m = torch.zeros(T, T, dtype=torch.bool)
    t = 0
    for row in w.rows:
        for (p, rs) in row:
            for i in range(p):
                m[t + i, t:t + i + 1] = True
            off = t + p
            for r in rs:
                for i in range(r):
                    m[off + i, t:t + p] = True
                    m[off + i, off:off + i + 1] = True
                off += r
            t = off
    return m


def _torch_masked_attention(q, k, v, mask, scale):
    """softmax(scale Q K^T + mask) V per head with GQA; returns O [T,Hq,D], LSE [Hq,T]."""
    T, Hq, D = q.shape
    r = Hq // k.shape[1]
    kk = k.repeat_interleave(r, dim=1)
    vv = v.repeat_interleave(r, dim=1)
    s = torch.einsum("ihd,jhd->hij", q, kk) * scale
    s = s.masked_fill(~mask[None], float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    o = torch.einsum("hij,jhd->ihd", torch.softmax(s, dim=-1), vv)
    return o, lse


CASES = [
    dict(seed=11, num_rows=1, groups_per_row=1, n_resp=2, hq=1, hkv=1, d=8),
    dict(seed=12, num_rows=2, groups_per_row=1, n_resp=3, hq=4, hkv=2, d=4),
    dict(seed=13, num_rows=1, groups_per_row=3, n_resp=2, hq=2, hkv=1, d=8),
    dict(seed=14, num_rows=2, groups_per_row=2, n_resp=1, hq=2, hkv=2, d=4),
    dict(seed=15, num_rows=1, groups_per_row=2, n_resp=4, hq=4, hkv=1, d=8, r_range=(1, 3)),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
def test_p2_torch_masked_attention(case):
    w = W.tiny(**case)
    q, k, v, do = w.tensors()
    mask = _python_mask(w)
    O, LSE, dQ, dK, dV = oracle.attn_fwd_bwd(w.descriptors(), q, k, v, do, w.softmax_scale)
    qf, kf, vf = (_f64(x).requires_grad_(True) for x in (q, k, v))
    o_ref, lse_ref = _torch_masked_attention(qf, kf, vf, mask, w.softmax_scale)
    (o_ref * _f64(do)).sum().backward()
    assert np.abs(O - o_ref.detach().numpy()).max() < 1e-12
    assert np.abs(LSE - lse_ref.detach().numpy()).max() < 1e-12
    assert np.abs(dQ - qf.grad.numpy()).max() < 1e-11
    assert np.abs(dK - kf.grad.numpy()).max() < 1e-11
    assert np.abs(dV - vf.grad.numpy()).max() < 1e-11


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
@pytest.mark.parametrize("weights", ["first", "random"])
def test_p1_unpacked_equivalence(case, weights):
    """Packed outputs/gradients == plain causal attention on every [x, y_k], prompt
    gradients summed over the K runs whose prompt-dO weights sum to one."""
    w = W.tiny(**case)
    q, k, v, do = w.tensors()
    scale = w.softmax_scale
    O, LSE, dQ, dK, dV = oracle.attn_fwd_bwd(w.descriptors(), q, k, v, do, scale)
    qf, kf, vf = (_f64(x).requires_grad_(True) for x in (q, k, v))
    dof = _f64(do)
    rng = np.random.default_rng(case["seed"])
    loss = 0.0
    t = 0
    for row in w.rows:
        for (p, rs) in row:
            K = len(rs)
            wk = np.zeros(K)
            if weights == "first":
                wk[0] = 1.0
            else:
                wk = rng.uniform(0.1, 1.0, K)
                wk /= wk.sum()
            off = t + p
            for kk, r in enumerate(rs):
                idx = torch.tensor(list(range(t, t + p)) + list(range(off, off + r)))
                L = p + r
                causal = torch.tril(torch.ones(L, L, dtype=torch.bool))
                o_run, lse_run = _torch_masked_attention(qf[idx], kf[idx], vf[idx], causal, scale)
                # forward identity on the prompt and on y_k
                assert np.abs(o_run.detach().numpy() - O[idx.numpy()]).max() < 1e-12
                assert np.abs(lse_run.detach().numpy() - LSE[:, idx.numpy()]).max() < 1e-12
                wrow = torch.cat([torch.full((p,), float(wk[kk]), dtype=torch.float64),
                                  torch.ones(r, dtype=torch.float64)])
                loss = loss + (o_run * dof[idx] * wrow[:, None, None]).sum()
                off += r
            t = off
    loss.backward()
    assert np.abs(dQ - qf.grad.numpy()).max() < 1e-11
    assert np.abs(dK - kf.grad.numpy()).max() < 1e-11
    assert np.abs(dV - vf.grad.numpy()).max() < 1e-11


def test_p1_full_prompt_dout_in_every_run_overcounts():
    """The wrong reading (full prompt dO fed to every run) must NOT match: guards the test."""
    w = W.tiny(seed=11, n_resp=2)
    q, k, v, do = w.tensors()
    _, _, dQ, _, _ = oracle.attn_fwd_bwd(w.descriptors(), q, k, v, do, w.softmax_scale)
    (p, rs), = w.rows[0]
    qf, kf, vf = (_f64(x).requires_grad_(True) for x in (q, k, v))
    loss, off = 0.0, p
    for r in rs:
        idx = torch.tensor(list(range(p)) + list(range(off, off + r)))
        causal = torch.tril(torch.ones(p + r, p + r, dtype=torch.bool))
        o_run, _ = _torch_masked_attention(qf[idx], kf[idx], vf[idx], causal, w.softmax_scale)
        loss = loss + (o_run * _f64(do)[idx]).sum()
        off += r
    loss.backward()
    assert np.abs(dQ[:p] - qf.grad.numpy()[:p]).max() > 1e-3


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
def test_p3_zero_query_closed_form(case):
    w = W.tiny(**case)
    q, k, v, _ = w.tensors()
    q = torch.zeros_like(q)
    O, LSE = oracle.attn_fwd(w.descriptors(), q, k, v, w.softmax_scale)
    vf = _f64(v).numpy()
    r = w.num_q_heads // w.num_kv_heads
    t = 0
    for row in w.rows:
        for (p, rs) in row:
            for i in range(p):
                assert np.allclose(LSE[:, t + i], math.log(i + 1), atol=1e-13)
                mean = vf[t:t + i + 1].mean(axis=0)
                assert np.abs(O[t + i] - np.repeat(mean, r, axis=0)).max() < 1e-13
            off = t + p
            for rl in rs:
                for i in range(rl):
                    assert np.allclose(LSE[:, off + i], math.log(p + i + 1), atol=1e-13)
                    vis = np.concatenate([vf[t:t + p], vf[off:off + i + 1]])
                    assert np.abs(O[off + i] - np.repeat(vis.mean(axis=0), r, axis=0)).max() < 1e-13
                off += rl
            t = off


def test_p4_single_response_is_plain_causal():
    w = W.tiny(seed=21, num_rows=1, groups_per_row=1, n_resp=1, p_range=(5, 9), r_range=(4, 7),
               hq=2, hkv=2, d=8)
    q, k, v, do = w.tensors()
    O, LSE, dQ, dK, dV = oracle.attn_fwd_bwd(w.descriptors(), q, k, v, do, w.softmax_scale)
    qf, kf, vf = (_f64(x).transpose(0, 1).unsqueeze(0).requires_grad_(True) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(qf, kf, vf, is_causal=True,
                                                         scale=w.softmax_scale)
    (o * _f64(do).transpose(0, 1).unsqueeze(0)).sum().backward()
    assert np.abs(O - o[0].transpose(0, 1).detach().numpy()).max() < 1e-12
    assert np.abs(dQ - qf.grad[0].transpose(0, 1).numpy()).max() < 1e-11
    assert np.abs(dK - kf.grad[0].transpose(0, 1).numpy()).max() < 1e-11
    assert np.abs(dV - vf.grad[0].transpose(0, 1).numpy()).max() < 1e-11


def test_p4_groups_do_not_interact():
    """Several groups in a row == each group run alone (block-diagonal, batch packing)."""
    w = W.tiny(seed=22, num_rows=1, groups_per_row=3, n_resp=2, hq=2, hkv=1, d=4)
    q, k, v, do = w.tensors()
    full = oracle.attn_fwd_bwd(w.descriptors(), q, k, v, do, w.softmax_scale)
    t = 0
    for (p, rs) in w.rows[0]:
        L = p + sum(rs)
        one = W.Workload("g", [[(p, rs)]], 2, 1, 4, seed=0)
        part = oracle.attn_fwd_bwd(one.descriptors(), q[t:t + L], k[t:t + L], v[t:t + L],
                                   do[t:t + L], w.softmax_scale)
        for a, b, lse in zip(full, part, (0, 1, 0, 0, 0)):
            a = a[:, t:t + L] if lse else a[t:t + L]
            assert np.array_equal(a, b)
        t += L


def test_p5_finite_differences():
    w = W.tiny(seed=31, num_rows=1, groups_per_row=2, n_resp=2, hq=2, hkv=1, d=4)
    q, k, v, do = w.tensors()
    desc, scale = w.descriptors(), w.softmax_scale
    _, _, dQ, dK, dV = oracle.attn_fwd_bwd(desc, q, k, v, do, scale)
    dof = _f64(do).numpy()
    # perturbations must stay exactly representable in bf16: flip to a neighbouring value
    rng = np.random.default_rng(0)
    for name, grad, pos in (("q", dQ, 0), ("k", dK, 1), ("v", dV, 2)):
        base = [q, k, v]
        x = base[pos]
        for _ in range(6):
            idx = tuple(int(rng.integers(0, s)) for s in x.shape)
            x0 = float(x[idx])
            h = 2.0 ** -6 * max(abs(x0), 0.25)      # bf16-representable step (power of two scale)
            xp = x.clone(); xp[idx] = x0 + h
            xm = x.clone(); xm[idx] = x0 - h
            hp, hm = float(xp[idx]) - x0, x0 - float(xm[idx])
            args_p = list(base); args_p[pos] = xp
            args_m = list(base); args_m[pos] = xm
            Op, _ = oracle.attn_fwd(desc, *args_p, scale)
            Om, _ = oracle.attn_fwd(desc, *args_m, scale)
            fd = ((Op - Om) * dof).sum() / (hp + hm)
            assert abs(fd - grad[idx]) <= 2e-3 * max(1.0, abs(grad[idx])), (name, idx, fd, grad[idx])


def test_p6_sibling_independence_and_permutation():
    w = W.Workload("p6", [[(6, (3, 5, 4))]], 2, 1, 8, seed=41)
    q, k, v, do = w.tensors()
    desc, scale = w.descriptors(), w.softmax_scale
    base = oracle.attn_fwd_bwd(desc, q, k, v, do, scale)
    # perturb response 2 (tokens 9..13): prompt and responses 1, 3 outputs must not move
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    q2[9:14] += 1.0; k2[9:14] -= 0.5; v2[9:14] *= 2.0
    pert = oracle.attn_fwd(desc, q2, k2, v2, scale)
    keep = np.r_[0:9, 14:18]
    assert np.array_equal(base[0][keep], pert[0][keep])
    assert np.array_equal(base[1][:, keep], pert[1][:, keep])
    assert not np.array_equal(base[0][9:14], pert[0][9:14])
    # permuting the responses permutes the results
    perm = np.r_[0:6, 9:14, 14:18, 6:9]            # (x, y2, y3, y1)
    wp = W.Workload("p6p", [[(6, (5, 4, 3))]], 2, 1, 8, seed=41)
    pt = torch.from_numpy(perm)
    permd = oracle.attn_fwd_bwd(wp.descriptors(), q[pt], k[pt], v[pt], do[pt], scale)
    for a, b, lse in zip(base, permd, (0, 1, 0, 0, 0)):
        a = a[:, perm] if lse else a[perm]
        # the prompt's dK/dV sums run over the responses in another order: rounding only
        assert np.abs(a - b).max() < 1e-13
    # dK/dV on response-k keys depend only on response-k queries
    do2 = do.clone(); do2[6:9] = 0; do2[14:18] = 0; do2[0:6] = 0
    only2 = oracle.attn_fwd_bwd(desc, q, k, v, do2, scale)
    do3 = do.clone(); do3[9:14] = 0
    without2 = oracle.attn_fwd_bwd(desc, q, k, v, do3, scale)
    assert np.abs(only2[3][9:14] - base[3][9:14]).max() < 1e-13
    assert np.abs(only2[4][9:14] - base[4][9:14]).max() < 1e-13
    assert np.abs(without2[3][9:14]).max() == 0 and np.abs(without2[4][9:14]).max() == 0


def test_p6_intermediate_invariants():
    w = W.tiny(seed=51, num_rows=1, groups_per_row=2, n_resp=2, hq=2, hkv=1, d=8)
    q, k, v, do = w.tensors()
    desc, scale = w.descriptors(), w.softmax_scale
    O, LSE, dQ, dK, dV = oracle.attn_fwd_bwd(desc, q, k, v, do, scale)
    S, P, dP, dS = oracle.dump_intermediates(desc, q, k, v, do, scale, 0, 1)
    mask = _python_mask(w).numpy()
    assert np.array_equal(np.isfinite(S), mask)
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-13
    assert np.abs(dS.sum(axis=1)).max() < 1e-12
    assert (LSE[1] >= np.where(mask, S, -np.inf).max(axis=1) - 1e-15).all()
    # the dumped matrices reproduce the oracle's outputs through plain matrix products
    qf, kf, vf, dof = (_f64(x).numpy() for x in (q, k, v, do))
    assert np.abs(P @ vf[:, 0] - O[:, 1]).max() < 1e-13
    assert np.abs(scale * dS @ kf[:, 0] - dQ[:, 1]).max() < 1e-12
    delta = (dof[:, 1] * O[:, 1]).sum(axis=1)
    assert np.abs((P * dP).sum(axis=1) - delta).max() < 1e-12
    S0, P0, dP0, dS0 = oracle.dump_intermediates(desc, q, k, v, do, scale, 0, 0)
    assert np.abs(P.T @ dof[:, 1] + P0.T @ dof[:, 0] - dV[:, 0]).max() < 1e-12
    assert np.abs(scale * (dS.T @ qf[:, 1] + dS0.T @ qf[:, 0]) - dK[:, 0]).max() < 1e-12


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
def test_p7_mask_and_pair_count(case):
    w = W.tiny(**case)
    desc = w.descriptors()
    mask = _python_mask(w).numpy()
    offs = w.row_offsets()
    total = 0
    for r in range(len(w.rows)):
        m = oracle.dense_mask(desc, r)
        assert np.array_equal(m, mask[offs[r]:offs[r + 1], offs[r]:offs[r + 1]])
        total += int(m.sum())
    # nothing visible across rows
    for r in range(len(w.rows)):
        blk = mask[offs[r]:offs[r + 1]].copy()
        blk[:, offs[r]:offs[r + 1]] = False
        assert not blk.any()
    assert total == w.useful_pairs()
    # column form of the mask: key j is seen by the contiguous queries [j, end_j)
    T = w.total_tokens
    for j in range(T):
        seen = np.nonzero(mask[:, j])[0]
        assert seen[0] == j and np.array_equal(seen, np.arange(j, j + len(seen)))


def test_config0_is_the_stated_tiny_case():
    w = W.config0()
    assert w.total_tokens == 144 and w.useful_pairs() == 8904
    assert oracle.dense_mask(w.descriptors(), 0).sum() == 8904


def test_descriptor_errors():
    with pytest.raises(ValueError):
        oracle.token_ids(([0, 1], [0], [0, 1], [3]))        # empty prompt
    with pytest.raises(ValueError):
        oracle.token_ids(([0, 1], [4], [0, 1], [0]))        # empty response
