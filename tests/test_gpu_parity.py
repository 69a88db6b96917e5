"""GPU parity: the CUDA path (through the C ABI) against the CPU fp64 oracle, element by
element on the same seeded inputs.

Tolerances (for unit-normal bf16 inputs): max-abs 2e-2 on O, 5e-3 on LSE, relative L2 2e-2
on dQ / dK / dV -- also checked per segment kind (prompt tokens only, response tokens only) so
that an error confined to short segments cannot hide inside a global norm.
"""
import numpy as np
import pytest
import torch

from paper_2602_24082_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL_O, TOL_LSE, TOL_GRAD = 2e-2, 5e-3, 2e-2


def _run_gpu(w, tens, desc_on_device=False, for_backward=False):
    """``for_backward``: the forward gets the backward's scratch and clears the dQ accumulator
    in it (the path the benchmark times); the scratch is filled with NaN bit patterns first, so
    a row the forward failed to clear would show."""
    from paper_2602_24082_b200 import binding as B
    q, k, v, do = (x.cuda() for x in tens)
    plan = B.plan_for(w, desc_on_device=desc_on_device)
    if for_backward:
        plan.bwd_scratch().fill_(0xFF)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, for_backward=for_backward)
    dq, dk, dv = B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    return tuple(x.float().cpu().numpy().astype(np.float64) for x in (o, lse, dq, dk, dv))


def _rel_l2(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def check_against_oracle(w, tens, gpu):
    import oracle
    O, LSE, dQ, dK, dV = oracle.attn_fwd_bwd(w.descriptors(), *tens, w.softmax_scale)
    o, lse, dq, dk, dv = gpu
    assert np.isfinite(o).all() and np.isfinite(lse).all()
    assert np.abs(o - O).max() <= TOL_O, f"O max-abs {np.abs(o - O).max()}"
    assert np.abs(lse - LSE).max() <= TOL_LSE, f"LSE max-abs {np.abs(lse - LSE).max()}"
    prompt = np.zeros(w.total_tokens, dtype=bool)
    for (s, l, _, _, seg) in w.segments():
        if seg == 0:
            prompt[s:s + l] = True
    def part_err(g, ref, part):
        # A part can have an exactly zero gradient (the dQ of a one-token prompt: its only
        # query sees only itself, the softmax is the constant 1); its error is then measured
        # against the share of the whole tensor's norm that a part of this size would carry.
        floor = 1e-2 * np.linalg.norm(ref) * np.sqrt(part.mean())
        return float(np.linalg.norm(g[part] - ref[part]) / max(np.linalg.norm(ref[part]), floor, 1e-30))

    for name, g, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
        assert np.isfinite(g).all(), name
        assert _rel_l2(g, ref) <= TOL_GRAD, f"{name} rel-L2 {_rel_l2(g, ref)}"
        assert part_err(g, ref, prompt) <= TOL_GRAD, f"{name} prompt rel-L2 {part_err(g, ref, prompt)}"
        assert part_err(g, ref, ~prompt) <= TOL_GRAD, f"{name} response rel-L2"


def test_config0_full():
    w = W.config0()
    tens = w.tensors()
    check_against_oracle(w, tens, _run_gpu(w, tens))


RAGGED = [
    # name, rows, Hq, Hkv, D   -- lengths around the tile size, primes, length-1 segments
    ("d64-ragged", [[(130, (1, 127, 129))]], 2, 1, 64),
    ("d128-ragged", [[(257, (5, 128, 31))], [(1, (1, 300))]], 4, 2, 128),
    ("d128-groups", [[(97, (64, 200)), (128, (128, 128)), (3, (2, 1))]], 2, 2, 128),
    ("d64-gqa4", [[(300, (140, 10, 77, 129))]], 4, 1, 64),
    ("d128-single-response", [[(200, (333,))]], 2, 1, 128),
    # backward key tiles are cut per group: tiles that hold the prompt's tail and several
    # whole responses, responses of one token, segment boundaries on and next to tile edges
    ("d64-many-short-responses", [[(100, (7, 1, 30, 1, 1, 64, 2, 90, 13))]], 2, 1, 64),
    ("d128-aligned-and-off-by-one", [[(128, (128, 127, 129)), (127, (1, 128)), (129, (130,))]], 2, 2, 128),
    ("d64-150-one-token-responses", [[(130, tuple([1] * 150))]], 2, 1, 64),
    ("d128-prompt-of-one", [[(1, (400, 1, 129))], [(1, (1,))]], 3, 1, 128),
    ("d128-exact-tiles", [[(256, (128, 256, 128))], [(128, (128,))]], 5, 5, 128),
    # a token's heads span 16 KB: the backward's preprocess walks memory order from there on
    ("d128-wide-heads", [[(70, (33, 129))], [(5, (64,))]], 64, 16, 128),
    # head_dim 96 runs in tiles of 128 whose upper columns the TMA loads fill with zeros
    ("d96-ragged", [[(257, (5, 128, 31))], [(1, (1, 300))]], 4, 2, 96),
    ("d96-groups-gqa3", [[(97, (64, 200)), (128, (128, 128)), (3, (2, 1))], [(300, (140, 10, 129))]], 6, 2, 96),
    ("d96-wide-heads", [[(70, (33, 129))], [(5, (64,))]], 96, 16, 96),
]


@pytest.mark.parametrize("name,rows,hq,hkv,d", RAGGED, ids=[r[0] for r in RAGGED])
@pytest.mark.parametrize("desc_on_device", [False, True], ids=["hostdesc", "devdesc"])
def test_ragged_shapes(name, rows, hq, hkv, d, desc_on_device):
    w = W.Workload(name, rows, hq, hkv, d, seed=100 + len(name))
    tens = w.tensors()
    check_against_oracle(w, tens, _run_gpu(w, tens, desc_on_device, for_backward=desc_on_device))


@pytest.mark.parametrize("seed", range(48))
def test_random_structures(seed):
    """Oracle parity on random structures; every other one also through the host step and
    the deterministic backward, which must agree with the default path (O, LSE, dK, dV bit
    for bit)."""
    from paper_2602_24082_b200 import binding as B
    w = W.random_structure(seed)
    tens = w.tensors()
    gpu = _run_gpu(w, tens, desc_on_device=bool(seed & 1), for_backward=bool(seed & 2))
    check_against_oracle(w, tens, gpu)
    if seed % 2 == 0:
        hs = B.HostStep(w)
        hs(*[t.contiguous().pin_memory() for t in tens])
        torch.cuda.synchronize()
        got = [x.float().numpy().astype(np.float64) for x in (hs.o, hs.lse, hs.dq, hs.dk, hs.dv)]
        for i in (0, 1, 3, 4):
            assert np.array_equal(got[i], gpu[i])
        assert _rel_l2(got[2], gpu[2]) < 1e-3
        q, k, v, do = (x.cuda() for x in tens)
        plan = B.plan_for(w)
        o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
        runs = [B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, deterministic=True)
                for _ in range(2)]
        torch.cuda.synchronize()
        assert plan.status() == (0, 0)
        for a, b in zip(*runs):
            assert torch.equal(a, b)
        assert _rel_l2(runs[0][0].float().cpu().numpy().astype(np.float64), gpu[2]) < 1e-3


@pytest.mark.parametrize("seed", range(100, 112))
def test_random_structures_head_dim_96(seed):
    """The random structures again with head_dim 96 (tiles of 128 with zero-filled columns)."""
    base = W.random_structure(seed, long=(seed % 4 == 0))
    w = W.Workload(f"random-d96-{seed}", base.rows, base.num_q_heads, base.num_kv_heads, 96,
                   seed=2000 + seed)
    tens = w.tensors()
    check_against_oracle(w, tens, _run_gpu(w, tens, desc_on_device=bool(seed & 1),
                                           for_backward=bool(seed & 2)))


@pytest.mark.parametrize("d", [64, 96, 128])
def test_growing_scores_take_the_rescale_path(d):
    """Later keys score far higher than earlier ones (queries and keys of later token ranges are
    amplified), so a row's running maximum jumps by more than the forward's lazy-rescale
    threshold (2^8) from one key tile to the next: the accumulator is rescaled and the tile
    redone.  Unit-variance inputs almost never get there."""
    w = W.Workload("growing", [[(600, (300, 200))], [(130, (270,))]], 4, 2, d, seed=77)
    q, k, v, do = w.tensors()
    T = w.total_tokens
    gain = torch.ones(T)
    for lo, hi, g in ((250, 420, 1.8), (420, 600, 2.6), (700, 900, 2.6), (950, 1100, 3.0), (1300, 1500, 2.4)):
        gain[lo:hi] = g
    q = (q.float() * gain[:, None, None]).to(q.dtype)
    k = (k.float() * gain[:, None, None]).to(k.dtype)
    tens = (q, k, v, do)
    # the jumps are there: per 128-key tile, the row maxima of the scaled scores in log2 units
    s = torch.einsum("qd,kd->qk", q[:600, 0].float(), k[:600, 0].float()) * w.softmax_scale * 1.4426950408889634
    s = s.masked_fill(torch.triu(torch.ones(600, 600, dtype=torch.bool), 1), float("-inf"))
    run = torch.cummax(torch.stack([s[:, i:i + 128].max(dim=1).values for i in range(0, 600, 128)], 1), 1).values
    assert ((run[:, 1:] - run[:, :-1]) > 8).any(dim=1).float().mean() > 0.1   # of the prompt rows
    check_against_oracle(w, tens, _run_gpu(w, tens, for_backward=True))


@pytest.mark.parametrize("seed", range(6))
def test_random_long_structures(seed):
    """Segments of many tiles: the whole workload on the GPU, one KV-head group of it against
    the oracle."""
    w = W.random_structure(seed, long=True)
    _subset_parity(w, list(range(len(w.rows))), [seed % w.num_kv_heads])


def _subset_parity(w, row_ids, kv_heads):
    """Run the GPU on the whole workload, compare an independent sub-problem with the oracle."""
    tens = w.tensors()
    gpu = _run_gpu(w, tens)
    sub, stens, tok, qh = W.slice_heads(w, tens, row_ids, kv_heads)
    tok, qh = tok.numpy(), qh.numpy()
    kh = np.asarray(kv_heads)
    o, lse, dq, dk, dv = gpu
    cut = (o[tok][:, qh], lse[qh][:, tok], dq[tok][:, qh], dk[tok][:, kh], dv[tok][:, kh])
    check_against_oracle(sub, stens, cut)


def _group_parity(w, groups, kv_heads, deterministic=False):
    """Run the GPU on the whole workload at full size (the launch configuration the benchmark
    times), then check whole groups x KV-head groups -- independent units -- element by
    element against the oracle."""
    from paper_2602_24082_b200 import binding as B
    tens = w.tensors()
    q, k, v, do = (x.cuda() for x in tens)
    plan = B.plan_for(w, desc_on_device=True)
    plan.bwd_scratch().fill_(0xFF)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, for_backward=True)
    dq, dk, dv = B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale,
                               deterministic=deterministic)
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    sub, stens, tok, qh = W.slice_groups(w, tens, groups, kv_heads)
    tok, qh, kh = tok.cuda(), qh.cuda(), torch.as_tensor(list(kv_heads)).cuda()
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    cut = (f64(o[tok][:, qh]), f64(lse[qh][:, tok]), f64(dq[tok][:, qh]), f64(dk[tok][:, kh]),
           f64(dv[tok][:, kh]))
    check_against_oracle(sub, stens, cut)
    # everything outside the checked slice must at least be finite
    for x in (o, lse, dq, dk, dv):
        assert bool(torch.isfinite(x).all())


def test_element_offsets_beyond_32_bits():
    """T * Hq * D above 2^31 elements (Q alone is 4.4 GB): every index computed in the kernels
    and the launchers must be 64-bit.  Two small groups -- one sitting where the element offset
    crosses 2^31, one at the very end -- are checked against the oracle on the highest KV head;
    everything else must be finite."""
    big = (8192, (4096, 4096))
    rows = [[big] * 32 + [(520, (300, 200))] + [big] + [(77, (130, 1, 64))]]
    w = W.Workload("beyond-32-bit", rows, 32, 8, 128, seed=91)
    assert w.total_tokens * 32 * 128 > 2 ** 31
    first_small = 32 * 16384
    assert first_small * 32 * 128 <= 2 ** 31 < (first_small + 1020) * 32 * 128
    _group_parity(w, [(0, 32), (0, 34)], [7])


def _smallest_groups(w, n):
    sizes = sorted((p + sum(rs), ri, gi) for ri, row in enumerate(w.rows) for gi, (p, rs) in enumerate(row))
    return [(ri, gi) for (_, ri, gi) in sizes[:n]]


def test_config1_full_all_rows_one_kv_group():
    w = W.config1()
    _group_parity(w, [(r, 0) for r in range(8)], [5])


def test_config2_full_size_sampled_group():
    w = W.config2()
    _group_parity(w, _smallest_groups(w, 1), [2])


def test_config3_full_size_sampled_groups():
    w = W.config3()
    small = _smallest_groups(w, 3)
    mid = sorted((p + sum(rs), ri, gi) for ri, row in enumerate(w.rows) for gi, (p, rs) in enumerate(row))
    pick = small + [(mid[len(mid) // 2][1], mid[len(mid) // 2][2])]
    _group_parity(w, pick, [6])


@pytest.mark.parametrize("point", range(len(W.CONFIG4_POINTS)),
                         ids=[f"rho{r}-n{n}" for r, n in W.CONFIG4_POINTS])
def test_config4_full_size_sampled_group(point):
    w = W.config4(point)
    _group_parity(w, _smallest_groups(w, 1), [point % 8])


def _largest_groups(w, n):
    sizes = sorted(((p + sum(rs), ri, gi) for ri, row in enumerate(w.rows) for gi, (p, rs) in enumerate(row)),
                   reverse=True)
    return [(ri, gi) for (_, ri, gi) in sizes[:n]]


# The long end of every full-size configuration: forward units of more than a hundred key
# tiles, backward units that walk every query tile of a 16K-token group for all query heads of
# the KV head.  One whole group x one KV-head group each (independent of everything else in
# the launch), element by element against the oracle.
def test_config2_full_size_largest_row():
    w = W.config2()
    _group_parity(w, _largest_groups(w, 1), [1])


def test_config3_full_size_largest_group():
    w = W.config3()
    _group_parity(w, _largest_groups(w, 1), [3])


@pytest.mark.parametrize("point,det", [(2, False), (5, False), (0, True)],
                         ids=["rho4-n2", "rho16-n4", "rho1-n2-deterministic"])
def test_config4_full_size_largest_group(point, det):
    w = W.config4(point)
    big = _largest_groups(w, 1)
    p, rs = w.rows[big[0][0]][big[0][1]]
    assert p + sum(rs) >= 12000
    _group_parity(w, big, [(point + 3) % 8], deterministic=det)


def test_many_tiny_groups_multi_kernel_plan():
    """More than 2048 tiles: the plan is built by the multi-kernel path instead of the fused
    single-block kernel; segments of 1..9 tokens, several rows."""
    rng = np.random.default_rng(5)
    rows = []
    for _ in range(3):
        rows.append([(int(rng.integers(1, 10)), tuple(int(x) for x in rng.integers(1, 10, size=int(rng.integers(1, 4)))))
                     for _ in range(420)])
    w = W.Workload("tiny-groups", rows, 2, 1, 64, seed=77)
    assert sum(len(rs) + 1 for row in rows for _, rs in row) > 2048
    tens = w.tensors()
    check_against_oracle(w, tens, _run_gpu(w, tens, desc_on_device=True))


def test_config1_subset():
    w = W.config1()
    lens = w.row_lengths()
    _subset_parity(w, [int(np.argmin(lens))], [3])


def test_config1_full_rows_two_heads():
    w = W.config1()
    _subset_parity(w, [0, 5], [0, 7])


def test_deterministic_forward_and_dkdv():
    """Forward, dK and dV have a fixed summation order: two runs agree bit for bit.  dQ is
    summed with floating-point reductions whose order may vary: compared within tolerance."""
    w = W.Workload("det", [[(300, (140, 77))], [(64, (200, 1))]], 4, 2, 128, seed=7)
    tens = w.tensors()
    a = _run_gpu(w, tens)
    b = _run_gpu(w, tens)
    for i in (0, 1, 3, 4):
        assert np.array_equal(a[i], b[i])
    assert _rel_l2(a[2], b[2]) < 1e-3


DET_CASES = [
    ("short", [[(300, (140, 77))], [(64, (200, 1))]], 4, 2, 128),
    # a long response starting inside a tile that also holds the tail of a short one, several
    # groups, tiles that straddle segments: the turn order has to follow the tile order
    ("inversions", [[(200, (150, 40, 900)), (127, (1, 128)), (513, (3, 700, 2))]], 4, 2, 64),
    ("many-heads", [[(1000, (300, 500))], [(129, (640,))]], 8, 2, 128),
    ("d96", [[(200, (150, 40, 300)), (127, (1, 128))]], 6, 2, 96),
]


@pytest.mark.parametrize("name,rows,hq,hkv,d", DET_CASES, ids=[c[0] for c in DET_CASES])
def test_deterministic_backward(name, rows, hq, hkv, d):
    """pp_attn_bwd_deterministic: dQ (and everything else) bit-identical between runs, and the
    same parity with the oracle as the default backward."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("det-" + name, rows, hq, hkv, d, seed=21)
    tens = w.tensors()
    q, k, v, do = (x.cuda() for x in tens)
    plan = B.plan_for(w)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
    runs = []
    for _ in range(3):
        plan.bwd_scratch().fill_(0xFF)
        runs.append([x.clone() for x in B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale,
                                                      deterministic=True)])
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    for r in runs[1:]:
        for a, b in zip(runs[0], r):
            assert torch.equal(a, b)
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    check_against_oracle(w, tens, (f64(o), f64(lse)) + tuple(f64(x) for x in runs[0]))


def test_deterministic_backward_full_size_config1():
    """The benchmark's configuration: bit-identical dQ over two runs at full size."""
    from paper_2602_24082_b200 import binding as B
    w = W.config1()
    q, k, v, do = (x.cuda() for x in w.tensors())
    plan = B.plan_for(w, desc_on_device=True)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
    a = [x.clone() for x in B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, deterministic=True)]
    b = B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, deterministic=True)
    c = B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    d = (a[0].float() - c[0].float()).norm() / c[0].float().norm()
    assert float(d) < 1e-3


def test_backward_clears_its_accumulator_when_the_forward_did_not():
    """One forward that cleared the accumulator, then TWO backward calls: the first skips its
    clearing pass, the second must clear for itself (the accumulator now holds the first
    call's sums); a forward without the scratch in between resets the hand-over as well."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("clear", [[(150, (70, 200))], [(40, (129,))]], 4, 2, 128, seed=11)
    q, k, v, do = (x.cuda() for x in w.tensors())
    plan = B.plan_for(w)
    plan.bwd_scratch().fill_(0xFF)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, for_backward=True)
    a = [x.clone() for x in B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)]
    b = [x.clone() for x in B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)]
    B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, for_backward=True)
    B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)          # cancels the hand-over
    c = [x.clone() for x in B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)]
    torch.cuda.synchronize()
    for x, y, z in zip(a, b, c):
        assert bool(torch.isfinite(x.float()).all())
        for other in (y, z):
            d = (x.float() - other.float()).norm() / x.float().norm()
            assert float(d) < 1e-3


def test_outputs_outside_tiles_untouched():
    """Guard bands: the kernels write only the rows they own."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("guard", [[(70, (33, 5))]], 2, 1, 64, seed=9)
    q, k, v, do = (x.cuda() for x in w.tensors())
    T, Hq, Hkv, D = w.total_tokens, 2, 1, 64
    pad = 64
    bufs = {}
    for name, shape in (("o", (T + 2 * pad, Hq, D)), ("dq", (T + 2 * pad, Hq, D)),
                        ("dk", (T + 2 * pad, Hkv, D)), ("dv", (T + 2 * pad, Hkv, D))):
        bufs[name] = torch.full(shape, 7.0, dtype=torch.bfloat16, device="cuda")
    plan = B.plan_for(w)
    o = bufs["o"][pad:pad + T]
    o2, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, o=o)
    B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, d_q=bufs["dq"][pad:pad + T],
                  d_k=bufs["dk"][pad:pad + T], d_v=bufs["dv"][pad:pad + T])
    torch.cuda.synchronize()
    for name, b in bufs.items():
        assert (b[:pad] == 7.0).all() and (b[pad + T:] == 7.0).all(), name


HOST_CASES = [
    W.Workload("host3", [[(300, (140, 77))], [(64, (200, 1))], [(129, (640,))]], 4, 2, 128, seed=31),
    W.Workload("host1", [[(200, (130, 5)), (3, (1,))]], 2, 1, 64, seed=32),
    W.Workload("host7", [[(10 + 37 * i, (3 + 50 * (i % 3), 1 + 20 * i)), (64 + i, (9, 130))]
                         for i in range(7)], 6, 2, 128, seed=33),
    W.Workload("host-lopsided", [[(1, (1,))], [(900, (300, 300))], [(2, (1, 1))], [(1, (2,))],
                                 [(5, (5,))], [(400, (1,))]], 2, 2, 128, seed=34),
]


@pytest.mark.parametrize("w", HOST_CASES, ids=lambda w: w.name)
def test_host_step_matches_the_device_path(w):
    """pp_attn_step_host (the step cut into runs of whole groups, copies overlapped on side
    streams) called twice back to back on the same arena: both results equal the
    device-resident path (forward, dK, dV bit for bit), for fewer groups than runs, more
    groups than runs (rows cut in the middle) and groups of very different sizes."""
    from paper_2602_24082_b200 import binding as B
    tens = w.tensors()
    ref = _run_gpu(w, tens)
    hs = B.HostStep(w)
    pinned = [t.contiguous().pin_memory() for t in tens]
    for _ in range(2):
        for out in (hs.o, hs.lse, hs.dq, hs.dk, hs.dv):
            out.fill_(7.0)
        hs(*pinned)
        torch.cuda.synchronize()
        got = [x.float().numpy().astype(np.float64) for x in (hs.o, hs.lse, hs.dq, hs.dk, hs.dv)]
        for i in (0, 1, 3, 4):
            assert np.array_equal(got[i], ref[i])
        assert _rel_l2(got[2], ref[2]) < 1e-3
    check_against_oracle(w, tens, tuple(got))


def test_step_can_be_captured_in_a_cuda_graph():
    """Plan building, forward and backward make no host synchronisation and no allocation, so
    the three calls can be stream-captured; replays reproduce the eager results (O, LSE, dK,
    dV bit for bit) also after the inputs have changed in place."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("graph", [[(300, (140, 77))], [(64, (200, 1))]], 4, 2, 128, seed=41)
    q, k, v, do = (x.cuda() for x in w.tensors())
    desc = w.descriptors()
    desc_dev = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in desc]
    problem, _keep = B.make_problem(desc, 4, 2, 128, w.total_tokens, desc_dev)
    ws = torch.empty(B.pp_plan_workspace_bytes(problem)[0], dtype=torch.uint8, device="cuda")
    o, lse = torch.empty_like(q), torch.empty(4, w.total_tokens, dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    hold = {}

    def step():
        plan = B.pp_build_plan(desc, 4, 2, 128, w.total_tokens, "cuda:0", device_arrays=desc_dev, workspace=ws)
        if "scratch" in hold:
            plan._bwd_scratch = hold["scratch"]
        B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, o=o, lse=lse, for_backward=True)
        B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, d_q=dq, d_k=dk, d_v=dv)
        hold["scratch"], hold["plan"] = plan.bwd_scratch(), plan

    step()                      # first calls configure the kernels: not inside a capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for scale_inputs in (1.0, 0.5):
        q.mul_(scale_inputs)
        step()
        torch.cuda.synchronize()
        want = [x.clone() for x in (o, lse, dk, dv, dq)]
        for x in (o, lse, dk, dv, dq):
            x.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert hold["plan"].status() == (0, 0)
        for got, ref in zip((o, lse, dk, dv), want):
            assert torch.equal(got, ref)
        assert _rel_l2(dq.float().cpu().numpy(), want[4].float().cpu().numpy()) < 1e-3
