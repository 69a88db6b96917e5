"""The device-built plan against a host re-derivation from the dense mask."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_24082_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    W.config0(),
    W.Workload("ragged", [[(257, (5, 128, 31))], [(1, (1, 300))]], 4, 2, 128, seed=4),
    W.Workload("groups", [[(97, (64, 200)), (128, (128, 128)), (3, (2, 1))], [(700, (1,))]], 2, 2, 64, seed=5),
    W.Workload("short-responses", [[(100, (7, 1, 30, 1, 1, 64, 2, 90, 13)), (127, (1, 128))]], 2, 1, 64, seed=6),
    W.config3(),
]


def _global_mask(w):
    T = w.total_tokens
    m = np.zeros((T, T), dtype=bool)
    offs = w.row_offsets()
    for r in range(len(w.rows)):
        m[offs[r]:offs[r + 1], offs[r]:offs[r + 1]] = oracle.dense_mask(w.descriptors(), r)
    return m


@pytest.mark.parametrize("seed", range(24))
def test_plan_matches_dense_mask_on_random_structures(seed):
    test_plan_matches_dense_mask(W.random_structure(seed), desc_on_device=bool(seed & 1))
    test_backward_units_order(W.random_structure(seed))


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("desc_on_device", [False, True], ids=["hostdesc", "devdesc"])
def test_plan_matches_dense_mask(w, desc_on_device):
    from paper_2602_24082_b200 import binding as B
    plan = B.plan_for(w, desc_on_device=desc_on_device)
    assert plan.status() == (0, 0)
    tiles, fwd_order, bwd_order, key_end = plan.read()
    mask = _global_mask(w)
    T = w.total_tokens
    # tiles partition the tokens, never straddle a segment
    segs = w.segments()
    covered = np.zeros(T, dtype=int)
    expect_tiles = sum((l + 127) // 128 for (_, l, *_rest) in segs)
    assert len(tiles) == expect_tiles
    for (start, ln, k0s, k0l, k1s, k1l, vis_end, work) in tiles.tolist():
        assert 1 <= ln <= 128
        covered[start:start + ln] += 1
        seg = [s for s in segs if s[0] <= start < s[0] + s[1]][0]
        assert start + ln <= seg[0] + seg[1] and (start - seg[0]) % 128 == 0
        # forward view: every row of the tile sees exactly kv0 U kv1 (FULL, no masked pair)
        # plus the causal part of its own tile (DIAG); nothing else (siblings are skipped)
        rows = mask[start:start + ln]
        want = np.zeros((ln, T), dtype=bool)
        want[:, k0s:k0s + k0l] = True
        want[:, k1s:k1s + k1l] = True
        want[:, start:start + ln] = np.tril(np.ones((ln, ln), dtype=bool))
        assert np.array_equal(rows, want)
        assert work == (k0l + 127) // 128 + (k1l + 127) // 128 + 1
        # column view: the queries that see these keys are exactly [start, vis_end),
        # fully below the tile, causally inside it
        cols = mask[:, start:start + ln]
        wantc = np.zeros((T, ln), dtype=bool)
        wantc[start:start + ln] = np.tril(np.ones((ln, ln), dtype=bool))
        wantc[start + ln:vis_end] = True
        assert np.array_equal(cols, wantc)
    assert (covered == 1).all()
    # backward key tiles: every group cut into 128-token tiles from its start
    btiles = plan.read_bwd_tiles()
    groups = {}
    for (s0, l0, _r, g, _k) in segs:
        lo, hi = groups.get(g, (s0, s0 + l0))
        groups[g] = (min(lo, s0), max(hi, s0 + l0))
    assert len(btiles) == sum((hi - lo + 127) // 128 for lo, hi in groups.values())
    bcov = np.zeros(T, dtype=int)
    prompt_len = {s0: l0 for (s0, l0, _r, _g, k) in segs if k == 0}   # by group start
    bt_start = {int(b[0]): i for i, b in enumerate(btiles.tolist())}
    for (start, ln, vis_end, dep_lo, gstart, gend, work, npc) in btiles.tolist():
        assert npc == (prompt_len[gstart] + 127) // 128
        assert 1 <= ln <= 128 and (start - gstart) % 128 == 0 and start + ln <= gend
        assert ln == 128 or start + ln == gend
        assert (gstart, gend) in groups.values()
        bcov[start:start + ln] += 1
        cols = mask[:, start:start + ln]
        seen = np.nonzero(cols.any(axis=1))[0]
        assert seen[0] == start and seen[-1] + 1 == vis_end
        # per-key bounds: key j is seen by exactly [j, key_end[j])
        for c in range(ln):
            q = np.nonzero(cols[:, c])[0]
            assert q[0] == start + c and q[-1] + 1 == key_end[start + c] and len(q) == key_end[start + c] - start - c
        assert vis_end == key_end[start:start + ln].max()
        # read as a query tile: the key tiles of the group whose keys some row of this tile sees
        # are the prompt tiles [0, npc) (up to the tile itself) and the tiles [dep_lo, own index]
        k_rel = (start - gstart) // 128
        seen_tiles = {kk for kk in range(k_rel + 1)
                      if mask[start:start + ln, gstart + 128 * kk:min(gstart + 128 * kk + 128, gend)].any()}
        assert seen_tiles == set(range(min(npc, k_rel + 1))) | set(range(dep_lo, k_rel + 1))
        assert work == 1 + (vis_end - start - ln + 127) // 128
    assert (bcov == 1).all()
    # column form of the mask: key j is visible to queries [j, key_end[j])
    for j in range(0, T, max(1, T // 997)):
        seen = np.nonzero(mask[:, j])[0]
        assert seen[0] == j and seen[-1] + 1 == key_end[j] and len(seen) == key_end[j] - j
    # orders are permutations, longest work first
    n, nb = len(tiles), len(btiles)
    bwd_order = bwd_order[:nb]
    assert sorted(fwd_order.tolist()) == list(range(n)) and sorted(bwd_order.tolist()) == list(range(nb))
    fw = tiles[fwd_order, 7]
    assert (np.diff(fw) <= 0).all()
    assert (np.diff(btiles[bwd_order, 6]) <= 0).all()


@pytest.mark.parametrize("w", CASES + [W.config4(3)], ids=lambda w: w.name)
def test_backward_units_order(w):
    """Every (backward tile, KV head) appears exactly once; groups are taken in order of decreasing
    backward work and merged into super-groups of about 600 units; inside a super-group units
    come longest first with all KV heads of a tile adjacent."""
    from paper_2602_24082_b200 import binding as B
    plan = B.plan_for(w, desc_on_device=True)
    btiles = plan.read_bwd_tiles()
    n, hkv = len(btiles), w.num_kv_heads
    units = plan.read_bwd_units(n)
    assert units.shape == (n * hkv, 2)
    assert sorted(map(tuple, units.tolist())) == [(h, t) for h in range(hkv) for t in range(n)]
    work = btiles[:, 6]
    grp = btiles[:, 4]                     # first token of the group = group identity
    gwork = {int(g): int(work[grp == g].sum()) for g in np.unique(grp)}
    ranked = sorted(gwork, key=lambda g: (-gwork[g], g))
    sgroup, rest = {}, n
    for g in ranked:
        sgroup[g] = (hkv * rest - 1) // 600     # blocks are cut from the end of the list
        rest -= int((grp == g).sum())
    expect = sorted(range(n), key=lambda t: (-sgroup[int(grp[t])], -int(work[t]), t))
    assert units[:, 1].reshape(n, hkv)[:, 0].tolist() == expect
    assert (units[:, 0].reshape(n, hkv) == np.arange(hkv)).all()
    assert (units[:, 1].reshape(n, hkv) == units[:, 1].reshape(n, hkv)[:, :1]).all()


def test_multi_kernel_plan_path_matches_fused_semantics():
    """> 2048 tiles forces the multi-kernel plan path; its tiles / orders obey the same
    rules (checked through the same dense-mask comparison on a prefix of the tokens)."""
    from paper_2602_24082_b200 import binding as B
    rows = [[(3 + (i % 5), (1 + (i % 3), 2)) for i in range(1100)]]
    w = W.Workload("many", rows, 2, 2, 64, seed=1)
    plan = B.plan_for(w, desc_on_device=True)
    assert plan.status() == (0, 0)
    tiles, fwd_order, bwd_order, key_end = plan.read()
    btiles = plan.read_bwd_tiles()
    n, nb = len(tiles), len(btiles)
    assert n == 3 * 1100 and n > 2048 and nb == 1100     # every group is shorter than a tile
    assert sorted(fwd_order.tolist()) == list(range(n)) and sorted(bwd_order[:nb].tolist()) == list(range(nb))
    segs = w.segments()
    assert [int(t[0]) for t in tiles] == [s[0] for s in segs] and [int(t[1]) for t in tiles] == [s[1] for s in segs]
    for (start, ln, k0s, k0l, k1s, k1l, vis_end, work), (s0, l0, _, g, seg) in zip(tiles.tolist(), segs):
        gs = [x for x in segs if x[3] == g and x[4] == 0][0]
        gend = max(x[0] + x[1] for x in segs if x[3] == g)
        if seg == 0:
            assert (k0s, k0l, k1l, vis_end) == (gs[0], 0, 0, gend)
        else:
            assert (k0s, k0l, k1s, k1l, vis_end) == (gs[0], gs[1], s0, 0, s0 + l0)
    units = plan.read_bwd_units(nb)
    assert sorted(map(tuple, units.tolist())) == [(h, t) for h in range(2) for t in range(nb)]
    gl = [sum(x[1] for x in segs if x[3] == g) for g in range(1100)]
    assert btiles[:, 1].tolist() == gl and (btiles[:, 6] == 1).all()
    assert (btiles[:, 2] == btiles[:, 5]).all()          # prompt keys reach the group's end
    for j in range(0, w.total_tokens, 97):
        seg = [x for x in segs if x[0] <= j < x[0] + x[1]][0]
        gend = max(x[0] + x[1] for x in segs if x[3] == seg[3])
        assert key_end[j] == (gend if seg[4] == 0 else seg[0] + seg[1])


def test_device_side_validation_reports_status():
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("bad", [[(5, (2, 4))], [(3, (1, 2))]], 2, 1, 64, seed=0)
    rgo, gpl, gro, rl = w.descriptors()
    bad_rl = rl.copy(); bad_rl[2] = 0
    plan = B.pp_build_plan((rgo, gpl, gro, bad_rl), 2, 1, 64, w.total_tokens, desc_on_device=True)
    st, det = plan.status()
    assert st == 1 and det == len(gpl) + 2
    bad_rl = rl.copy(); bad_rl[0] += 3
    plan = B.pp_build_plan((rgo, gpl, gro, bad_rl), 2, 1, 64, w.total_tokens, desc_on_device=True)
    assert plan.status() == (2, w.total_tokens + 3)
    # kernels given a failed plan do nothing and report nothing new
    import torch
    q, k, v, do = (x.cuda() for x in w.tensors())
    o = torch.full_like(q, 3.0)
    B.pp_attn_fwd(plan, q, k, v, 0.125, o=o)
    torch.cuda.synchronize()
    assert (o == 3.0).all()


@pytest.mark.parametrize("groups", [40, 1100, 2500], ids=["small-block", "large-block", "copied"])
def test_host_descriptors_reach_the_device_unchanged(groups):
    """Host descriptors travel as a kernel argument (two block sizes) or, beyond that, by
    copies: each route gives the plan that device-resident descriptors give."""
    from paper_2602_24082_b200 import binding as B
    rows = [[(1 + (i % 7), (1 + (i % 2),)) for i in range(groups)]]
    w = W.Workload("desc", rows, 2, 1, 64, seed=2)
    got = B.plan_for(w, desc_on_device=False)
    want = B.plan_for(w, desc_on_device=True)
    assert got.status() == (0, 0) and want.status() == (0, 0)
    nb = len(want.read_bwd_tiles())
    assert np.array_equal(got.read_bwd_tiles(), want.read_bwd_tiles())
    for a, b in zip(got.read(), want.read()):   # (tiles, fwd_order, bwd_order, key_end)
        assert a.shape == b.shape
    (t0, f0, b0, k0), (t1, f1, b1, k1) = got.read(), want.read()
    assert np.array_equal(t0, t1) and np.array_equal(f0, f1) and np.array_equal(k0, k1)
    assert np.array_equal(b0[:nb], b1[:nb])      # entries past the backward tiles are unused
    assert np.array_equal(got.read_bwd_units(nb), want.read_bwd_units(nb))


def test_bounded_wait_gives_up_and_later_kernels_do_nothing():
    """A wait that runs out (one thread, no copy or MMA in flight, 4096 polls on a barrier that
    nobody arrives at) records status 3 with its site id and returns; the kernels of later
    calls on that plan then return at once and leave the outputs untouched."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("expire", [[(150, (70, 33))]], 2, 1, 64, seed=3)
    q, k, v, do = (x.cuda() for x in w.tensors())
    plan = B.plan_for(w)
    o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
    torch.cuda.synchronize()
    assert plan.status() == (0, 0)
    B.pp_debug_expire_wait(plan, 57)
    torch.cuda.synchronize()
    assert plan.status() == (3, 57)
    o2 = torch.full_like(q, 7.0)
    dq, dk, dv = torch.full_like(q, 7.0), torch.full_like(k, 7.0), torch.full_like(v, 7.0)
    B.pp_attn_fwd(plan, q, k, v, w.softmax_scale, o=o2)
    B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale, d_q=dq, d_k=dk, d_v=dv)
    torch.cuda.synchronize()
    assert plan.status() == (3, 57)
    assert (o2 == 7.0).all() and (dk == 7.0).all() and (dv == 7.0).all()
    # a fresh plan in the same workspace works again
    plan2 = B.pp_build_plan(w.descriptors(), 2, 1, 64, w.total_tokens, workspace=plan.workspace)
    o3, _ = B.pp_attn_fwd(plan2, q, k, v, w.softmax_scale)
    torch.cuda.synchronize()
    assert plan2.status() == (0, 0) and torch.equal(o3, o)


def test_device_descriptors_are_copied_by_the_plan():
    """Descriptors given on the device are only read by the first plan kernel: overwriting the
    caller's arrays afterwards changes nothing for the plan's later users (position ids,
    rotary embedding, loss)."""
    from oracle import loss as OL
    from oracle import rope as OR
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("desc-copy", [[(97, (64, 200)), (128, (128, 31))], [(5, (3, 1, 9))]], 2, 1, 64, seed=8)
    desc = w.descriptors()
    desc_dev = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in desc]
    plan = B.pp_build_plan(desc, 2, 1, 64, w.total_tokens, device_arrays=desc_dev)
    torch.cuda.synchronize()
    for t in desc_dev:
        t.fill_(-12345)
    torch.cuda.synchronize()
    pos = B.pp_position_ids(plan).cpu().numpy()
    assert np.array_equal(pos.astype(np.int64), OR.position_ids(w.rows))
    rng = np.random.default_rng(2)
    lp = (-rng.gamma(2.0, 1.0, w.total_tokens)).astype(np.float32)
    s, r, loss, grad = B.pp_preference_loss(plan, torch.from_numpy(lp).cuda(), None, 0.05)
    S, Rw, Ls, G = OL.preference_loss(w.rows, lp, None, 0.05)
    assert np.abs(s.cpu().numpy() - S).max() <= 1e-4 * max(1.0, np.abs(S).max())
    assert np.abs(loss.cpu().numpy() - Ls).max() <= 1e-4 * max(1.0, np.abs(Ls).max())
    q, k, _, _ = w.tensors()
    qd, kd = q.cuda().clone(), k.cuda().clone()
    B.pp_rope_qk(plan, qd, kd, 10000.0)
    ref = OR.rope(q.double().numpy(), OR.position_ids(w.rows), 10000.0)
    assert np.abs(qd.float().cpu().numpy() - ref).max() <= 2e-2
    assert plan.status() == (0, 0)


def test_this_device_passes_the_compute_capability_check():
    """pp_build_plan refuses devices that are not compute capability 10.x with
    PP_ERR_UNSUPPORTED; the B200 the suite runs on must pass."""
    from paper_2602_24082_b200 import binding as B
    assert torch.cuda.get_device_capability(0)[0] == 10
    plan = B.plan_for(W.config0())
    assert plan.status() == (0, 0)


@pytest.mark.gpu
def test_profile_event_ring():
    """Kernel event timing over several calls without a synchronisation in between: the ring
    returns one duration per call, oldest first, and restarts when profiling is re-enabled."""
    from paper_2602_24082_b200 import binding as B
    w = W.Workload("ring", [[(300, (140, 77))], [(64, (200, 1))]], 4, 2, 128, seed=3)
    q, k, v, do = (x.cuda() for x in w.tensors())
    plan = B.plan_for(w)
    B.pp_profile_enable(True)
    try:
        for _ in range(5):
            o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
            B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)
        torch.cuda.synchronize()
        f, b = B.pp_profile_read_all(64)
        assert len(f) == 5 and len(b) == 5 and all(x > 0 for x in f + b)
        last_f, last_b = B.pp_profile_read()
        assert last_f == f[-1] and last_b == b[-1]
        f2, b2 = B.pp_profile_read_all(3)
        assert f2 == f[-3:] and b2 == b[-3:]
        B.pp_profile_enable(True, backward_only=True)
        o, lse = B.pp_attn_fwd(plan, q, k, v, w.softmax_scale)
        B.pp_attn_bwd(plan, q, k, v, o, lse, do, w.softmax_scale)
        torch.cuda.synchronize()
        f3, b3 = B.pp_profile_read_all(64)
        assert f3 == [] and len(b3) == 1
    finally:
        B.pp_profile_enable(False)
    assert plan.status() == (0, 0)
