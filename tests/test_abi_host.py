"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2602_24082_b200 import binding as B
from paper_2602_24082_b200 import build as build_mod
from paper_2602_24082_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "pp_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pp_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_error_strings(lib):
    assert lib.pp_error_string(0) == b"ok"
    seen = {lib.pp_error_string(c) for c in range(-6, 1)}
    assert len(seen) == 7
    assert lib.pp_error_string(-99) == b"unknown error"


def _problem(w, **over):
    p, keep = B.make_problem(w.descriptors(), w.num_q_heads, w.num_kv_heads, w.head_dim,
                             w.total_tokens)
    for k, v in over.items():
        setattr(p, k, v)
    return p, keep


def test_workspace_query_and_shape_errors(lib):
    w = W.config1()
    p, keep = _problem(w)
    plan_b, fwd_b, bwd_b = B.pp_plan_workspace_bytes(p)
    assert plan_b > 4 * w.total_tokens and fwd_b == 0
    assert bwd_b >= 4 * w.total_tokens * w.num_q_heads * (w.head_dim + 2)
    for over, code in ((dict(head_dim=80), -2), (dict(head_dim=256), -2), (dict(num_kv_heads=5), -1), (dict(num_rows=0), -1),
                       (dict(total_tokens=0), -1), (dict(num_q_heads=0), -1)):
        bad, keep2 = _problem(w, **over)
        with pytest.raises(B.PPError) as e:
            B.pp_plan_workspace_bytes(bad)
        assert e.value.code == code


def _build(lib, p, ws_ptr, ws_bytes):
    h = ctypes.c_void_p(0)
    rc = lib.pp_build_plan(ctypes.byref(p), ws_ptr, ws_bytes, None, ctypes.byref(h))
    assert h.value is None or rc == 0
    return rc


def test_build_plan_rejects_bad_descriptors_before_any_device_work(lib):
    """All of these must fail on the host: the pointer handed in as workspace is not even
    device memory."""
    w = W.Workload("e", [[(5, (2, 4))], [(3, (1, 2))]], 2, 1, 64, seed=0)
    fake_ws = 256 * 4096          # 256-byte aligned, never dereferenced
    p, keep = _problem(w)
    need = B.pp_plan_workspace_bytes(p)[0]
    assert _build(lib, p, None, need) == -1
    assert _build(lib, p, fake_ws + 8, need) == -4
    assert _build(lib, p, fake_ws, need - 1) == -3
    rgo, gpl, gro, rl = w.descriptors()
    cases = []
    a = gpl.copy(); a[0] = 0; cases.append((rgo, a, gro, rl))                 # empty prompt
    a = rl.copy(); a[1] = 0; cases.append((rgo, gpl, gro, a))                 # empty response
    a = rl.copy(); a[1] += 1; cases.append((rgo, gpl, gro, a))                # total mismatch
    a = gro.copy(); a[1] = 5; cases.append((rgo, gpl, a, rl))                 # offsets not monotone
    a = gro.copy(); a[1] = 0; cases.append((rgo, gpl, a, rl))                 # group with n = 0
    a = rgo.copy(); a[1] = 2; cases.append((a, gpl, gro, rl))                 # empty row
    for desc in cases:
        bad, keep2 = B.make_problem(desc, 2, 1, 64, w.total_tokens)
        assert _build(lib, bad, fake_ws, need) == -1
    nullp, keep3 = _problem(w)
    nullp.resp_len = None
    assert _build(lib, nullp, fake_ws, need) == -1


def test_attn_calls_reject_null_and_misaligned(lib):
    assert lib.pp_attn_fwd(None, 16, 16, 16, 1.0, 16, 16, None, 0, None) == -1
    assert lib.pp_attn_bwd(None, 16, 16, 16, 16, 16, 16, 1.0, 16, 16, 16, 16, 0, None) == -1
    assert lib.pp_plan_status(None, None, None, None) == -1
    assert lib.pp_plan_max_tiles(None) == -1
    assert lib.pp_destroy_plan(None) == 0


def test_binding_fails_loudly_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        B.plan_for(W.config0())


def _runs(w):
    problem, _keep = B.make_problem(w.descriptors(), w.num_q_heads, w.num_kv_heads, w.head_dim,
                                    w.total_tokens)
    return B.pp_step_host_runs(problem)


def test_host_step_runs_partition_the_groups(lib):
    """The host step is cut at group boundaries into at most eight runs of about equal token
    counts; runs are non-empty, contiguous and cover everything; tiny problems stay whole."""
    rows = [[(50 + 13 * i, (20 + i, 7 * (i % 4) + 1)), (9 + i, (30,))] for i in range(11)]
    w = W.Workload("runs", rows, 8, 2, 128, seed=1)
    gb, tb = _runs(w)
    rgo, gpl, gro, rl = w.descriptors()
    glen = np.array([gpl[g] + rl[gro[g]:gro[g + 1]].sum() for g in range(len(gpl))])
    gstart = np.concatenate([[0], np.cumsum(glen)])
    assert len(gb) - 1 == 8 and gb[0] == 0 and gb[-1] == len(gpl) and (np.diff(gb) >= 1).all()
    assert tb.tolist() == gstart[gb].tolist() and tb[-1] == w.total_tokens
    # balance: no run exceeds the ideal share by more than the longest group
    assert np.diff(tb).max() <= w.total_tokens / 8 + glen.max()
    # fewer groups than runs: one group per run
    w3 = W.Workload("runs3", [[(300, (140, 77))], [(64, (200, 1))], [(129, (640,))]], 4, 2, 128, seed=2)
    gb, tb = _runs(w3)
    assert gb.tolist() == [0, 1, 2, 3]
    # under a quarter MiB of input per run: fewer runs (here: one)
    tiny = W.Workload("tiny", [[(5, (2, 4)), (3, (1,))], [(3, (1, 2))]], 2, 1, 64, seed=3)
    gb, tb = _runs(tiny)
    assert gb.tolist() == [0, 3] and tb.tolist() == [0, tiny.total_tokens]
    # one very long group among short ones keeps every later run non-empty
    lop = W.Workload("lop", [[(1, (1,))], [(900, (300, 300))], [(2, (1, 1))], [(1, (2,))],
                             [(5, (5,))], [(400, (1,))]], 16, 2, 128, seed=4)
    gb, tb = _runs(lop)
    assert gb[0] == 0 and gb[-1] == 6 and (np.diff(gb) >= 1).all() and (np.diff(tb) >= 1).all()
