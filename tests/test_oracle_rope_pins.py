"""Pins for the position-id / rotary oracle (oracle/rope.py)."""
import numpy as np

from oracle import rope as R
from paper_2602_24082_b200 import workloads as W


def test_positions_equal_unpacked_positions():
    """Sec. 3.2: each response keeps the positions of its own sequence (x, y_k): gathering the
    packed ids of x and y_k gives 0 .. P + R_k - 1."""
    w = W.Workload("p", [[(5, (2, 4)), (3, (1,))], [(7, (3, 3, 2))]], 1, 1, 8, seed=0)
    pos = R.position_ids(w.rows)
    assert len(pos) == w.total_tokens
    t = 0
    for row in w.rows:
        for (p, rs) in row:
            off = t + p
            for r in rs:
                idx = list(range(t, t + p)) + list(range(off, off + r))
                assert pos[idx].tolist() == list(range(p + r))
                off += r
            t = off


def test_rope_matches_complex_multiplication():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, 2, 16))
    pos = np.array([0, 1, 5, 17, 100, 4097])
    base = 10000.0
    got = R.rope(x, pos, base)
    half = 8
    z = x[..., :half] + 1j * x[..., half:]
    ang = pos[:, None] * base ** (-2.0 * np.arange(half) / 16)
    zr = z * np.exp(1j * ang)[:, None, :]
    assert np.abs(got[..., :half] - zr.real).max() < 1e-12
    assert np.abs(got[..., half:] - zr.imag).max() < 1e-12


def test_rope_relative_position_invariance_identity_and_norm():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((1, 1, 32))
    k = rng.standard_normal((1, 1, 32))
    base = 500000.0
    dots = []
    for shift in (0, 3, 1000):
        qr = R.rope(q, np.array([7 + shift]), base)
        kr = R.rope(k, np.array([2 + shift]), base)
        dots.append(float((qr * kr).sum()))
    assert abs(dots[0] - dots[1]) < 1e-9 and abs(dots[0] - dots[2]) < 1e-9
    assert np.array_equal(R.rope(q, np.array([0]), base), q)
    assert abs(np.linalg.norm(R.rope(q, np.array([12345]), base)) - np.linalg.norm(q)) < 1e-12
