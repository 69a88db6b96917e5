"""TEST INFRASTRUCTURE: plain numpy fp64 oracle for the packed position ids and the rotary
embedding applied with them (the step right before attention in the paper's Sec. 3.2).

Position ids follow the paper's statement that every response keeps the positions it would
have in its own sequence (x, y^k): a prompt token's position is its index inside the prompt,
a response token's position is P plus its index inside the response.  The rotary embedding
is the textbook rotate-half form, angle = position * base^(-2 i / D).

Pinned by tests/test_oracle_rope_pins.py (unpacked positions are arange; relative-position
invariance; complex-multiplication form through numpy's own complex arithmetic; position 0 is
the identity; norms are preserved).  Shares no code with the CUDA library.
"""
from __future__ import annotations

import numpy as np


def position_ids(rows) -> np.ndarray:
    """rows: list of rows, each a list of (P, (R_1, .., R_n)).  Returns int64 [T]."""
    out = []
    for row in rows:
        for (p, rs) in row:
            out.extend(range(p))
            for r in rs:
                out.extend(range(p, p + r))
    return np.asarray(out, dtype=np.int64)


def rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """x: [T, H, D] float64; returns the rotated copy."""
    T, H, D = x.shape
    half = D // 2
    out = np.empty_like(x)
    for t in range(T):
        for i in range(half):
            ang = float(positions[t]) * base ** (-2.0 * i / D)
            c, s = np.cos(ang), np.sin(ang)
            a, b = x[t, :, i], x[t, :, i + half]
            out[t, :, i] = a * c - b * s
            out[t, :, i + half] = b * c + a * s
    return out
