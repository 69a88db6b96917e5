"""The paper's closed-form cost model (Sec. 3.2.1), for reports only.

``l_in`` is the prompt length, ``l_resp`` the K response lengths.  The formulas charge a
dense mask (sibling blocks included); the kernels here skip sibling tiles, so the
measured saving is at least the one predicted.
"""
from __future__ import annotations

import math
from typing import Sequence


def attention_cost_ratio(l_in: float, l_resp: Sequence[float]) -> float:
    """C_pp / C_original = (l_in + sum l_resp)^2 / (K (l_in + max l_resp)^2)."""
    k = len(l_resp)
    return (l_in + sum(l_resp)) ** 2 / (k * (l_in + max(l_resp)) ** 2)


def memory_ratio(l_in: float, l_resp: Sequence[float]) -> float:
    """Linear-memory (flash-attention) ratio (l_in + sum l_resp) / (K (l_in + max l_resp))."""
    k = len(l_resp)
    return (l_in + sum(l_resp)) / (k * (l_in + max(l_resp)))


def packing_wins(l_in: float, l_resp: Sequence[float]) -> bool:
    """Eq. (1): l_in + sum l_resp < sqrt(K) (l_in + max l_resp)."""
    return l_in + sum(l_resp) < math.sqrt(len(l_resp)) * (l_in + max(l_resp))
