"""Seeded synthetic inputs for preference-packed attention.

This module only *describes* inputs: segment lengths, descriptor arrays, random
Q/K/V/dO tensors and bookkeeping counts.  It contains none of the attention
arithmetic, so both the CUDA path's tests and the CPU oracle's tests can draw
their inputs from it without sharing any of the method's code.

Vocabulary (paper Sec. 3.1-3.2): a *group* is one preference sample
``(x, y^1 .. y^K)`` laid out as ``[prompt | response 1 | ... | response K]``;
a *row* is one sequence holding one group (plain preference packing) or several
groups end to end (preference packing combined with batch packing, Sec. 2.2).

The five workload recipes mirror the length statistics of the paper's
experiments (Table 1 means; "< 16K tokens" in Sec. 5.2) -- no dataset item is
reproduced, only lengths drawn from simple distributions.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import numpy as np
import torch

Group = Tuple[int, Tuple[int, ...]]          # (prompt_len, (resp_len, ...))


@dataclasses.dataclass
class Workload:
    name: str
    rows: List[List[Group]]
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    seed: int
    # token ranges [lo, hi) (absolute) whose Q/K/V rows are scaled by low_std
    low_var_ranges: List[Tuple[int, int]] = dataclasses.field(default_factory=list)
    low_std: float = 1.0

    # ---- descriptor arrays in the C-ABI's format -------------------------------
    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    def descriptors(self):
        """(row_group_off, grp_prompt_len, grp_resp_off, resp_len) int32 arrays."""
        row_group_off = [0]
        grp_prompt_len: List[int] = []
        grp_resp_off = [0]
        resp_len: List[int] = []
        for row in self.rows:
            for (p, rs) in row:
                grp_prompt_len.append(int(p))
                resp_len.extend(int(r) for r in rs)
                grp_resp_off.append(len(resp_len))
            row_group_off.append(len(grp_prompt_len))
        a = lambda x: np.asarray(x, dtype=np.int32)
        return a(row_group_off), a(grp_prompt_len), a(grp_resp_off), a(resp_len)

    @property
    def total_tokens(self) -> int:
        return sum(p + sum(rs) for row in self.rows for (p, rs) in row)

    def row_lengths(self) -> List[int]:
        return [sum(p + sum(rs) for (p, rs) in row) for row in self.rows]

    def row_offsets(self) -> List[int]:
        off = [0]
        for l in self.row_lengths():
            off.append(off[-1] + l)
        return off

    def segments(self):
        """List of (start, length, row, group_index, seg) with seg=0 for the prompt."""
        out = []
        t = 0
        g = 0
        for r, row in enumerate(self.rows):
            for (p, rs) in row:
                out.append((t, p, r, g, 0))
                t += p
                for k, rl in enumerate(rs):
                    out.append((t, rl, r, g, k + 1))
                    t += rl
                g += 1
        return out

    # ---- bookkeeping (counts only; used for FLOP accounting) ------------------
    def useful_pairs(self) -> int:
        """Number of (query, key) pairs that the packing mask leaves visible."""
        u = 0
        for row in self.rows:
            for (p, rs) in row:
                u += p * (p + 1) // 2
                for r in rs:
                    u += r * p + r * (r + 1) // 2
        return u

    def useful_flops(self) -> Tuple[int, int]:
        """(forward, backward) useful FLOPs: 2 GEMMs fwd, 5 GEMMs bwd, 2*D per pair each."""
        u = self.useful_pairs()
        per = 2 * self.head_dim * self.num_q_heads * u
        return 2 * per, 5 * per

    # ---- tensors ---------------------------------------------------------------
    def tensors(self, device: str = "cpu"):
        """bf16 Q [T,Hq,D], K, V [T,Hkv,D], dO [T,Hq,D]; N(0,1), drawn in this order."""
        g = torch.Generator(device="cpu").manual_seed(self.seed)
        T, Hq, Hkv, D = self.total_tokens, self.num_q_heads, self.num_kv_heads, self.head_dim
        q = torch.randn(T, Hq, D, generator=g, dtype=torch.float32)
        k = torch.randn(T, Hkv, D, generator=g, dtype=torch.float32)
        v = torch.randn(T, Hkv, D, generator=g, dtype=torch.float32)
        do = torch.randn(T, Hq, D, generator=g, dtype=torch.float32)
        for (lo, hi) in self.low_var_ranges:
            q[lo:hi] *= self.low_std
            k[lo:hi] *= self.low_std
            v[lo:hi] *= self.low_std
        out = tuple(x.to(torch.bfloat16) for x in (q, k, v, do))
        if device != "cpu":
            out = tuple(x.to(device) for x in out)
        return out

    # ---- sub-problems (rows / KV-head groups are independent units) -----------
    def select_rows(self, row_ids: Sequence[int]) -> "Workload":
        offs = self.row_offsets()
        lv = []
        new_off = 0
        for r in row_ids:
            for (lo, hi) in self.low_var_ranges:
                a, b = max(lo, offs[r]), min(hi, offs[r + 1])
                if a < b:
                    lv.append((a - offs[r] + new_off, b - offs[r] + new_off))
            new_off += offs[r + 1] - offs[r]
        return dataclasses.replace(self, name=self.name + f"/rows{list(row_ids)}",
                                   rows=[self.rows[r] for r in row_ids], low_var_ranges=lv)

    def token_index_of_rows(self, row_ids: Sequence[int]) -> torch.Tensor:
        offs = self.row_offsets()
        return torch.cat([torch.arange(offs[r], offs[r + 1]) for r in row_ids])


def slice_heads(w: Workload, tens, row_ids: Sequence[int], kv_heads: Sequence[int]):
    """Cut an independent sub-problem: the given rows and KV heads with all their query heads.

    Returns (sub_workload, (q, k, v, do), token_index, q_head_index)."""
    r = w.num_q_heads // w.num_kv_heads
    tok = w.token_index_of_rows(row_ids)
    qh = torch.tensor([c * r + i for c in kv_heads for i in range(r)], dtype=torch.long)
    kh = torch.tensor(list(kv_heads), dtype=torch.long)
    q, k, v, do = tens
    dev = q.device
    tok_d, qh_d, kh_d = tok.to(dev), qh.to(dev), kh.to(dev)
    sub = w.select_rows(row_ids)
    sub = dataclasses.replace(sub, num_q_heads=len(qh), num_kv_heads=len(kh))
    sq = q.index_select(0, tok_d).index_select(1, qh_d).contiguous()
    sk = k.index_select(0, tok_d).index_select(1, kh_d).contiguous()
    sv = v.index_select(0, tok_d).index_select(1, kh_d).contiguous()
    sdo = do.index_select(0, tok_d).index_select(1, qh_d).contiguous()
    return sub, (sq, sk, sv, sdo), tok, qh


def slice_groups(w: Workload, tens, groups: Sequence[Tuple[int, int]], kv_heads: Sequence[int]):
    """Independent sub-problem made of whole groups (row, index-in-row) and KV heads with all
    their query heads; each selected group becomes a row of its own.  Attention never crosses
    a group, so the sub-problem's results equal the corresponding slice of the full results.

    Returns (sub_workload, (q, k, v, do), token_index, q_head_index)."""
    r = w.num_q_heads // w.num_kv_heads
    offs = w.row_offsets()
    rows, tok, lv, new_off = [], [], [], 0
    for (ri, gi) in groups:
        t0 = offs[ri] + sum(p + sum(rs) for (p, rs) in w.rows[ri][:gi])
        p, rs = w.rows[ri][gi]
        L = p + sum(rs)
        rows.append([(p, tuple(rs))])
        tok.append(torch.arange(t0, t0 + L))
        for (lo, hi) in w.low_var_ranges:
            a, b = max(lo, t0), min(hi, t0 + L)
            if a < b:
                lv.append((a - t0 + new_off, b - t0 + new_off))
        new_off += L
    tok = torch.cat(tok)
    qh = torch.tensor([c * r + i for c in kv_heads for i in range(r)], dtype=torch.long)
    kh = torch.tensor(list(kv_heads), dtype=torch.long)
    q, k, v, do = tens
    dev = q.device
    tok_d, qh_d, kh_d = tok.to(dev), qh.to(dev), kh.to(dev)
    sub = dataclasses.replace(w, name=w.name + f"/groups{list(groups)}", rows=rows,
                              num_q_heads=len(qh), num_kv_heads=len(kh), low_var_ranges=lv)
    sq = q.index_select(0, tok_d).index_select(1, qh_d).contiguous()
    sk = k.index_select(0, tok_d).index_select(1, kh_d).contiguous()
    sv = v.index_select(0, tok_d).index_select(1, kh_d).contiguous()
    sdo = do.index_select(0, tok_d).index_select(1, qh_d).contiguous()
    return sub, (sq, sk, sv, sdo), tok, qh


# ------------------------------------------------------------------------------
# The five workload recipes
# ------------------------------------------------------------------------------

def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _lognormal_int(rng, median, sigma, lo, hi) -> int:
    return int(np.clip(round(median * math.exp(sigma * rng.standard_normal())), lo, hi))


def config0() -> Workload:
    """One row, one head, D=64, P=64, responses (32, 48); the tiny full-oracle case."""
    return Workload("config0", [[(64, (32, 48))]], 1, 1, 64, seed=0)


def config1(seed: int = 1) -> Workload:
    """Llama-3-8B attention shape, 8 rows, pairwise responses (Table 1-like lengths)."""
    rng = _rng(seed)
    rows = []
    for _ in range(8):
        p = _lognormal_int(rng, 512, 0.5, 64, 2048)
        rs = tuple(int(rng.integers(64, 513)) for _ in range(2))
        rows.append([(p, rs)])
    return Workload("config1", rows, 32, 8, 128, seed=seed)


def config2(seed: int = 2, low_std: float = math.sqrt(0.5)) -> Workload:
    """Multi-response ranking with a long image-like prompt prefix of lower variance."""
    rng = _rng(seed)
    rows, lv, t = [], [], 0
    for _ in range(4):
        p = int(rng.integers(1024, 4097))
        img = int(rng.integers(1024, min(2048, p) + 1))
        rs = tuple(int(rng.integers(128, 1025)) for _ in range(4))
        rows.append([(p, rs)])
        lv.append((t, t + img))
        t += p + sum(rs)
    return Workload("config2", rows, 28, 4, 128, seed=seed, low_var_ranges=lv, low_std=low_std)


def _fill_row(rng, row_len: int, draw_group) -> List[Group]:
    """Draw groups until the next does not fit, then shrink that one to fill the row exactly."""
    groups: List[Group] = []
    left = row_len
    while left > 0:
        p, rs = draw_group(rng)
        tot = p + sum(rs)
        if tot <= left:
            groups.append((p, tuple(rs)))
            left -= tot
            continue
        if left < 8 and groups:
            lp, lrs = groups[-1]
            groups[-1] = (lp, tuple(lrs[:-1]) + (lrs[-1] + left,))
            left = 0
            break
        n = len(rs)
        if left < n + 1:
            n = max(1, left - 1)
            rs = rs[:n]
            tot = p + sum(rs)
        new_rs = [max(1, int(r * left / tot)) for r in rs]
        while sum(new_rs) >= left:
            new_rs[int(np.argmax(new_rs))] -= 1
        groups.append((left - sum(new_rs), tuple(new_rs)))
        left = 0
    assert sum(p + sum(rs) for p, rs in groups) == row_len
    return groups


def config3(seed: int = 3) -> Workload:
    """72B-class shape: 2 rows x 8192 tokens, several (prompt, 2-response) groups per row."""
    rng = _rng(seed)

    def draw(rng):
        p = _lognormal_int(rng, 768, 0.5, 64, 4096)
        return p, [int(rng.integers(64, 769)) for _ in range(2)]

    rows = [_fill_row(rng, 8192, draw) for _ in range(2)]
    return Workload("config3", rows, 64, 8, 128, seed=seed)


CONFIG4_POINTS = [(rho, n) for rho in (1, 4, 16) for n in (2, 4)]


def config4(point: int = 0, num_rows: int = 2, row_len: int = 32768) -> Workload:
    """Length-sorted long rows; sweep point = (prompt : mean-response ratio, n)."""
    rho, n = CONFIG4_POINTS[point]
    seed = 400 + point
    rng = _rng(seed)
    totals = sorted((_lognormal_int(rng, 4096, 0.6, 1024, 16384) for _ in range(64)), reverse=True)
    it = iter(totals)

    def draw(rng):
        g = next(it)
        rbar = g / (rho + n)
        rs = [max(16, int(round(rbar * rng.uniform(0.75, 1.25)))) for _ in range(n)]
        return max(1, g - sum(rs)), rs

    rows = [_fill_row(rng, row_len, draw) for _ in range(num_rows)]
    return Workload(f"config4[rho={rho},n={n}]", rows, 32, 8, 128, seed=seed)


def all_configs() -> List[Workload]:
    return [config0(), config1(), config2(), config3()] + [config4(s) for s in range(len(CONFIG4_POINTS))]


def tiny(seed: int, num_rows=1, groups_per_row=1, n_resp=2, p_range=(3, 9), r_range=(1, 6),
         hq=1, hkv=1, d=8) -> Workload:
    """Small random structure for brute-force checks."""
    rng = _rng(seed)
    rows = []
    for _ in range(num_rows):
        row = []
        for _ in range(groups_per_row):
            p = int(rng.integers(p_range[0], p_range[1] + 1))
            rs = tuple(int(rng.integers(r_range[0], r_range[1] + 1)) for _ in range(n_resp))
            row.append((p, rs))
        rows.append(row)
    return Workload(f"tiny{seed}", rows, hq, hkv, d, seed=seed)


# ------------------------------------------------------------------------------
# The unpacked paired baseline: every [x, y_k] as its own single-response group
# ------------------------------------------------------------------------------

def unpacked(w: Workload, padded: bool = True):
    """Workload in which each (x, y_k) is an independent plain-causal sequence.

    Returns (workload, gather) where gather[t'] is the packed token whose Q/K/V row
    stands at unpacked position t' (pad positions re-use the prompt's first token;
    their results are discarded).  With ``padded`` every pair of a group is padded to
    P + max_k R_k (paper Sec. 3.2.1, l_original)."""
    rows, gather = [], []
    t = 0
    for row in w.rows:
        new_row = []
        for (p, rs) in row:
            rmax = max(rs)
            off = t + p
            for r in rs:
                rl = rmax if padded else r
                new_row.append((p, (rl,)))
                gather.extend(range(t, t + p))
                gather.extend(range(off, off + r))
                gather.extend([t] * (rl - r))
                off += r
            t += p + sum(rs)
        rows.append(new_row)
    uw = dataclasses.replace(w, name=w.name + ("/unpacked-padded" if padded else "/unpacked"),
                             rows=rows, low_var_ranges=[])
    return uw, torch.tensor(gather, dtype=torch.long)


def random_structure(seed: int, long: bool = False) -> Workload:
    """Seeded random packing structure for tests: 1-3 rows of 1-3 groups with 1-5 responses
    each, lengths drawn so that segment ends fall before, on and after 128-token tile
    boundaries; random GQA ratio (odd ones included) and head size.  ``long``: segments of up
    to a dozen tiles (uniform lengths in [1, 1500])."""
    rng = np.random.default_rng(seed + (7919 if long else 0))
    if long:
        pick = lambda: int(rng.integers(1, 1501))
    else:
        pick = lambda: int(rng.choice([1, 2, 17, 63, 64, 65, 127, 128, 129, 200, 257]))
    rows = [[(pick(), tuple(pick() for _ in range(rng.integers(1, 6))))
             for _ in range(rng.integers(1, 4))] for _ in range(rng.integers(1, 4))]
    hkv = int(rng.choice([1, 2, 3]))
    r = int(rng.choice([1, 2, 3, 4, 5]))
    d = int(rng.choice([64, 128]))
    return Workload(f"random{'-long' if long else ''}{seed}", rows, hkv * r, hkv, d, seed=1000 + seed)
