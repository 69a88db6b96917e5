"""Oracle for the row builder (test infrastructure: only tests, smoke() and the benchmark's CPU
legs may import this package; the product path never does).

The step before the attention path (paper Sec. 2.2; used with preference packing in Sec. 5.2,
Table 2): preference groups
[prompt | responses] of varying length are put into rows of at most `capacity` tokens.

Reading of the paper (it names the two techniques and gives no algorithm):
  * batch sorting (samples of similar length share a batch): the groups are ordered by total
    length (prompt + all responses), longest first; ties keep their original order;
  * batch packing (sequences concatenated up to a length limit): consecutive groups of that
    order are concatenated into one row while the row stays within `capacity` (next fit), so
    a row holds groups of similar length;
  * rows therefore come out in decreasing length, and a data-parallel step takes consecutive
    rows, one per rank, which is what keeps the ranks' work similar; `row_cost` (visible
    query-key pairs, the attention cost of Sec. 3.2.1) is reported for that purpose.

Plain Python loops over numpy int64 arrays; written from the definitions, no shared code with
the CUDA path.
"""
import numpy as np


def group_tokens(grp_prompt_len, grp_resp_off, resp_len):
    """Total tokens of each group: prompt + all of its responses."""
    P = np.asarray(grp_prompt_len, dtype=np.int64)
    off = np.asarray(grp_resp_off, dtype=np.int64)
    R = np.asarray(resp_len, dtype=np.int64)
    return np.array([P[g] + R[off[g]:off[g + 1]].sum() for g in range(len(P))], dtype=np.int64)


def group_pairs(grp_prompt_len, grp_resp_off, resp_len):
    """Visible (query, key) pairs of each group under the packing mask (Sec. 3.2): the prompt
    is causal, P (P + 1) / 2; every response token sees the whole prompt and its own response
    causally, R P + R (R + 1) / 2."""
    P = np.asarray(grp_prompt_len, dtype=np.int64)
    off = np.asarray(grp_resp_off, dtype=np.int64)
    R = np.asarray(resp_len, dtype=np.int64)
    out = np.zeros(len(P), dtype=np.int64)
    for g in range(len(P)):
        u = P[g] * (P[g] + 1) // 2
        for r in R[off[g]:off[g + 1]]:
            u += r * P[g] + r * (r + 1) // 2
        out[g] = u
    return out


def build_rows(grp_prompt_len, grp_resp_off, resp_len, capacity):
    """Returns a dict:
      order          [G]   original index of the group at each sorted position
      row_group_off  [rows + 1]  sorted positions [off[r], off[r+1]) form row r
      row_tokens     [rows]
      row_cost       [rows]  visible pairs
      grp_prompt_len, grp_resp_off, resp_len   the descriptors in row order
    Raises ValueError if a group alone exceeds the capacity."""
    tok = group_tokens(grp_prompt_len, grp_resp_off, resp_len)
    cost = group_pairs(grp_prompt_len, grp_resp_off, resp_len)
    G = len(tok)
    if G and tok.max() > capacity:
        raise ValueError("a group is longer than the row capacity")
    order = sorted(range(G), key=lambda g: (-int(tok[g]), g))
    row_group_off, row_tokens, row_cost = [0], [], []
    cur_t, cur_c = 0, 0
    for pos, g in enumerate(order):
        if pos > row_group_off[-1] and cur_t + tok[g] > capacity:
            row_group_off.append(pos)
            row_tokens.append(cur_t)
            row_cost.append(cur_c)
            cur_t, cur_c = 0, 0
        cur_t += int(tok[g])
        cur_c += int(cost[g])
    if G:
        row_group_off.append(G)
        row_tokens.append(cur_t)
        row_cost.append(cur_c)
    P = np.asarray(grp_prompt_len, dtype=np.int64)
    off = np.asarray(grp_resp_off, dtype=np.int64)
    R = np.asarray(resp_len, dtype=np.int64)
    new_P = [int(P[g]) for g in order]
    new_off, new_R = [0], []
    for g in order:
        new_R.extend(int(x) for x in R[off[g]:off[g + 1]])
        new_off.append(len(new_R))
    i32 = lambda a: np.asarray(a, dtype=np.int32)
    return {"order": i32(order), "row_group_off": i32(row_group_off),
            "row_tokens": np.asarray(row_tokens, dtype=np.int64),
            "row_cost": np.asarray(row_cost, dtype=np.int64),
            "grp_prompt_len": i32(new_P), "grp_resp_off": i32(new_off), "resp_len": i32(new_R)}


def assign_rows(row_cost, num_ranks):
    """Rows -> data-parallel ranks (Sec. 2.2: sorting by length exists so that no rank waits for
    the one holding the longest sequences).  Reading: longest-processing-time list scheduling
    on the attention cost -- rows in order of decreasing cost (ties: lower index first), each
    to the rank with the least total so far (ties: lowest rank).
    Returns (order [rows], rank_of_row [rows], rank_cost [ranks])."""
    cost = [int(c) for c in row_cost]
    order = sorted(range(len(cost)), key=lambda r: (-cost[r], r))
    load = [0] * num_ranks
    rank_of_row = [0] * len(cost)
    for r in order:
        k = min(range(num_ranks), key=lambda i: (load[i], i))
        rank_of_row[r] = k
        load[k] += cost[r]
    return (np.asarray(order, dtype=np.int32), np.asarray(rank_of_row, dtype=np.int32),
            np.asarray(load, dtype=np.int64))
