"""TEST INFRASTRUCTURE: plain numpy fp64 oracle of the loss-side consumer (paper Sec. 2.1).

Splits packed rows back into responses: s_k = sum of the response's token log-probs; reward
r_k = beta (s_k - s_k_ref) (DPO with the log-ratio; beta s_k without a reference); responses
are ranked as in Sec. 3.1 (a preferred over b for a > b); group loss = mean over pairs a > b of
-log sigmoid(r_a - r_b).  Gradients are written out from the definition.

Pinned by tests/test_oracle_loss_pins.py: torch logsigmoid + autograd on independently sliced
sequences, the K = 2 closed form of the DPO loss, equal rewards -> log 2, finite differences.
Shares no code with the CUDA library.
"""
from __future__ import annotations

import numpy as np


def preference_loss(rows, token_logp, ref_token_logp, beta):
    """Returns (resp_logp [N], resp_reward [N], grp_loss [G], d_token_logp [T]) in fp64."""
    lp = np.asarray(token_logp, dtype=np.float64)
    ref = None if ref_token_logp is None else np.asarray(ref_token_logp, dtype=np.float64)
    resp_logp, resp_reward, grp_loss = [], [], []
    grad = np.zeros_like(lp)
    t = 0
    for row in rows:
        for (p, rs) in row:
            off = t + p
            spans, rew = [], []
            for r in rs:
                s = lp[off:off + r].sum()
                sr = 0.0 if ref is None else ref[off:off + r].sum()
                resp_logp.append(s)
                rew.append(beta * (s - sr))
                spans.append((off, off + r))
                off += r
            resp_reward.extend(rew)
            n = len(rs)
            pairs = [(a, b) for a in range(n) for b in range(a)]
            loss = 0.0
            g = np.zeros(n)
            for (a, b) in pairs:
                d = rew[a] - rew[b]
                loss += np.log1p(np.exp(-d)) if d > -30 else -d          # -log sigmoid(d)
                sneg = 1.0 / (1.0 + np.exp(d))                            # sigmoid(-d)
                g[a] -= sneg
                g[b] += sneg
            if pairs:
                loss /= len(pairs)
                g /= len(pairs)
            grp_loss.append(loss)
            for k, (a, b) in enumerate(spans):
                grad[a:b] = beta * g[k]
            t = off
    return (np.asarray(resp_logp), np.asarray(resp_reward), np.asarray(grp_loss), grad)
