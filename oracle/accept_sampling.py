"""Oracle: prefix verification under a sampling target policy (temperature > 0).

TEST INFRASTRUCTURE ONLY -- see the package docstring.

"Prefix verifier" paragraph: P is the target policy's next-token distribution
at a packed row, here P = softmax(logits / temperature).  The drafter's
candidate x is deterministic (its top-1), so it is accepted with probability
P(x).  At the first rejection the successor is drawn from P with x removed
and the rest renormalised; if all k_i - 1 selected candidates pass, it is
drawn from the unmodified P of the last selected row.  Row offset_i + a_i
supplies the successor.  The random numbers are inputs (one uniform per
packed row for the acceptance test, one per request for the draw), so the
lengths never depend on them and both sides of a parity test see the same
draws.

Everything is evaluated in binary64, in the order of the definition:
normaliser by a plain sum, acceptance by `u < P(x)`, the draw by the first
index whose cumulative (unnormalised) weight exceeds `u * total`.
"""
from __future__ import annotations

import numpy as np


def row_distribution(logits_row: np.ndarray, temperature: float) -> np.ndarray:
    """Unnormalised weights w_v = exp((l_v - max) / T) in binary64."""
    z = np.asarray(logits_row, dtype=np.float64) / float(temperature)
    return np.exp(z - z.max())


def draw_index(weights: np.ndarray, u: float) -> int:
    """Inverse CDF: first v with sum_{w <= v} weights[w] > u * sum(weights)."""
    c = np.cumsum(weights)
    target = float(u) * float(c[-1])
    v = int(np.searchsorted(c, target, side="right"))
    return min(v, len(weights) - 1)


def accept_sampling(logits, vocab: int, temperature: float, u_accept, u_draw, tokens, k, offset,
                    n_live: int, n_bs: int, W: int = 16):
    """Returns dict(accept_len, next_anchor, out_tokens, out_len, p_draft) where
    p_draft[s] = P(tokens[s + 1]) at packed row s (0 where the row has no candidate)."""
    logits = np.asarray(logits)
    accept_len = np.zeros(n_bs, dtype=np.int32)
    next_anchor = np.full(n_bs, -1, dtype=np.int32)
    out_tokens = np.full((n_bs, W), -1, dtype=np.int32)
    out_len = np.zeros(n_bs, dtype=np.int32)
    p_draft = np.zeros(logits.shape[0], dtype=np.float64)
    for i in range(int(n_live)):
        ki, oi = int(k[i]), int(offset[i])
        a = 0
        rejected = False
        while a < ki - 1:
            w = row_distribution(logits[oi + a, :vocab], temperature)
            x = int(tokens[oi + a + 1])
            px = float(w[x] / w.sum())
            p_draft[oi + a] = px
            if float(u_accept[oi + a]) < px:
                a += 1
            else:
                rejected = True
                break
        w = row_distribution(logits[oi + a, :vocab], temperature)
        if rejected:
            w = w.copy()
            w[int(tokens[oi + a + 1])] = 0.0          # remove the rejected candidate, renormalise
        nxt = draw_index(w, float(u_draw[i]))
        accept_len[i] = a
        next_anchor[i] = nxt
        for j in range(a):
            out_tokens[i, j] = tokens[oi + 1 + j]
        out_tokens[i, a] = nxt
        out_len[i] = a + 1
    return dict(accept_len=accept_len, next_anchor=next_anchor, out_tokens=out_tokens,
                out_len=out_len, p_draft=p_draft)


def draw_interval(weights: np.ndarray, v: int):
    """[lo, hi) of u for which draw_index returns v: for tolerance-aware checks."""
    c = np.cumsum(weights)
    lo = 0.0 if v == 0 else float(c[v - 1] / c[-1])
    return lo, float(c[v] / c[-1])
