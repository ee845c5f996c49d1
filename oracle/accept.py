"""Oracle: greedy prefix verification and output building.

TEST INFRASTRUCTURE ONLY -- see the package docstring.

Greedy decoding (temperature 0): the target's token at a packed row is the
index of the largest logit of that row, lowest index among equal maxima; a
NaN never counts as a maximum.  Request i accepts its candidates in order
while the target token predicted by the previous slot equals the candidate
("Prefix verifier" paragraph): slot j's logits decide on the token in slot j+1.
After a_i accepted candidates the row offset_i + a_i supplies the successor,
which is also the next anchor; if all k_i - 1 selected candidates pass, the
last selected row supplies it.  Outputs follow Algorithm 2, lines 21-26:
tokens (accepted candidates then successor), length a_i + 1, next.
"""
from __future__ import annotations

import numpy as np


def row_argmax(logits: np.ndarray, n_rows: int, vocab: int) -> np.ndarray:
    """top1[s] for s < n_rows over columns [0, vocab); first index of the max."""
    top1 = np.zeros(logits.shape[0], dtype=np.int32)
    for s in range(int(n_rows)):
        row = np.asarray(logits[s, :vocab], dtype=np.float32)
        row = np.where(np.isnan(row), -np.inf, row)
        top1[s] = int(np.argmax(row))            # numpy returns the first maximum
    return top1


def accept_prefix(top1, tokens, k, offset, n_live: int, n_bs: int, W: int = 16,
                  ctx_len=None):
    """Sequential acceptance loop per request.

    Returns dict(accept_len, next_anchor, out_tokens, out_len[, ctx_len])."""
    accept_len = np.zeros(n_bs, dtype=np.int32)
    next_anchor = np.full(n_bs, -1, dtype=np.int32)
    out_tokens = np.full((n_bs, W), -1, dtype=np.int32)
    out_len = np.zeros(n_bs, dtype=np.int32)
    new_ctx = None if ctx_len is None else np.array(ctx_len, dtype=np.int32, copy=True)
    for i in range(int(n_live)):
        ki, oi = int(k[i]), int(offset[i])
        a = 0
        while a < ki - 1 and int(top1[oi + a]) == int(tokens[oi + a + 1]):
            a += 1
        nxt = int(top1[oi + a])
        accept_len[i] = a
        next_anchor[i] = nxt
        for j in range(a):
            out_tokens[i, j] = tokens[oi + 1 + j]
        out_tokens[i, a] = nxt
        out_len[i] = a + 1
        if new_ctx is not None:
            new_ctx[i] += a + 1
    res = dict(accept_len=accept_len, next_anchor=next_anchor,
               out_tokens=out_tokens, out_len=out_len)
    if new_ctx is not None:
        res["ctx_len"] = new_ctx
    return res


def accept(logits, vocab: int, tokens, k, offset, n_live: int, n_bs: int,
           W: int = 16, ctx_len=None):
    """row_argmax over the M_live = (W/2) * n_live live rows, then the loop."""
    m_live = int(offset[int(n_live)])
    top1 = row_argmax(np.asarray(logits), m_live, vocab)
    res = accept_prefix(top1, tokens, k, offset, n_live, n_bs, W, ctx_len)
    res["top1"] = top1
    return res
