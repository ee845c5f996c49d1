"""Oracle: target token per packed row from the LM head, by the definition.

TEST INFRASTRUCTURE ONLY -- see the package docstring.

logits[s, v] = sum_h hidden[s, h] * weight[v, h] (binary64 on the bf16-valued
inputs), top1[s] = first index of the row maximum.  This is what the fused
LM-head + argmax kernel must reproduce without ever writing the logits; the
acceptance loop afterwards is oracle/accept.py's.
"""
from __future__ import annotations

import numpy as np

from . import accept as _acc


def lm_head_logits(hidden: np.ndarray, weight: np.ndarray) -> np.ndarray:
    return np.asarray(hidden, dtype=np.float64) @ np.asarray(weight, dtype=np.float64).T


def lm_head_accept(hidden, weight, tokens, k, offset, n_live: int, n_bs: int, W: int = 16):
    logits = lm_head_logits(hidden, weight)
    res = _acc.accept(logits, logits.shape[1], tokens, k, offset, n_live, n_bs, W)
    res["logits"] = logits
    return res
