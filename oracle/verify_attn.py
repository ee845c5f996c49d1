"""Oracle: packed ragged verify attention, written as its plain definition.

TEST INFRASTRUCTURE ONLY -- see the package docstring.

For live request i (k_i query rows packed at offset_i .. offset_i + k_i - 1),
q-head h with kv-head g = h // (H_q / H_kv), the result is ordinary softmax
attention

    o = softmax(q K^T * sm_scale + mask) V

over that request's own keys, gathered from the paged cache through its
block table, where row j may see the logical keys 0 .. ctx_i + j inclusive
(request-local causal masking inside the verify window, everything before
it; Eq. 15 and the sentence after it).  Rows of sentinel requests and slots
at or beyond M_live are defined as zero.

`verify_attn` works on the packed layout.  `verify_attn_padded` is the
unpacked formulation (every request carries all W = 16 rows, one dense mask
over ctx_i + 16 keys); the two must agree on the live rows, which is one of
the pins of this file.  Matrix products and exp come from numpy; nothing is
blocked, fused or reordered.
"""
from __future__ import annotations

import numpy as np

PAGE = 16


def gather_kv(cache: np.ndarray, block_table_row, n_tokens: int, kv_head: int) -> np.ndarray:
    """Dense [n_tokens, D] view of one request's keys (or values) for one
    kv-head.  cache is [num_pages, H_kv, PAGE, D]; logical token t lives in
    physical page block_table_row[t // PAGE], slot t % PAGE."""
    n_pages = (n_tokens + PAGE - 1) // PAGE
    pages = np.asarray(block_table_row[:n_pages], dtype=np.int64)
    dense = cache[pages, kv_head]                       # [n_pages, PAGE, D]
    return dense.reshape(n_pages * PAGE, -1)[:n_tokens]


def _softmax_rows(S: np.ndarray) -> np.ndarray:
    m = S.max(axis=-1, keepdims=True)
    P = np.exp(S - m)
    return P / P.sum(axis=-1, keepdims=True)


def verify_attn(q, k_cache, v_cache, block_table, ctx_len, k, offset, n_live,
                n_q_heads: int, n_kv_heads: int, sm_scale: float,
                dtype=np.float32) -> np.ndarray:
    """Packed verify attention.

    q        [M_bs, H_q, D]  packed query rows (values already bf16-rounded)
    k_cache  [num_pages, H_kv, PAGE, D], v_cache likewise
    k, offset  lengths and packed offsets from the allocation
    Returns out [M_bs, H_q, D] in `dtype`; rows >= M_live are zero.
    """
    q = np.asarray(q, dtype=dtype)
    k_cache = np.asarray(k_cache)
    v_cache = np.asarray(v_cache)
    M_bs, H_q, D = q.shape
    G = n_q_heads // n_kv_heads
    out = np.zeros((M_bs, H_q, D), dtype=dtype)
    for i in range(int(n_live)):
        ki, ci, oi = int(k[i]), int(ctx_len[i]), int(offset[i])
        n_keys = ci + ki
        # mask[j][t] = (t <= ctx_i + j), materialised
        t_idx = np.arange(n_keys)[None, :]
        j_idx = np.arange(ki)[:, None]
        mask = t_idx <= (ci + j_idx)
        for g in range(n_kv_heads):
            K = gather_kv(k_cache, block_table[i], n_keys, g).astype(dtype)
            V = gather_kv(v_cache, block_table[i], n_keys, g).astype(dtype)
            for h in range(g * G, (g + 1) * G):
                Qh = q[oi:oi + ki, h, :]
                S = (Qh @ K.T) * dtype(sm_scale)
                S = np.where(mask, S, dtype(-np.inf))
                P = _softmax_rows(S)
                out[oi:oi + ki, h, :] = P @ V
    return out


def verify_attn_padded(q_unpacked, k_cache, v_cache, block_table, ctx_len, n_live,
                       n_q_heads: int, n_kv_heads: int, sm_scale: float,
                       W: int = 16, dtype=np.float32) -> np.ndarray:
    """Unpacked verify: every live request has all W rows.

    q_unpacked [n_bs, W, H_q, D] -> out [n_bs, W, H_q, D]; row j attends to
    logical keys 0 .. ctx_i + j of a cache that holds ctx_i + W tokens."""
    q_unpacked = np.asarray(q_unpacked, dtype=dtype)
    n_bs, Wq, H_q, D = q_unpacked.shape
    assert Wq == W
    G = n_q_heads // n_kv_heads
    out = np.zeros_like(q_unpacked)
    for i in range(int(n_live)):
        ci = int(ctx_len[i])
        n_keys = ci + W
        allowed = np.tril(np.ones((W, W), dtype=bool))          # window: causal
        mask = np.concatenate([np.ones((W, ci), dtype=bool), allowed], axis=1)
        for h in range(H_q):
            g = h // G
            K = gather_kv(k_cache, block_table[i], n_keys, g).astype(dtype)
            V = gather_kv(v_cache, block_table[i], n_keys, g).astype(dtype)
            S = (q_unpacked[i, :, h, :] @ K.T) * dtype(sm_scale)
            S[~mask] = -np.inf
            out[i, :, h, :] = _softmax_rows(S) @ V
    return out


def verify_attn_row(q_row, k_cache, v_cache, block_table_row, n_visible: int,
                    kv_head: int, sm_scale: float, dtype=np.float64) -> np.ndarray:
    """One output row by the definition: a single query vector against its
    first `n_visible` logical keys.  Used to spot-check full-size runs."""
    K = gather_kv(k_cache, block_table_row, n_visible, kv_head).astype(dtype)
    V = gather_kv(v_cache, block_table_row, n_visible, kv_head).astype(dtype)
    s = (K @ np.asarray(q_row, dtype=dtype)) * dtype(sm_scale)
    p = np.exp(s - s.max())
    return (p / p.sum()) @ V
