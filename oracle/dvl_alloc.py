"""Oracle: DVL allocation and flat-pack (Algorithm 1), step by step.

TEST INFRASTRUCTURE ONLY -- see the package docstring.

The allocation is an iteration with a tie-break, so this file follows the
algorithm's steps in the paper's order and notation instead of a closed
form.  All score arithmetic is IEEE binary32 with round-to-nearest-even and
no reassociation, because the integer lengths depend on it:

* Eq. 6   q_0 = 1, q_j = min(q_{j-1}, s_j)            (min only, exact)
* Eq. 7   l_hat = ((q_1 + q_2) + q_3) + ... + q_{W-1}  (left to right, fp32)
          k0 = min(W, max(1, floor(l_hat + 1/2)))      (fp32 add, then floor)
* Eq. 9   grow: argmax_{k_i<W} q[i][k_i]; shrink: argmin_{k_i>1} q[i][k_i-1];
          the lowest request index wins a tie in both branches.
* Eq. 10  offset_i = sum_{j<i} k_j
* Eq. 11  buffer.field[offset_i + j] = field_i[j], 0 <= j < k_i
* Algorithm 1, last two lines: sentinels for i >= N and slots >= M_live.

Readings taken where the paper is silent (tie-break, summation order,
round-half-up, the meaning of "positions" and "KV refs" for a paged cache)
are the ones listed in the design notes of the repository.
"""
from __future__ import annotations

import math

import numpy as np

W_DEFAULT = 16
PAGE = 16

_F32 = np.float32


def sigmoid_f32(x) -> np.float32:
    """sigma(x) of Algorithm 1 line 2, evaluated in binary64 and rounded once
    to binary32 (the only transcendental on the path; used in logits mode)."""
    return _F32(1.0 / (1.0 + math.exp(-float(x))))


def prefix_scores(s_row, logits_mode: bool = False, W: int = W_DEFAULT) -> np.ndarray:
    """Eq. 6: Q row of length W with q_0 = 1 and a running minimum after it.

    s_row holds the W-1 per-position scores (slot j=1..W-1): acceptance
    probabilities, or predictor logits when logits_mode is set."""
    q = np.empty(W, dtype=_F32)
    q[0] = _F32(1.0)
    for j in range(1, W):
        s = sigmoid_f32(s_row[j - 1]) if logits_mode else _F32(s_row[j - 1])
        q[j] = s if s < q[j - 1] else q[j - 1]
    return q


def seed_length(q: np.ndarray, W: int = W_DEFAULT) -> int:
    """Eq. 7: round the draft-only score sum half up and clip to [1, W].

    The anchor is *not* added: l_hat = 6.2 gives 6 slots = anchor + 5."""
    l_hat = _F32(0.0)
    for j in range(1, W):
        l_hat = _F32(l_hat + q[j])          # sequential fp32 accumulation
    r = int(math.floor(float(_F32(l_hat + _F32(0.5)))))
    return min(W, max(1, r))


def budget_adjust(Q: np.ndarray, k0, budget: int, W: int = W_DEFAULT):
    """Algorithm 1 lines 4-12 (Eq. 8-9): the serial grow / shrink loop.

    Returns (k, n_updates).  Q is [N, W] float32, k0 the integer seeds."""
    k = [int(x) for x in k0]
    N = len(k)
    delta = budget - sum(k)
    updates = 0
    while delta > 0:
        best_i, best_q = -1, None
        for i in range(N):
            if k[i] < W:
                v = Q[i][k[i]]
                if best_i < 0 or v > best_q:     # strict: lowest index keeps a tie
                    best_i, best_q = i, v
        if best_i < 0:
            raise ValueError("budget exceeds N*W")
        k[best_i] += 1
        delta -= 1
        updates += 1
    while delta < 0:
        best_i, best_q = -1, None
        for i in range(N):
            if k[i] > 1:
                v = Q[i][k[i] - 1]
                if best_i < 0 or v < best_q:     # strict: lowest index keeps a tie
                    best_i, best_q = i, v
        if best_i < 0:
            raise ValueError("budget below N")
        k[best_i] -= 1
        delta += 1
        updates += 1
    return k, updates


def offsets_of(k) -> list:
    """Eq. 10: exclusive prefix sum, with the end boundary appended."""
    off = [0]
    for x in k:
        off.append(off[-1] + int(x))
    return off


def dvl_alloc(n_bs: int, n_live: int, scores, draft_tokens, ctx_len, block_table,
              logits_mode: bool = False, W: int = W_DEFAULT, budget: int | None = None,
              capacity: int | None = None):
    """Whole of Algorithm 1 from the scores down.

    scores        [n_bs, W-1] float32, slot j=1..W-1
    draft_tokens  [n_bs, W]   int, slot 0 = anchor
    ctx_len       [n_bs]      committed tokens already cached (anchor excluded)
    block_table   [n_bs, max_pages] physical page of logical page p

    budget        total verification rows M_live (default (W/2) N, Eq. 3); any total
                  in [N, W N] that fits the packed capacity: Eq. 9 does not depend on it
    capacity      rows of the packed arrays (default (W/2) n_bs, the paper's M_bs)

    Returns a dict with k, k0, offset, q_start, q_end, tokens, positions,
    kv_refs, row_req, Q, n_updates.  Packed arrays have (W/2)*n_bs slots.
    """
    scores = np.asarray(scores, dtype=_F32)
    draft_tokens = np.asarray(draft_tokens)
    ctx_len = np.asarray(ctx_len)
    block_table = np.asarray(block_table)
    N = int(n_live)
    assert 1 <= N <= n_bs
    M_bs = (W // 2) * n_bs if capacity is None else int(capacity)
    M_live = (W // 2) * N if budget is None else int(budget)
    assert N <= M_live <= min(W * N, M_bs), "budget outside [N, min(W N, capacity)]"

    Q = np.stack([prefix_scores(scores[i], logits_mode, W) for i in range(N)])
    k0 = [seed_length(Q[i], W) for i in range(N)]
    k_live, n_updates = budget_adjust(Q, k0, M_live, W)
    off_live = offsets_of(k_live)

    k = np.zeros(n_bs, dtype=np.int32)
    offset = np.zeros(n_bs + 1, dtype=np.int32)
    k[:N] = k_live
    offset[: N + 1] = off_live
    offset[N + 1:] = M_live                      # sentinel boundaries

    tokens = np.zeros(M_bs, dtype=np.int32)
    positions = np.zeros(M_bs, dtype=np.int32)
    kv_refs = np.zeros(M_bs, dtype=np.int32)
    row_req = np.full(M_bs, -1, dtype=np.int32)

    def ref(i, j):
        t = int(ctx_len[i]) + j
        return int(block_table[i][t // PAGE]) * PAGE + t % PAGE

    for i in range(N):
        for j in range(k_live[i]):
            s = off_live[i] + j
            tokens[s] = draft_tokens[i][j]
            positions[s] = int(ctx_len[i]) + j
            kv_refs[s] = ref(i, j)
            row_req[s] = i
    tail_ref = ref(0, 0)                         # "KV refs of request 1, slot 0"
    for s in range(M_live, M_bs):
        tokens[s] = 0
        positions[s] = 0
        kv_refs[s] = tail_ref

    k0_full = np.zeros(n_bs, dtype=np.int32)
    k0_full[:N] = k0
    return dict(k=k, k0=k0_full, offset=offset,
                q_start=offset[:-1].copy(), q_end=(offset[:-1] + k).astype(np.int32),
                tokens=tokens, positions=positions, kv_refs=kv_refs, row_req=row_req,
                Q=Q, n_updates=n_updates, m_live=M_live)


def prefix_objective(Q: np.ndarray, k) -> float:
    """Objective of Eq. 8: sum_i sum_{j<k_i} q_ij, in binary64."""
    return float(sum(float(Q[i][j]) for i in range(len(k)) for j in range(int(k[i]))))
