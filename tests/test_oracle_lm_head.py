"""Pins for oracle/lm_head.py (CPU only)."""
import numpy as np

from oracle import lm_head as OL


def test_logits_by_explicit_loops_on_a_tiny_case():
    rng = np.random.default_rng(0)
    h = rng.normal(size=(3, 5)); w = rng.normal(size=(7, 5))
    ref = np.zeros((3, 7))
    for s in range(3):
        for v in range(7):
            for d in range(5):
                ref[s, v] += h[s, d] * w[v, d]
    np.testing.assert_allclose(OL.lm_head_logits(h, w), ref, rtol=1e-13)


def test_planted_winner_and_acceptance():
    """hidden rows are built along chosen weight rows, so the winner of every row is known."""
    rng = np.random.default_rng(1)
    V, H = 50, 16
    w = rng.normal(size=(V, H))
    tokens = np.array([9, 11, 12, 13, 20, 21, 0, 0])       # two requests: k = 4 and 2
    k, off = [4, 2], [0, 4, 6]
    win = [11, 12, 40, 3, 21, 5, 0, 0]                      # row s -> winning token
    h = np.stack([3.0 * w[t] / (w[t] @ w[t]) * 8 for t in win])
    r = OL.lm_head_accept(h, w, tokens, k, off, 2, 2)
    assert list(r["top1"][:6]) == win[:6]
    assert list(r["accept_len"]) == [2, 1] and list(r["next_anchor"]) == [40, 5]
