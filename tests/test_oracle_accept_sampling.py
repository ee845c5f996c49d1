"""Pins for oracle/accept_sampling.py (CPU only)."""
import numpy as np
import pytest

from dscale_inputs import CONFIGS, make_logits_unpacked, make_requests, rows_to_packed, small_variant
from oracle import accept as OG
from oracle import accept_sampling as OS
from oracle import dvl_alloc as OA


def test_draw_index_closed_forms():
    w = np.ones(8)
    for u, v in ((0.0, 0), (0.124, 0), (0.125, 1), (0.5, 4), (0.99, 7)):
        assert OS.draw_index(w, u) == v                      # uniform weights: floor(8 u)
    w = np.array([0.0, 2.0, 0.0, 6.0])
    assert OS.draw_index(w, 0.0) == 1 and OS.draw_index(w, 0.2499) == 1
    assert OS.draw_index(w, 0.25) == 3 and OS.draw_index(w, 0.999) == 3   # zero weights are never drawn
    lo, hi = OS.draw_interval(w, 3)
    assert (lo, hi) == (0.25, 1.0)


def _single(logits_rows, tokens, u_acc, u_draw, T=1.0):
    k = [len(tokens)]
    off = [0, len(tokens)]
    lg = np.zeros((8, logits_rows.shape[1]), dtype=np.float32)
    lg[: len(logits_rows)] = logits_rows
    ua = np.zeros(8); ua[: len(u_acc)] = u_acc
    return OS.accept_sampling(lg, logits_rows.shape[1], T, ua, [u_draw], np.array(tokens + [0] * 8), k, off, 1, 1)


def test_first_emitted_token_follows_the_target_distribution():
    """Accept x with probability P(x), otherwise draw from P without x, renormalised: the first
    emitted token is then distributed exactly as P.  Checked by enumerating a grid of uniforms."""
    rng = np.random.default_rng(0)
    V, x = 6, 2
    rows = rng.normal(0, 1.5, size=(2, V)).astype(np.float32)
    P = OS.row_distribution(rows[0], 0.8); P = P / P.sum()
    n = 300
    us = (np.arange(n) + 0.5) / n
    counts = np.zeros(V)
    for ua in us:
        for ud in us:
            r = _single(rows, [9, x], [ua], ud, T=0.8)
            counts[r["out_tokens"][0, 0]] += 1
    np.testing.assert_allclose(counts / n ** 2, P, atol=2.5 / n)


def test_acceptance_threshold_and_all_pass():
    rng = np.random.default_rng(1)
    V = 7
    rows = rng.normal(0, 1, size=(3, V)).astype(np.float32)
    toks = [0, 4, 5]
    p0 = OS.row_distribution(rows[0], 1.0); p0 = p0[4] / p0.sum()
    p1 = OS.row_distribution(rows[1], 1.0); p1 = p1[5] / p1.sum()
    r = _single(rows, toks, [p0 * 0.999, p1 * 0.999], 0.0)
    assert r["accept_len"][0] == 2 and r["out_len"][0] == 3           # both pass: successor from the last row
    w2 = OS.row_distribution(rows[2], 1.0)
    assert r["next_anchor"][0] == OS.draw_index(w2, 0.0)
    np.testing.assert_allclose(r["p_draft"][:2], [p0, p1], rtol=1e-12)
    r = _single(rows, toks, [p0 * 1.001, 0.0], 0.3)
    assert r["accept_len"][0] == 0                                     # first candidate rejected
    w0 = OS.row_distribution(rows[0], 1.0); w0[4] = 0
    assert r["next_anchor"][0] == OS.draw_index(w0, 0.3) != 4          # the rejected token cannot come back
    r = _single(rows, toks, [0.0, p1 * 1.001], 0.9)
    assert r["accept_len"][0] == 1 and r["out_tokens"][0, 0] == 4


def test_all_pass_draws_from_the_last_rows_unmodified_distribution():
    """When every candidate passes, the successor comes from the last selected row's P as it
    stands ("Prefix verifier" paragraph): no token is removed, the last candidate itself can be
    drawn again.  The last row's P is fixed by hand (logits = log of 0.1, 0.2, 0.3, 0.4), so the
    expected token for each uniform follows from the cumulative sums 0.1, 0.3, 0.6, 1.0."""
    probs = np.array([0.1, 0.2, 0.3, 0.4])
    rows = np.zeros((3, 4), dtype=np.float32)                 # rows 0 and 1: uniform P = 1/4 each
    rows[2] = np.log(probs).astype(np.float32)
    toks = [0, 2, 3]                                          # anchor, candidates 2 and 3
    for u, want in ((0.05, 0), (0.15, 1), (0.29, 1), (0.31, 2), (0.59, 2), (0.61, 3), (0.95, 3)):
        r = _single(rows, toks, [0.2, 0.2], u)                # 0.2 < 1/4: both candidates pass
        assert r["accept_len"][0] == 2 and r["out_len"][0] == 3
        assert r["next_anchor"][0] == want, (u, r["next_anchor"][0])
        assert list(r["out_tokens"][0, :3]) == [2, 3, want]
    # the same uniforms after a rejection of candidate 3 at row 1 draw from row 1's P without token 3:
    # uniform over {0, 1, 2}, thirds
    for u, want in ((0.1, 0), (0.4, 1), (0.9, 2)):
        r = _single(rows, toks, [0.2, 0.3], u)                # 0.3 > 1/4: the second candidate is rejected
        assert r["accept_len"][0] == 1 and r["next_anchor"][0] == want, (u, r["next_anchor"][0])


def test_low_temperature_reduces_to_greedy():
    """As the temperature goes to 0 the policy puts all mass on the arg-max: sampling
    verification must then return exactly the greedy result, whatever the uniforms."""
    cfg = small_variant(CONFIGS["tiny"], vocab=1500)
    req = make_requests(cfg)
    alloc = OA.dvl_alloc(req["n_bs"], req["n_live"], req["scores"], req["draft_tokens"],
                         req["ctx_len"], req["block_table"])
    lp = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], req["n_live"],
                        8 * req["n_bs"]).numpy()
    greedy = OG.accept(lp, cfg.vocab, alloc["tokens"], alloc["k"], alloc["offset"], req["n_live"], req["n_bs"])
    rng = np.random.default_rng(3)
    for _ in range(3):
        s = OS.accept_sampling(lp, cfg.vocab, 1e-3, rng.uniform(0.001, 0.999, size=lp.shape[0]),
                               rng.uniform(0.001, 0.999, size=req["n_bs"]), alloc["tokens"], alloc["k"],
                               alloc["offset"], req["n_live"], req["n_bs"])
        for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
            np.testing.assert_array_equal(s[f], greedy[f], err_msg=f)
