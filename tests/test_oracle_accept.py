"""Pins for oracle/accept.py and for the input generators (CPU only)."""
import numpy as np
import pytest

from conftest import read_golden
from dscale_inputs import (CONFIGS, make_logits_unpacked, make_requests, planted_expectation,
                           rows_to_packed, small_variant)
from oracle import accept as OC
from oracle import dvl_alloc as OA


def _planted_case(cfg):
    req = make_requests(cfg)
    alloc = OA.dvl_alloc(req["n_bs"], req["n_live"], req["scores"], req["draft_tokens"],
                         req["ctx_len"], req["block_table"])
    lu = make_logits_unpacked(req)
    lp = rows_to_packed(lu, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"]).numpy()
    return req, alloc, lp


@pytest.mark.parametrize("name,n", [("tiny", 4), ("qwen3_4b_layer", 8)])
def test_acceptance_recovers_planted_truth(name, n):
    cfg = CONFIGS[name]
    if cfg.vocab > 4096:
        cfg = small_variant(cfg, vocab=4099)
    req, alloc, lp = _planted_case(cfg)
    res = OC.accept(lp, cfg.vocab, alloc["tokens"], alloc["k"], alloc["offset"],
                    req["n_live"], req["n_bs"], ctx_len=req["ctx_len"])
    exp = planted_expectation(req, alloc["k"])
    np.testing.assert_array_equal(res["accept_len"], exp["accept_len"])
    np.testing.assert_array_equal(res["next_anchor"], exp["next_anchor"])
    np.testing.assert_array_equal(res["out_len"][:n], exp["accept_len"][:n] + 1)
    for i in range(n):
        a = res["accept_len"][i]
        np.testing.assert_array_equal(res["out_tokens"][i, :a], req["draft_tokens"][i, 1:a + 1])
        assert res["out_tokens"][i, a] == res["next_anchor"][i]
        assert (res["out_tokens"][i, a + 1:] == -1).all()
        assert res["ctx_len"][i] == req["ctx_len"][i] + a + 1
    # whole-step figure of merit: verified tokens = sum (a + 1)
    assert res["out_len"].sum() == (exp["accept_len"][:n] + 1).sum()


def test_argmax_first_index_on_ties_and_nan():
    x = np.zeros((4, 8), dtype=np.float32)
    x[0] = [1, 5, 5, 2, 5, 0, 0, 0]          # tie -> first maximum
    x[1] = [np.nan, 1, 3, np.nan, 3, 0, 0, 0]  # NaN never wins
    x[2] = np.nan                             # all-NaN row -> 0
    x[3] = -np.inf                            # all -inf -> 0
    x[3, 6] = -1e30
    t = OC.row_argmax(x, 4, 8)
    assert list(t) == [1, 2, 0, 6]
    # vocab limit respected when ld > vocab
    y = np.zeros((1, 8), dtype=np.float32)
    y[0, 7] = 9
    assert OC.row_argmax(y, 1, 7)[0] == 0


def _manual(tokens_per_req, top1_per_req):
    k = [len(t) for t in tokens_per_req]
    off = OA.offsets_of(k)
    n = len(k)
    tokens = np.concatenate(tokens_per_req).astype(np.int32)
    top1 = np.concatenate(top1_per_req).astype(np.int32)
    return OC.accept_prefix(top1, tokens, k, off, n, n)


def test_hand_cases():
    r = _manual(
        [[10, 11, 12, 13],      # all three candidates accepted -> a=3, successor from last row
         [20],                  # k=1: a=0, successor from the anchor row
         [30, 31, 32],          # mismatch at row 0 -> a=0
         [40, 41, 42, 43, 44]], # accepted 41,42 then rejection; later match must not count
        [[11, 12, 13, 99],
         [77],
         [5, 32, 6],
         [41, 42, 7, 44, 8]])
    assert list(r["accept_len"]) == [3, 0, 0, 2]
    assert list(r["next_anchor"]) == [99, 77, 5, 7]
    assert list(r["out_len"]) == [4, 1, 1, 3]
    assert list(r["out_tokens"][0][:5]) == [11, 12, 13, 99, -1]
    assert list(r["out_tokens"][3][:4]) == [41, 42, 7, -1]


def test_sentinels_get_neutral_outputs():
    k = [2, 0, 0]
    off = [0, 2, 2, 2]
    r = OC.accept_prefix(np.array([5, 6, 0, 0]), np.array([1, 5, 0, 0]), k, off, 1, 3)
    assert list(r["accept_len"]) == [1, 0, 0]
    assert list(r["next_anchor"]) == [6, -1, -1]
    assert list(r["out_len"]) == [2, 0, 0]
    assert (r["out_tokens"][1:] == -1).all()


def test_tile_padding_numbers_of_the_paper():
    g = read_golden("eq2_tile_padding.txt")
    rows = lambda ell, B: B * -(-ell // B)
    ell = g["ell"][0]
    assert rows(ell, 128) == g["rows_128"][0] and rows(ell, 128) - ell == g["masked_128"][0]
    assert 1 - ell / rows(ell, 128) == g["padding_128"][0]
    assert rows(ell, 16) == g["rows_16"][0] and 1 - ell / rows(ell, 16) == g["padding_16"][0]


def test_generators_are_seeded_and_shaped():
    for name, cfg in CONFIGS.items():
        if cfg.ctx_hi > 4096:
            cfg = small_variant(cfg, ctx_lo=cfg.ctx_lo // 16, ctx_hi=cfg.ctx_hi // 16)
        a, b = make_requests(cfg), make_requests(cfg)
        for key in ("scores", "draft_tokens", "ctx_len", "block_table", "planted_a"):
            np.testing.assert_array_equal(a[key], b[key])
        n = cfg.n
        assert (a["ctx_len"][:n] >= cfg.ctx_lo).all() and (a["ctx_len"][:n] <= cfg.ctx_hi).all()
        used = a["block_table"][a["block_table"] >= 0]
        assert len(np.unique(used)) == len(used) and used.max() < a["num_pages"]
        assert (a["planted_a"] >= 0).all() and (a["planted_a"] <= 15).all()
        assert (np.diff(a["scores"][:n], axis=1) <= 0).all()
        assert a["max_pages"] % 4 == 0
