"""Pins for oracle/verify_attn.py (CPU only)."""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_q_unpacked, make_requests,
                           rows_to_packed, small_variant)
from oracle import dvl_alloc as OA
from oracle import verify_attn as OV

SCALE = 1.0 / np.sqrt(128.0)


def _case(cfg=None, poison=True, valid_extra=16):
    cfg = cfg or CONFIGS["tiny"]
    req = make_requests(cfg)
    alloc = OA.dvl_alloc(req["n_bs"], req["n_live"], req["scores"], req["draft_tokens"],
                         req["ctx_len"], req["block_table"])
    kc, vc = make_kv_layer(req, 0, poison=poison, valid_extra=valid_extra)
    qu = make_q_unpacked(req, 0)
    qp = rows_to_packed(qu, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"])
    return req, alloc, kc.float().numpy(), vc.float().numpy(), qu.float().numpy(), qp.float().numpy()


def _run(req, alloc, kc, vc, qp, dtype=np.float32, ctx_len=None, block_table=None):
    cfg = req["cfg"]
    return OV.verify_attn(qp, kc, vc, req["block_table"] if block_table is None else block_table,
                          req["ctx_len"] if ctx_len is None else ctx_len,
                          alloc["k"], alloc["offset"], req["n_live"],
                          cfg.n_q_heads, cfg.n_kv_heads, SCALE, dtype=dtype)


def test_single_row_is_textbook_decode_attention():
    """k_i = 1: one query against ctx+1 keys; checked against torch SDPA on the
    gathered dense K/V (a library routine, not this file's formula)."""
    cfg = small_variant(CONFIGS["tiny"], n=1)
    req = make_requests(cfg)
    kc, vc = make_kv_layer(req, 0)
    qu = make_q_unpacked(req, 0)
    k = np.array([1], dtype=np.int32)
    off = np.array([0, 1], dtype=np.int32)
    qp = rows_to_packed(qu, k, off, 1, 8).float().numpy()
    out = OV.verify_attn(qp, kc.float().numpy(), vc.float().numpy(), req["block_table"],
                         req["ctx_len"], k, off, 1, cfg.n_q_heads, cfg.n_kv_heads, SCALE,
                         dtype=np.float64)
    ctx = int(req["ctx_len"][0])
    n_keys = ctx + 1
    pages = torch.as_tensor(req["block_table"][0, : (n_keys + 15) // 16], dtype=torch.long)
    for h in range(cfg.n_q_heads):
        g = h // (cfg.n_q_heads // cfg.n_kv_heads)
        Kd = kc[pages, g].reshape(-1, 128)[:n_keys].double()
        Vd = vc[pages, g].reshape(-1, 128)[:n_keys].double()
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(qp[0, h]).double()[None, None, :], Kd[None], Vd[None])
        np.testing.assert_allclose(out[0, h], ref[0, 0].numpy(), rtol=1e-9, atol=1e-12)
    assert np.all(out[1:] == 0)


def test_packed_agrees_with_unpacked_w16_on_live_rows():
    req, alloc, kc, vc, qu, qp = _case()
    cfg = req["cfg"]
    packed = _run(req, alloc, kc, vc, qp, dtype=np.float64)
    padded = OV.verify_attn_padded(qu, kc, vc, req["block_table"], req["ctx_len"], req["n_live"],
                                   cfg.n_q_heads, cfg.n_kv_heads, SCALE, dtype=np.float64)
    for i in range(req["n_live"]):
        ki, oi = alloc["k"][i], alloc["offset"][i]
        np.testing.assert_allclose(packed[oi:oi + ki], padded[i, :ki], rtol=1e-10, atol=1e-12)
    assert np.isfinite(packed).all()


def test_fp32_and_fp64_agree():
    req, alloc, kc, vc, qu, qp = _case()
    a = _run(req, alloc, kc, vc, qp, dtype=np.float32)
    b = _run(req, alloc, kc, vc, qp, dtype=np.float64)
    assert np.abs(a - b).max() <= 1e-5


def test_never_reads_past_the_visible_keys():
    """Slots at logical positions >= ctx_i + k_i are NaN: the packed result
    must stay finite and equal the run where they hold ordinary data."""
    req, alloc, kc, vc, qu, qp = _case()
    ref = _run(req, alloc, kc, vc, qp)
    kc2, vc2 = kc.copy(), vc.copy()
    for i in range(req["n_live"]):
        first_hidden = int(req["ctx_len"][i]) + int(alloc["k"][i])
        for t in range(first_hidden, int(req["ctx_len"][i]) + 16):
            pg = req["block_table"][i, t // 16]
            kc2[pg, :, t % 16, :] = np.nan
            vc2[pg, :, t % 16, :] = np.nan
    out = _run(req, alloc, kc2, vc2, qp)
    assert np.isfinite(out).all()
    np.testing.assert_array_equal(out, ref)


def test_constant_v_gives_constant_output():
    req, alloc, kc, vc, qu, qp = _case(poison=False)
    vc[:] = 0.625
    out = _run(req, alloc, kc, vc, qp, dtype=np.float64)
    m_live = 8 * req["n_live"]
    np.testing.assert_allclose(out[:m_live], 0.625, rtol=1e-12)
    assert np.all(out[m_live:] == 0)


def test_future_keys_do_not_matter():
    """Row j must not change when keys/values after ctx_i + j change."""
    req, alloc, kc, vc, qu, qp = _case(poison=False)
    ref = _run(req, alloc, kc, vc, qp)
    i = int(np.argmax(alloc["k"]))
    ki, oi, ci = int(alloc["k"][i]), int(alloc["offset"][i]), int(req["ctx_len"][i])
    assert ki >= 3
    j = 1
    kc2, vc2 = kc.copy(), vc.copy()
    for t in range(ci + j + 1, ci + ki):
        pg = req["block_table"][i, t // 16]
        kc2[pg, :, t % 16, :] += 3.0
        vc2[pg, :, t % 16, :] -= 5.0
    out = _run(req, alloc, kc2, vc2, qp)
    np.testing.assert_array_equal(out[oi:oi + j + 1], ref[oi:oi + j + 1])       # rows 0..j untouched
    assert np.abs(out[oi + j + 1:oi + ki] - ref[oi + j + 1:oi + ki]).max() > 1e-3  # later rows see it


def test_page_permutation_invariance():
    req, alloc, kc, vc, qu, qp = _case(poison=False)
    ref = _run(req, alloc, kc, vc, qp)
    rng = np.random.default_rng(5)
    perm = rng.permutation(req["num_pages"])              # new physical home of page p
    kc2 = np.empty_like(kc); vc2 = np.empty_like(vc)
    kc2[perm] = kc; vc2[perm] = vc
    bt2 = req["block_table"].copy()
    valid = bt2 >= 0
    bt2[valid] = perm[bt2[valid]]
    out = _run(req, alloc, kc2, vc2, qp, block_table=bt2)
    np.testing.assert_array_equal(out, ref)


def test_same_query_in_a_gqa_group_gives_same_output():
    req, alloc, kc, vc, qu, qp = _case()
    G = req["cfg"].n_q_heads // req["cfg"].n_kv_heads
    qp[:, 1] = qp[:, 0]                    # heads 0 and 1 share kv-head 0
    qp[:, G] = qp[:, 0]                    # head G uses kv-head 1
    out = _run(req, alloc, kc, vc, qp)
    m_live = 8 * req["n_live"]
    np.testing.assert_array_equal(out[:m_live, 1], out[:m_live, 0])
    assert np.abs(out[:m_live, G] - out[:m_live, 0]).max() > 1e-3


@pytest.mark.parametrize("where", ["first", "last_visible", "first_hidden", "page_edge_lo",
                                   "page_edge_hi"])
def test_needle_key(where):
    """One key carries a huge dot product with the query of row j of request i.
    If it is visible the output row is that key's value row; if it is the first
    hidden key nothing changes.  An off-by-one in the mask fails by O(1)."""
    req, alloc, kc, vc, qu, qp = _case(poison=False)
    i = int(np.argmax(alloc["k"]))
    ki, oi, ci = int(alloc["k"][i]), int(alloc["offset"][i]), int(req["ctx_len"][i])
    j = min(2, ki - 2)
    assert ki - 1 > j >= 0
    t = {"first": 0, "last_visible": ci + j, "first_hidden": ci + j + 1,
         "page_edge_lo": (ci // 16) * 16 - 1, "page_edge_hi": (ci // 16) * 16}[where]
    h, g = 5, 5 // (req["cfg"].n_q_heads // req["cfg"].n_kv_heads)
    ref = _run(req, alloc, kc, vc, qp)
    pg = req["block_table"][i, t // 16]
    qrow = qp[oi + j, h]
    kc[pg, g, t % 16, :] = qrow * 8.0                     # score ~ 8 |q|^2 / sqrt(128) ~ 90
    vc[pg, g, t % 16, :] = np.linspace(-2, 2, 128)
    out = _run(req, alloc, kc, vc, qp)
    if where == "first_hidden":
        np.testing.assert_array_equal(out[oi + j, h], ref[oi + j, h])
    else:
        np.testing.assert_allclose(out[oi + j, h], np.linspace(-2, 2, 128), atol=1e-4)


def test_single_row_helper_matches_full_oracle():
    req, alloc, kc, vc, qu, qp = _case()
    full = _run(req, alloc, kc, vc, qp, dtype=np.float64)
    i = 2
    oi, ci = int(alloc["offset"][i]), int(req["ctx_len"][i])
    j = int(alloc["k"][i]) - 1
    row = OV.verify_attn_row(qp[oi + j, 3], kc, vc, req["block_table"][i], ci + j + 1, 0, SCALE)
    np.testing.assert_allclose(row, full[oi + j, 3], rtol=1e-10, atol=1e-12)
