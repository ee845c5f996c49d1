"""dscale_verify_step_host: the whole step from pinned host buffers, against the oracle."""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_logits_unpacked, make_q_unpacked,
                           make_requests, planted_expectation, rows_to_packed, small_variant)
from gpu_case import SCALE, attn_close, oracle_accept, oracle_alloc, oracle_attn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_layers", [1, 3])
def test_host_step_matches_oracle(n_layers):
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=5000, n=6, seed=31, ctx_lo=10, ctx_hi=700)
    req = make_requests(cfg, n_bs=8)
    n_bs, n = req["n_bs"], req["n_live"]
    alloc = oracle_alloc(req)
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    layers, cpu_layers = [], []
    for l in range(n_layers):
        kc, vc = make_kv_layer(req, l)
        qp = rows_to_packed(make_q_unpacked(req, l), alloc["k"], alloc["offset"], n, 8 * n_bs)
        cpu_layers.append((kc, vc, qp))
        layers.append((qp.cuda().contiguous(), kc.cuda(), vc.cuda(),
                       torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")))
    lp = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], n, 8 * n_bs)
    hs = P.HostStep(ws, req["max_pages"], req["num_pages"], layers, lp.cuda().contiguous(), cfg.vocab, SCALE)
    hs.h_n_live[0] = n
    hs.h_scores.copy_(torch.as_tensor(req["scores"]))
    hs.h_draft.copy_(torch.as_tensor(req["draft_tokens"]))
    hs.h_ctx_len.copy_(torch.as_tensor(req["ctx_len"]))
    hs.h_block_table.copy_(torch.as_tensor(req["block_table"]))
    for _ in range(2):                                 # twice: the step must be repeatable
        hs.run()
        torch.cuda.synchronize()
    assert ws.status() == 0
    exp = oracle_accept(req, alloc, lp)
    np.testing.assert_array_equal(hs.h_accept_len.numpy(), exp["accept_len"])
    np.testing.assert_array_equal(hs.h_next_anchor.numpy(), exp["next_anchor"])
    np.testing.assert_array_equal(hs.h_out_tokens.numpy(), exp["out_tokens"])
    np.testing.assert_array_equal(hs.h_out_len.numpy(), exp["out_len"])
    truth = planted_expectation(req, alloc["k"])
    np.testing.assert_array_equal(hs.h_accept_len.numpy(), truth["accept_len"])
    for (kc, vc, qp), (_, _, _, out) in zip(cpu_layers, layers):
        ok, max_abs, worst = attn_close(out, oracle_attn(req, alloc, kc, vc, qp))
        assert ok, f"max|d|={max_abs} at {worst}"
    assert hs.h2d_bytes == 4 + n_bs * (15 + 16 + 1 + req["max_pages"]) * 4
