"""dscale_verify_step_host: the whole step from pinned host buffers, against the oracle."""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_logits_unpacked, make_q_unpacked,
                           make_requests, planted_expectation, rows_to_packed, small_variant)
from gpu_case import SCALE, attn_close, oracle_accept, oracle_alloc, oracle_attn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_layers,pinned", [(1, True), (3, True), (2, False)])
def test_host_step_matches_oracle(n_layers, pinned):
    """pinned: the staged inputs and the results travel through the buffers' device mapping (one
    small kernel each way); pageable: through ordinary copies."""
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
    hs = P.HostStep(ws, req["max_pages"], req["num_pages"], layers, lp.cuda().contiguous(), cfg.vocab, SCALE,
                    pinned=pinned)
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


def test_host_step_as_one_replayed_graph():
    """dscale_verify_step_host_graph: the first call captures, the following calls replay the same
    graph on whatever the fixed-address buffers hold; two different steps against the oracle."""
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=3000, n=7, seed=33, ctx_lo=10, ctx_hi=600)
    req = make_requests(cfg, n_bs=8)
    n_bs, n, n_layers = req["n_bs"], req["n_live"], 2
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    kvs = [make_kv_layer(req, l) for l in range(n_layers)]
    layers = [(torch.zeros((8 * n_bs, cfg.n_q_heads, 128), dtype=torch.bfloat16, device="cuda"),
               kc.cuda(), vc.cuda(),
               torch.zeros((8 * n_bs, cfg.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")) for kc, vc in kvs]
    logits = torch.zeros((8 * n_bs, cfg.vocab), dtype=torch.float32, device="cuda")
    hs = P.HostStep(ws, req["max_pages"], req["num_pages"], layers, logits, cfg.vocab, SCALE)
    hs.h_n_live[0] = n
    hs.h_draft.copy_(torch.as_tensor(req["draft_tokens"]))
    hs.h_ctx_len.copy_(torch.as_tensor(req["ctx_len"]))
    hs.h_block_table.copy_(torch.as_tensor(req["block_table"]))
    side = torch.cuda.Stream()
    rng = np.random.default_rng(5)
    for step in range(3):
        r = dict(req)
        if step:                                          # other scores: other lengths, same addresses
            r["scores"] = req["scores"][rng.permutation(n_bs)].copy()
            r["scores"][n:] = 0
        alloc = oracle_alloc(r)
        hs.h_scores.copy_(torch.as_tensor(r["scores"]))
        qps = []
        for l in range(n_layers):
            qp = rows_to_packed(make_q_unpacked(r, l), alloc["k"], alloc["offset"], n, 8 * n_bs)
            layers[l][0].copy_(qp); layers[l][3].fill_(float("nan")); qps.append(qp)
        lp = rows_to_packed(make_logits_unpacked(r), alloc["k"], alloc["offset"], n, 8 * n_bs)
        logits.copy_(lp)
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            hs.run(graph=True)
        side.synchronize()
        assert ws.status() == 0
        exp = oracle_accept(r, alloc, lp)
        np.testing.assert_array_equal(hs.h_accept_len.numpy(), exp["accept_len"])
        np.testing.assert_array_equal(hs.h_next_anchor.numpy(), exp["next_anchor"])
        np.testing.assert_array_equal(hs.h_out_tokens.numpy(), exp["out_tokens"])
        np.testing.assert_array_equal(hs.h_out_len.numpy(), exp["out_len"])
        for l in range(n_layers):
            ok, max_abs, worst = attn_close(layers[l][3], oracle_attn(r, alloc, kvs[l][0], kvs[l][1], qps[l]))
            assert ok, f"step {step} layer {l}: max|d|={max_abs} at {worst}"
