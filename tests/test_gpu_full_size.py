"""Full-size GPU checks in the launch configuration bench.py times (one captured
graph: allocation -> attention -> acceptance), for the Qwen3-8B-shaped full step
(one of its 36 layers) and the skewed workload.  Allocation and acceptance are
compared in full with the oracle; attention is compared with the oracle on EVERY
live element (the oracle does a full-size layer in about a second), a few rows
are recomputed one by one from the definition in fp64, and the properties that
hold at any size are checked (finite rows, zero capacity rows).  The error
figures (max abs, max rel over |ref| > 1e-2, ||d||_2 / ||ref||_2) are printed.
"""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_logits_unpacked, make_q_unpacked,
                           make_requests, planted_expectation, rows_to_packed)
from gpu_case import (ALLOC_FIELDS, SCALE, StagedRequests, attn_close, attn_stats, oracle_accept, oracle_alloc,
                      oracle_attn)
from oracle import verify_attn as OV

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n_bs", [("qwen3_8b_step", 40), ("skew", 32), ("qwen3_8b_layer", 16)])
def test_full_size_step_in_one_graph(name, n_bs):
    import paper_2609_37532_b200 as P
    cfg = CONFIGS[name]
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req)
    n = req["n_live"]
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    st = StagedRequests(req)
    kc, vc = make_kv_layer(req, 0, device="cuda", poison=False)
    qp = rows_to_packed(make_q_unpacked(req, 0, device="cuda"), alloc["k"], alloc["offset"], n,
                        8 * n_bs).contiguous()
    lp = rows_to_packed(make_logits_unpacked(req, device="cuda"), alloc["k"], alloc["offset"], n,
                        8 * n_bs).contiguous()
    out = torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    o = dict(accept_len=torch.zeros(n_bs, dtype=torch.int32, device="cuda"),
             next_anchor=torch.zeros(n_bs, dtype=torch.int32, device="cuda"),
             out_tokens=torch.zeros((n_bs, 16), dtype=torch.int32, device="cuda"),
             out_len=torch.zeros(n_bs, dtype=torch.int32, device="cuda"))

    def step():
        P.alloc_verify(ws, st.n_live, st.scores, st.draft, st.ctx_len, st.block_table, req["num_pages"])
        P.verify_attn(ws, qp, kc, vc, st.block_table, SCALE, out)
        P.accept(ws, lp, cfg.vocab, o["accept_len"], o["next_anchor"], o["out_tokens"], o["out_len"], None)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
        torch.cuda.synchronize()
        out.fill_(float("nan"))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        graph.replay()
        graph.replay()                      # replays must be idempotent (tickets reset themselves)
    torch.cuda.synchronize()
    assert ws.status() == 0

    for f in ALLOC_FIELDS:
        np.testing.assert_array_equal(ws.field(f).cpu().numpy(), alloc[f], err_msg=f)

    got = out.float().cpu().numpy()
    m_live = 8 * n
    assert np.isfinite(got[:m_live]).all()
    assert (got[m_live:] == 0).all()
    # every live element against the oracle (fp32, dense masked softmax)
    kc_cpu, vc_cpu, qp_cpu = kc.cpu(), vc.cpu(), qp.cpu()
    ref = oracle_attn(req, alloc, kc_cpu, vc_cpu, qp_cpu)
    ok, max_abs, worst_at = attn_close(out, ref)
    st = attn_stats(got, ref)
    print(f"\n{name}: attention vs oracle on all {m_live * cfg.n_q_heads * 128} live elements: max abs {st['max_abs']:.2e}, "
          f"max rel (|ref| > 1e-2) {st['max_rel']:.2e}, ||d||/||ref|| {st['rel_l2']:.2e}, worst row {st['worst_row_rel_l2']:.2e}")
    assert ok, f"max|d|={max_abs} at {worst_at}"
    assert st["max_abs"] < 5e-3 and st["rel_l2"] < 4e-3
    # a few rows by the definition in fp64: first / last rows of the longest and shortest windows and contexts
    rng = np.random.default_rng(0)
    kc_h, vc_h, q_h = kc_cpu.float().numpy(), vc_cpu.float().numpy(), qp_cpu.float().numpy()
    G = cfg.n_q_heads // cfg.n_kv_heads
    picks = [(i, j) for i in (int(np.argmax(alloc["k"])), int(np.argmin(alloc["k"][:n])),
                              int(np.argmax(req["ctx_len"][:n])), int(np.argmin(req["ctx_len"][:n])))
             for j in (0, int(alloc["k"][i]) - 1)]
    for (i, j) in picks:
        h = int(rng.integers(0, cfg.n_q_heads))
        s = int(alloc["offset"][i]) + j
        ref64 = OV.verify_attn_row(q_h[s, h], kc_h, vc_h, req["block_table"][i],
                                   int(req["ctx_len"][i]) + j + 1, h // G, SCALE)
        err = np.abs(got[s, h] - ref64)
        assert (err <= np.maximum(1e-2, 1e-2 * np.abs(ref64))).all(), f"row ({i},{j}) head {h}: max|d|={err.max()}"
        assert np.linalg.norm(err) <= 8e-3 * np.linalg.norm(ref64) + 2e-4

    exp = oracle_accept(req, alloc, lp.cpu())
    for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
        np.testing.assert_array_equal(o[f].cpu().numpy(), exp[f], err_msg=f)
    truth = planted_expectation(req, alloc["k"])
    np.testing.assert_array_equal(o["accept_len"].cpu().numpy(), truth["accept_len"])
    np.testing.assert_array_equal(o["next_anchor"].cpu().numpy(), truth["next_anchor"])
