"""The whole verify-side decision chain in ONE captured CUDA graph, replayed on two different
steps at the same addresses:

    dscale_predict_scores -> dscale_alloc_verify (logits mode) -> dscale_verify_attn x L
    -> dscale_lm_head_accept

Each stage is compared with the oracle on the inputs it actually saw: the predictor's
predLogits within their tolerance; the allocation bit-exactly against the oracle run on the
device's own predLogits (an integer decision is only ever compared on identical scores);
attention within the bounds of gpu_case.attn_close; the LM-head tokens by the margin rule of
test_gpu_lm_head.py and the acceptance outputs against the sequential loop on those tokens."""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_predictor_inputs, make_q_unpacked, make_requests,
                           rows_to_packed, small_variant)
from gpu_case import ALLOC_FIELDS, SCALE, assert_alloc_equal, attn_close
from oracle import accept as OC
from oracle import dvl_alloc as OA
from oracle import lm_head as OL
from oracle import predictor as OP
from oracle import verify_attn as OV

pytestmark = pytest.mark.gpu

N_BS, LAYERS, HID_DRAFT, HID_TARGET = 8, 2, 128, 256


def test_decision_graph_replays_two_steps():
    import paper_2609_37532_b200 as P
    base = small_variant(CONFIGS["tiny"], vocab=4096, ctx_lo=30, ctx_hi=700)
    reqs = [make_requests(small_variant(base, n=n, seed=seed), n_bs=N_BS) for n, seed in ((8, 91), (5, 92))]
    cfg = reqs[0]["cfg"]
    V = cfg.vocab
    max_pages = max(r["max_pages"] for r in reqs)
    num_pages = max(r["num_pages"] for r in reqs)
    dev = "cuda"
    i32 = dict(dtype=torch.int32, device=dev)

    ws = P.VerifyWorkspace(N_BS, cfg.n_q_heads, cfg.n_kv_heads)
    t = dict(n_live=torch.ones(1, **i32), draft=torch.zeros((N_BS, 16), **i32), ctx_len=torch.zeros(N_BS, **i32),
             block_table=torch.zeros((N_BS, max_pages), **i32),
             draft_logits=torch.zeros((N_BS, 15, V), dtype=torch.float32, device=dev),
             draft_hidden=torch.zeros((N_BS, 15, HID_DRAFT), dtype=torch.bfloat16, device=dev),
             pred=torch.zeros((N_BS, 15), dtype=torch.float32, device=dev),
             kv=[(torch.zeros((num_pages, cfg.n_kv_heads, 16, 128), dtype=torch.bfloat16, device=dev),
                  torch.zeros((num_pages, cfg.n_kv_heads, 16, 128), dtype=torch.bfloat16, device=dev))
                 for _ in range(LAYERS)],
             q=[torch.zeros((8 * N_BS, cfg.n_q_heads, 128), dtype=torch.bfloat16, device=dev) for _ in range(LAYERS)],
             out=[torch.zeros((8 * N_BS, cfg.n_q_heads, 128), dtype=torch.bfloat16, device=dev) for _ in range(LAYERS)],
             hidden=torch.zeros((8 * N_BS, HID_TARGET), dtype=torch.bfloat16, device=dev),
             accept_len=torch.zeros(N_BS, **i32), next_anchor=torch.zeros(N_BS, **i32),
             out_tokens=torch.zeros((N_BS, 16), **i32), out_len=torch.zeros(N_BS, **i32))
    # fixed parameters of the step: predictor matrices and the LM head
    par = make_predictor_inputs(reqs[0], HID_DRAFT, device=dev)
    g = torch.Generator(device=dev).manual_seed(7)
    lm_w = torch.randn((V, HID_TARGET), generator=g, device=dev).to(torch.bfloat16)

    def step():
        P.predict_scores(ws, t["n_live"], t["draft_logits"], V, t["draft_hidden"], par["p_hidden"], par["p_logit"],
                         par["w1"], par["b1"], par["w2"], par["b2"], t["pred"])
        P.alloc_verify(ws, t["n_live"], t["pred"], t["draft"], t["ctx_len"], t["block_table"], num_pages,
                       scores_are_logits=True)
        for l in range(LAYERS):
            P.verify_attn(ws, t["q"][l], t["kv"][l][0], t["kv"][l][1], t["block_table"], SCALE, t["out"][l])
        P.lm_head_accept(ws, t["hidden"], lm_w, t["accept_len"], t["next_anchor"], t["out_tokens"], t["out_len"])

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                             # warm-up outside the capture (first-call queries)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()

    for r in reqs:
        n = r["n_live"]
        d = make_predictor_inputs(r, HID_DRAFT, device="cpu")
        bt = np.full((N_BS, max_pages), -1, dtype=np.int32)
        bt[:, : r["max_pages"]] = r["block_table"]
        t["n_live"].fill_(n)
        t["draft"].copy_(torch.as_tensor(r["draft_tokens"])); t["ctx_len"].copy_(torch.as_tensor(r["ctx_len"]))
        t["block_table"].copy_(torch.as_tensor(bt))
        t["draft_logits"].copy_(d["draft_logits"][:, :, :V]); t["draft_hidden"].copy_(d["draft_hidden"])
        kvs = []
        for l in range(LAYERS):
            k_cpu, v_cpu = make_kv_layer(r, l, poison=False)
            t["kv"][l][0].zero_(); t["kv"][l][1].zero_()
            t["kv"][l][0][: k_cpu.shape[0]].copy_(k_cpu); t["kv"][l][1][: v_cpu.shape[0]].copy_(v_cpu)
            kvs.append((k_cpu, v_cpu))
        # the upstream model's rows are laid out by the allocation of THIS step, which the graph
        # computes itself: write Q and the final hidden states for every slot of every request at
        # capacity and let the test pack them after a first replay has produced the allocation
        graph.replay(); torch.cuda.synchronize()
        assert ws.status() == 0
        alloc_dev = {f: ws.field(f).cpu().numpy().copy() for f in ALLOC_FIELDS}
        k_dev, off_dev = alloc_dev["k"], alloc_dev["offset"]
        qps = []
        for l in range(LAYERS):
            qp = rows_to_packed(make_q_unpacked(r, l), k_dev, off_dev, n, 8 * N_BS)
            t["q"][l].copy_(qp); qps.append(qp)
        gh = torch.Generator().manual_seed(1000 + r["cfg"].seed)
        hid = (torch.randn((8 * N_BS, HID_TARGET), generator=gh) * 0.3).to(torch.bfloat16)
        t["hidden"].copy_(hid)
        graph.replay(); torch.cuda.synchronize()
        assert ws.status() == 0

        # 1. predictor
        host = {key: (v.float().numpy() if torch.is_tensor(v) else v) for key, v in d.items()}
        exp = OP.predict(host["draft_logits"][:, :, :V], host["draft_hidden"], par["p_hidden"].float().cpu().numpy(),
                         par["p_logit"].float().cpu().numpy(), par["w1"].cpu().numpy(), par["b1"].cpu().numpy(),
                         par["w2"].cpu().numpy(), par["b2"].cpu().numpy(), n, N_BS)
        pred = t["pred"].cpu().numpy()
        np.testing.assert_allclose(pred[:n], exp["pred_logits"][:n], rtol=3e-3, atol=3e-3)
        # 2. allocation, on the device's own scores
        scores = np.zeros((N_BS, 15), dtype=np.float32); scores[:n] = pred[:n]
        want = OA.dvl_alloc(N_BS, n, scores, r["draft_tokens"], r["ctx_len"], bt, logits_mode=True)
        got = {f: ws.field(f).cpu().numpy() for f in ALLOC_FIELDS}
        assert_alloc_equal(got, want)
        assert_alloc_equal(got, alloc_dev)                 # the second replay allocated the same
        # 3. attention per layer
        for l in range(LAYERS):
            ref = OV.verify_attn(qps[l].float().numpy(), kvs[l][0].float().numpy(), kvs[l][1].float().numpy(),
                                 bt, r["ctx_len"], want["k"], want["offset"], n, cfg.n_q_heads, cfg.n_kv_heads, SCALE)
            ok, max_abs, worst = attn_close(t["out"][l], ref)
            assert ok, (l, max_abs, worst)
        # 4. LM head + acceptance
        ref = OL.lm_head_accept(hid.float().numpy(), lm_w.float().cpu().numpy(), want["tokens"], want["k"],
                                want["offset"], n, N_BS)
        m_live = int(want["offset"][n])
        top1 = ws.field("top1").cpu().numpy()
        logits = ref["logits"]
        mx = logits[:m_live].max(axis=1)
        assert (logits[np.arange(m_live), top1[:m_live]] >= mx - 1e-3 * (1 + np.abs(mx))).all()
        own = OC.accept_prefix(top1, want["tokens"], want["k"], want["offset"], n, N_BS)
        for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
            np.testing.assert_array_equal(t[f].cpu().numpy(), own[f], err_msg=f)
