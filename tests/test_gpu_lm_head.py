"""dscale_lm_head_accept against the binary64 LM-head oracle.

The kernel accumulates bf16 products in fp32 on the tensor cores, so a packed row's
token may differ from the oracle's only where two oracle logits are closer than the
fp32 rounding of a dot product; the test accepts the kernel's token iff its oracle
logit is within 1e-3 (1 + |max|) of the row maximum, requires exact agreement on
every planted row (margin of several units), and requires the acceptance outputs to
be the sequential loop applied to the kernel's own tokens."""
import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, make_lm_head_unpacked, make_requests, rows_to_packed, small_variant
from gpu_case import StagedRequests, gpu_alloc, oracle_alloc
from oracle import accept as OC
from oracle import lm_head as OL

pytestmark = pytest.mark.gpu


def _case(P, cfg, n_bs, hidden_dim, gen_device="cpu"):
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req)
    n = req["n_live"]
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    gpu_alloc(P, ws, StagedRequests(req))
    weight, hid_unpacked = make_lm_head_unpacked(req, hidden_dim, device=gen_device)
    hidden = rows_to_packed(hid_unpacked, alloc["k"], alloc["offset"], n, 8 * n_bs)
    exp = OL.lm_head_accept(hidden.float().cpu().numpy(), weight.float().cpu().numpy(), alloc["tokens"],
                            alloc["k"], alloc["offset"], n, n_bs)
    m_live = int(alloc["offset"][n])
    o = [torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs, 16), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs,), -9, dtype=torch.int32, device="cuda")]
    ctx = torch.as_tensor(req["ctx_len"]).cuda()
    row_max = torch.zeros(8 * n_bs, dtype=torch.float32, device="cuda")
    hd, wd = hidden.cuda().contiguous(), weight.cuda().contiguous()
    for rep in range(2):                                  # twice: the ticket resets itself
        ctx.copy_(torch.as_tensor(req["ctx_len"]))
        P.lm_head_accept(ws, hd, wd, o[0], o[1], o[2], o[3], ctx, row_max)
        torch.cuda.synchronize()
        assert int(ws.field("status")[0]) == 0
        top1 = ws.field("top1").cpu().numpy()[:8 * n_bs]
        logits = exp["logits"]
        mx = logits[:m_live].max(axis=1)
        got_logit = logits[np.arange(m_live), top1[:m_live]]
        assert (got_logit >= mx - 1e-3 * (1 + np.abs(mx))).all(), \
            np.argwhere(got_logit < mx - 1e-3 * (1 + np.abs(mx)))[:4]
        np.testing.assert_allclose(row_max.cpu().numpy()[:m_live], got_logit, rtol=2e-3, atol=2e-3)
        margin = mx - np.partition(logits[:m_live], -2, axis=1)[:, -2]
        clear = margin > 1e-2
        np.testing.assert_array_equal(top1[:m_live][clear], exp["top1"][:m_live][clear])
        assert (top1[m_live:] == 0).all()
        own = OC.accept_prefix(top1, alloc["tokens"], alloc["k"], alloc["offset"], n, n_bs,
                               ctx_len=req["ctx_len"])
        acc, nxt, toks, ln = (t.cpu().numpy() for t in o)
        np.testing.assert_array_equal(acc, own["accept_len"])
        np.testing.assert_array_equal(nxt, own["next_anchor"])
        np.testing.assert_array_equal(toks, own["out_tokens"])
        np.testing.assert_array_equal(ln, own["out_len"])
        np.testing.assert_array_equal(ctx.cpu().numpy(), own["ctx_len"])
        # the planted acceptance survives: a_i = min(planted a_i, k_i - 1)
        want = np.minimum(req["planted_a"][:n], alloc["k"][:n] - 1)
        np.testing.assert_array_equal(acc[:n], want)
    return exp, clear


@pytest.mark.parametrize("n_bs,n,vocab,hidden_dim", [
    (4, 4, 1024, 256),        # 32 rows: one short row tile, 7 vocabulary columns per CTA
    (20, 16, 4099, 512),      # dead tail rows, vocabulary not a multiple of 16
    (40, 40, 50000, 320),     # 320 rows: three row tiles, several column tiles per CTA
    (64, 61, 2000, 64),       # largest n_bs: four row tiles, a single k step
])
def test_lm_head_small_shapes(n_bs, n, vocab, hidden_dim):
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=vocab, n=n, seed=61 + n_bs)
    _case(P, cfg, n_bs, hidden_dim)


def test_lm_head_ties_take_the_lowest_index():
    """Duplicate weight rows give bit-identical logits in any accumulation order."""
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=3000, n=8, seed=67)
    n_bs = 8
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req)
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    gpu_alloc(P, ws, StagedRequests(req))
    g = torch.Generator().manual_seed(5)
    weight = torch.randn((cfg.vocab, 128), generator=g).to(torch.bfloat16)
    hidden = torch.zeros((8 * n_bs, 128), dtype=torch.bfloat16)
    m_live = int(alloc["offset"][req["n_live"]])
    lo = np.array([(37 * s + 5) % 1400 for s in range(m_live)])
    hi = lo + 1500                                        # lands in another CTA's columns
    for s in range(m_live):
        w = weight[lo[s]].float()
        hidden[s] = (8.0 * w / float(w @ w)).to(torch.bfloat16)
        weight[hi[s]] = weight[lo[s]]
    o = [torch.zeros(n_bs, dtype=torch.int32, device="cuda"), torch.zeros(n_bs, dtype=torch.int32, device="cuda"),
         torch.zeros((n_bs, 16), dtype=torch.int32, device="cuda"), torch.zeros(n_bs, dtype=torch.int32, device="cuda")]
    P.lm_head_accept(ws, hidden.cuda(), weight.cuda(), *o)
    torch.cuda.synchronize()
    top1 = ws.field("top1").cpu().numpy()
    np.testing.assert_array_equal(top1[:m_live], lo)
    exp = OL.lm_head_accept(hidden.float().numpy(), weight.float().numpy(), alloc["tokens"], alloc["k"],
                            alloc["offset"], req["n_live"], n_bs)
    np.testing.assert_array_equal(exp["top1"][:m_live], lo)


def test_lm_head_full_size_qwen3_8b():
    """B = 32 at the 8B head: 256 packed rows, vocabulary 151936, hidden size 4096."""
    import paper_2609_37532_b200 as P
    cfg = CONFIGS["qwen3_8b_step"]
    exp, clear = _case(P, cfg, cfg.n, 4096, gen_device="cuda")
    assert clear.sum() >= 0.9 * clear.size


def test_lm_head_rejects_bad_shapes():
    import paper_2609_37532_b200 as P
    ws = P.VerifyWorkspace(4, 32, 8)
    o = [torch.zeros(4, dtype=torch.int32, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda"),
         torch.zeros((4, 16), dtype=torch.int32, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda")]
    h = torch.zeros((32, 96), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((100, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(RuntimeError):
        P.lm_head_accept(ws, h, w, *o)                    # hidden size not a multiple of 64
