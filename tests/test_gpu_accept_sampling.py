"""dscale_accept_sampling against the fp64 oracle.  Accept lengths are compared exactly on
uniforms kept away from the acceptance thresholds; a drawn successor is valid iff the
request's uniform lies in that token's interval of the oracle's cumulative distribution
(within 2e-5), which allows the neighbouring token exactly at a rounding boundary."""
import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, make_logits_unpacked, make_requests, rows_to_packed, small_variant
from gpu_case import StagedRequests, gpu_alloc, oracle_alloc
from oracle import accept_sampling as OS

pytestmark = pytest.mark.gpu


def _case(P, cfg, n_bs, temperature, seed):
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req)
    n = req["n_live"]
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    gpu_alloc(P, ws, StagedRequests(req))
    lp = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], n, 8 * n_bs)
    rng = np.random.default_rng(seed)
    u_acc = rng.uniform(0, 1, size=8 * n_bs)
    u_draw = rng.uniform(0, 1, size=n_bs)
    # keep the acceptance uniforms away from the thresholds (fp32 vs fp64 decisions)
    probe = OS.accept_sampling(lp.numpy(), cfg.vocab, temperature, np.zeros(8 * n_bs), u_draw,
                               alloc["tokens"], alloc["k"], alloc["offset"], n, n_bs)   # u = 0: every P(x)
    p = probe["p_draft"]
    close = np.abs(u_acc - p) < 1e-3 * np.maximum(p, 1e-3)
    u_acc[close] = np.where(np.arange(8 * n_bs)[close] % 2 == 0, p[close] * 0.5, p[close] + (1 - p[close]) * 0.5)
    u_acc = u_acc.astype(np.float32).astype(np.float64)
    u_draw = u_draw.astype(np.float32).astype(np.float64)
    exp = OS.accept_sampling(lp.numpy(), cfg.vocab, temperature, u_acc, u_draw, alloc["tokens"],
                             alloc["k"], alloc["offset"], n, n_bs)
    o = [torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs, 16), -9, dtype=torch.int32, device="cuda"),
         torch.full((n_bs,), -9, dtype=torch.int32, device="cuda")]
    pd = torch.zeros(8 * n_bs, dtype=torch.float32, device="cuda")
    ld = (cfg.vocab + 3) // 4 * 4                        # rows padded to a multiple of 4 floats
    lp_dev = torch.full((8 * n_bs, ld), float("nan"), dtype=torch.float32, device="cuda")
    lp_dev[:, :cfg.vocab] = lp.cuda()
    for _ in range(2):                                   # twice: the ticket resets itself
        P.accept_sampling(ws, lp_dev, cfg.vocab, temperature, torch.as_tensor(u_acc, dtype=torch.float32).cuda(),
                          torch.as_tensor(u_draw, dtype=torch.float32).cuda(), o[0], o[1], o[2], o[3], pd)
        torch.cuda.synchronize()
    acc, nxt, toks, ln = (t.cpu().numpy() for t in o)
    np.testing.assert_array_equal(acc, exp["accept_len"])
    np.testing.assert_array_equal(ln, exp["out_len"])
    has = exp["p_draft"] > 0
    np.testing.assert_allclose(pd.cpu().numpy()[has], exp["p_draft"][has], rtol=2e-4, atol=1e-9)
    n_same = 0
    for i in range(n):
        a, ki, oi = int(acc[i]), int(alloc["k"][i]), int(alloc["offset"][i])
        np.testing.assert_array_equal(toks[i, :a], alloc["tokens"][oi + 1: oi + 1 + a])
        assert toks[i, a] == nxt[i] and (toks[i, a + 1:] == -1).all()
        w = OS.row_distribution(lp.numpy()[oi + a, :cfg.vocab], temperature)
        if a < ki - 1:
            w[int(alloc["tokens"][oi + a + 1])] = 0.0
            assert nxt[i] != alloc["tokens"][oi + a + 1]          # the rejected candidate never comes back
        lo, hi = OS.draw_interval(w, int(nxt[i]))
        assert w[nxt[i]] > 0 and lo - 2e-5 <= u_draw[i] < hi + 2e-5, (i, nxt[i], lo, hi, u_draw[i])
        n_same += int(nxt[i] == exp["next_anchor"][i])
    assert n_same >= n - 1                                         # boundary ties are rare
    assert (acc[n:] == 0).all() and (nxt[n:] == -1).all() and (ln[n:] == 0).all()
    return exp


def test_sampling_small_vocab_mixed_outcomes():
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=1024, n=16, seed=51)
    exp = _case(P, cfg, 20, 1.0, 1)
    a = exp["accept_len"][:16]
    assert a.max() >= 2 and a.min() == 0                           # both outcomes occur


@pytest.mark.parametrize("temperature", [1.0, 0.5])
def test_sampling_full_vocab(temperature):
    import paper_2609_37532_b200 as P
    _case(P, CONFIGS["qwen3_4b_layer"], 8, temperature, 2)
    _case(P, small_variant(CONFIGS["tiny"], vocab=70001), 4, temperature, 3)
