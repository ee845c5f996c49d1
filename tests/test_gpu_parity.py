"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle,
element by element, on the same seeded inputs.  Integer results must be
bit-exact; bf16 attention outputs must satisfy |gpu - ref| <= max(1e-2, 1e-2 |ref|)
per element and, per (row, q-head) vector, |gpu - ref|_2 <= 8e-3 |ref|_2 + 2e-4
(gpu_case.attn_close).
"""
import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_logits_unpacked, make_requests, planted_expectation,
                           rows_to_packed, small_variant)
from gpu_case import (ALLOC_FIELDS, SCALE, StagedRequests, assert_alloc_equal, attn_close, dev,
                      full_case, gpu_accept, gpu_alloc, oracle_accept, oracle_alloc, oracle_attn,
                      poison_hidden_slots)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_2609_37532_b200 as pkg
    assert torch.cuda.is_available()
    return pkg


def _ws(P, req):
    cfg = req["cfg"]
    return P.VerifyWorkspace(req["n_bs"], cfg.n_q_heads, cfg.n_kv_heads)


# ------------------------------------------------------------------ allocation
@pytest.mark.parametrize("name", list(CONFIGS))
def test_alloc_matches_oracle_on_the_named_workloads(P, name):
    cfg = CONFIGS[name]
    for n_bs in (cfg.n, min(64, cfg.n + 5)):
        req = make_requests(cfg, n_bs=n_bs)
        ws = _ws(P, req)
        got = gpu_alloc(P, ws, StagedRequests(req))
        assert_alloc_equal(got, oracle_alloc(req))
        assert ws.status() == 0
        assert got["k"][:cfg.n].sum() == 8 * cfg.n


def _random_req(seed):
    rng = np.random.default_rng(1000 + seed)
    n_bs = int(rng.integers(1, 65))
    n = int(rng.integers(1, n_bs + 1)) if seed % 3 else n_bs
    cfg = small_variant(CONFIGS["tiny"], n=n, seed=seed, ctx_lo=0, ctx_hi=300)
    req = make_requests(cfg, n_bs=n_bs)
    mode = seed % 5
    if mode == 1:      # non-monotone scores: the running minimum matters
        req["scores"] = rng.uniform(0, 1, size=(n_bs, 15)).astype(np.float32)
    elif mode == 2:    # plateaus and cross-request ties
        req["scores"] = (np.round(rng.uniform(0, 1, size=(n_bs, 15)) * 8) / 8).astype(np.float32)
    elif mode == 3:    # high scores: forces the shrink branch
        q = rng.uniform(0.96, 0.999, size=n_bs)
        req["scores"] = (q[:, None] ** np.arange(1, 16)[None, :]).astype(np.float32)
    elif mode == 4:    # bimodal, ties everywhere
        q = rng.choice([0.3, 0.97], size=n_bs)
        req["scores"] = (q[:, None] ** np.arange(1, 16)[None, :]).astype(np.float32)
    return req


@pytest.mark.parametrize("seed", range(40))
def test_alloc_matches_oracle_random(P, seed):
    req = _random_req(seed)
    ws = _ws(P, req)
    got = gpu_alloc(P, ws, StagedRequests(req))
    assert_alloc_equal(got, oracle_alloc(req))
    assert ws.status() == 0


@pytest.mark.parametrize("seed", range(8))
def test_alloc_other_budgets(P, seed):
    """dscale_alloc_verify_budget: every total from N to min(16 N, 8 n_bs) that was sampled must
    give the oracle's allocation bit for bit (Eq. 9 does not depend on the total)."""
    rng = np.random.default_rng(300 + seed)
    n_bs = int(rng.integers(2, 33))
    n = int(rng.integers(1, n_bs + 1))
    cfg = small_variant(CONFIGS["tiny"], n=n, seed=700 + seed)
    req = make_requests(cfg, n_bs=n_bs)
    hi = min(16 * n, 8 * n_bs)
    budgets = sorted({n, n + 1, 3 * n, 8 * n - 1, 8 * n, min(8 * n + 1, hi), (n + hi) // 2, hi - 1, hi}
                     & set(range(n, hi + 1)))
    ws = _ws(P, req)
    st = StagedRequests(req)
    for b in budgets:
        got = gpu_alloc(P, ws, st, budget=b)
        assert_alloc_equal(got, oracle_alloc(req, budget=b))
        assert int(got["k"][:n].sum()) == b and int(got["offset"][n]) == b
    assert ws.status() == 0
    # out of range: clamped and flagged
    got = gpu_alloc(P, ws, st, budget=n - 1)
    assert_alloc_equal(got, oracle_alloc(req, budget=n))
    assert ws.status() & 4
    ws2 = _ws(P, req)
    got = gpu_alloc(P, ws2, st, budget=16 * n_bs + 5)
    assert_alloc_equal(got, oracle_alloc(req, budget=hi))
    assert ws2.status() & 4


@pytest.mark.parametrize("W", [2, 4, 8, 12])
def test_alloc_other_block_widths(P, W):
    """dscale_alloc_verify_ex with a narrower block: the oracle run with the same W on the first
    W - 1 scores and W tokens.  The workspace keeps its 8 n_bs packed rows, the oracle's arrays have
    (W / 2) n_bs: the common prefix must agree bit for bit, default and other budgets."""
    for seed in range(3):
        rng = np.random.default_rng(40 * W + seed)
        n_bs = int(rng.integers(2, 40))
        n = int(rng.integers(1, n_bs + 1))
        cfg = small_variant(CONFIGS["tiny"], n=n, seed=800 + 10 * W + seed)
        req = make_requests(cfg, n_bs=n_bs)
        ws = _ws(P, req)
        st = StagedRequests(req)
        hi = min(W * n, 8 * n_bs)
        for budget in (None, n, hi, (n + hi) // 2):
            got = gpu_alloc(P, ws, st, budget=budget, block_width=W)
            exp = oracle_alloc(req, budget=budget, block_width=W)
            for f in ALLOC_FIELDS:
                m = len(exp[f])
                np.testing.assert_array_equal(got[f][:m], exp[f], err_msg=f"W={W} budget={budget} field {f}")
            assert got["k"][:n].max() <= W and got["k"][:n].min() >= 1
        assert ws.status() == 0
    import ctypes as C
    assert P.lib.dscale_alloc_verify_ex(C.c_void_p(ws.ptr), n_bs, None, None, 0, None, None, None, 1, 1, 7,
                                        None, None) == -2          # odd width
    assert P.lib.dscale_alloc_verify_ex(C.c_void_p(ws.ptr), n_bs, None, None, 0, None, None, None, 1, 1, 18,
                                        None, None) == -2          # wider than the 16 slots there are


@pytest.mark.parametrize("W,budget", [(16, 52), (8, None), (8, 29), (4, None)])
def test_other_budget_and_width_through_attention_and_accept(P, W, budget):
    """A step under another budget (13 rows per request) or a narrower block: the downstream calls
    read M_live, lengths and offsets from the workspace and need no other change."""
    cfg = small_variant(CONFIGS["tiny"], n=4, seed=77, vocab=2048)
    req, _, kc, vc, qu, _ = full_case(cfg, n_bs=8)
    n, n_bs = 4, 8
    b = (W // 2) * n if budget is None else budget
    alloc = oracle_alloc(req, budget=budget, block_width=W)
    ws = _ws(P, req)
    st = StagedRequests(req)
    assert_alloc_equal(gpu_alloc(P, ws, st, budget=budget, block_width=W), alloc)
    qp = rows_to_packed(qu, alloc["k"], alloc["offset"], n, 8 * n_bs)
    out = torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    P.verify_attn(ws, qp.cuda(), kc.cuda(), vc.cuda(), st.block_table, SCALE, out)
    torch.cuda.synchronize()
    ok, max_abs, worst = attn_close(out, oracle_attn(req, alloc, kc, vc, qp))
    assert ok, (max_abs, worst)
    assert (out[b:].float() == 0).all()
    lp = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], n, 8 * n_bs)
    got = gpu_accept(P, ws, lp.cuda(), cfg.vocab, n_bs)
    exp = oracle_accept(req, alloc, lp)
    np.testing.assert_array_equal(got["top1"][:b], exp["top1"][:b])
    for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
        np.testing.assert_array_equal(got[f], exp[f], err_msg=f)
    assert ws.status() == 0


def test_alloc_extremes(P):
    cfg = small_variant(CONFIGS["tiny"], n=64, seed=9)
    for fill in (0.0, 1.0, 0.5):
        req = make_requests(cfg)
        req["scores"][:] = fill
        ws = _ws(P, req)
        got = gpu_alloc(P, ws, StagedRequests(req))
        assert_alloc_equal(got, oracle_alloc(req))
    # N = 1: the single request takes the whole budget of 8
    req = make_requests(small_variant(CONFIGS["tiny"], n=1), n_bs=1)
    ws = _ws(P, req)
    got = gpu_alloc(P, ws, StagedRequests(req))
    assert got["k"][0] == 8
    assert_alloc_equal(got, oracle_alloc(req))


def test_alloc_logits_mode(P):
    rng = np.random.default_rng(3)
    req = make_requests(small_variant(CONFIGS["tiny"], n=24, seed=5))
    req["scores"] = rng.normal(1.0, 2.0, size=(24, 15)).astype(np.float32)
    ws = _ws(P, req)
    got = gpu_alloc(P, ws, StagedRequests(req), logits_mode=True)
    assert_alloc_equal(got, oracle_alloc(req, logits_mode=True))


def test_alloc_flags_bad_inputs_and_stays_in_bounds(P):
    req = make_requests(small_variant(CONFIGS["tiny"], n=6, seed=2), n_bs=8)
    req["scores"][1, 3] = np.nan
    req["scores"][2, 0] = 1.5
    ws = _ws(P, req)
    got = gpu_alloc(P, ws, StagedRequests(req))
    assert ws.status() & 1
    assert got["k"][:6].sum() == 48 and (got["k"][:6] >= 1).all() and (got["k"][:6] <= 16).all()
    assert got["offset"][6] == 48
    # bad context length and bad N are clamped and flagged
    req = make_requests(small_variant(CONFIGS["tiny"], n=4, seed=2), n_bs=4)
    req["ctx_len"][2] = 10 ** 6
    st = StagedRequests(req)
    st.n_live.fill_(9)
    ws = _ws(P, req)
    got = gpu_alloc(P, ws, st)
    assert ws.status() & 4
    assert got["k"].sum() == 32 and got["positions"].max() < req["max_pages"] * 16


def test_host_side_argument_validation(P):
    req = make_requests(CONFIGS["tiny"])
    ws = _ws(P, req)
    st = StagedRequests(req)
    lib = P.lib
    import ctypes as C
    null = C.c_void_p(0)
    ok = [C.c_void_p(ws.ptr), 4, C.c_void_p(st.n_live.data_ptr()), C.c_void_p(st.scores.data_ptr()),
          0, C.c_void_p(st.draft.data_ptr()), C.c_void_p(st.ctx_len.data_ptr()),
          C.c_void_p(st.block_table.data_ptr()), req["max_pages"], req["num_pages"], null]
    assert lib.dscale_alloc_verify(*ok) == 0
    bad = list(ok); bad[3] = null
    assert lib.dscale_alloc_verify(*bad) == -1
    bad = list(ok); bad[1] = 5                     # capacity does not match the workspace
    assert lib.dscale_alloc_verify(*bad) == -4
    bad = list(ok); bad[0] = C.c_void_p(ws.ptr + 256)   # not an initialised workspace
    assert lib.dscale_alloc_verify(*bad) == -4
    # a destroyed workspace is unknown to every call until it is initialised again
    assert lib.dscale_workspace_destroy(C.c_void_p(ws.ptr)) == 0
    assert lib.dscale_workspace_destroy(C.c_void_p(ws.ptr)) == -4
    assert lib.dscale_alloc_verify(*ok) == -4
    assert lib.dscale_workspace_init(C.c_void_p(ws.ptr), ws.nbytes, 4, 8, 2, 128, ws.num_sms, null) == 0
    assert lib.dscale_alloc_verify(*ok) == 0
    assert lib.dscale_workspace_bytes(65, 32, 8, 128, 148) == 0
    assert lib.dscale_workspace_bytes(8, 32, 8, 64, 148) == 0
    assert lib.dscale_workspace_bytes(8, 30, 8, 128, 148) == 0
    torch.cuda.synchronize()


# ------------------------------------------------------------------ acceptance
@pytest.mark.parametrize("name,vocab", [("tiny", 1024), ("tiny", 1023), ("qwen3_4b_layer", 151936),
                                        ("qwen3_8b_layer", 50001)])
def test_accept_matches_oracle_and_planted_truth(P, name, vocab):
    cfg = small_variant(CONFIGS[name], vocab=vocab)
    req = make_requests(cfg, n_bs=cfg.n + 3)
    alloc = oracle_alloc(req)
    ws = _ws(P, req)
    st = StagedRequests(req)
    gpu_alloc(P, ws, st)
    lu = make_logits_unpacked(req)
    lp = rows_to_packed(lu, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"])
    ld = (vocab + 3) // 4 * 4
    lp_dev = torch.full((8 * req["n_bs"], ld), float("nan"), dtype=torch.float32, device="cuda")
    lp_dev[:, :vocab] = lp.cuda()
    ctx_dev = st.ctx_len.clone()
    got = gpu_accept(P, ws, lp_dev, vocab, req["n_bs"], ctx_dev)
    exp = oracle_accept(req, alloc, lp, with_ctx=True)
    for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
        np.testing.assert_array_equal(got[f], exp[f], err_msg=f)
    np.testing.assert_array_equal(got["top1"][:8 * cfg.n], exp["top1"][:8 * cfg.n])
    np.testing.assert_array_equal(ctx_dev.cpu().numpy(), exp["ctx_len"])
    truth = planted_expectation(req, alloc["k"])
    np.testing.assert_array_equal(got["accept_len"], truth["accept_len"])
    np.testing.assert_array_equal(got["next_anchor"], truth["next_anchor"])


def test_accept_ties_nan_and_edge_rows(P):
    cfg = small_variant(CONFIGS["tiny"], vocab=70000, n=4)
    req = make_requests(cfg)
    alloc = oracle_alloc(req)
    ws = _ws(P, req)
    gpu_alloc(P, ws, StagedRequests(req))
    rng = np.random.default_rng(0)
    lp = torch.from_numpy(rng.integers(-3, 4, size=(32, 70000)).astype(np.float32))  # many ties
    lp[1, :] = float("nan")
    lp[2, :] = float("-inf")
    lp[3, 17] = float("nan"); lp[3, 69999] = 50.0
    lp[4, 0] = 60.0; lp[4, 69999] = 60.0
    lp[5, 17499] = 9.0; lp[5, 17500] = 9.0           # tie across a chunk boundary (4 chunks of 17500)
    got = gpu_accept(P, ws, lp.cuda(), 70000, 4)
    exp = oracle_accept(req, alloc, lp)
    np.testing.assert_array_equal(got["top1"][:32], exp["top1"][:32])
    for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
        np.testing.assert_array_equal(got[f], exp[f], err_msg=f)


# ------------------------------------------------------------------- attention
def _attn_parity(P, impl, cfg, n_bs=None, ctx_override=None, hidden_poison=True):
    req, alloc, kc, vc, qu, qp = full_case(cfg, n_bs=n_bs, ctx_override=ctx_override)
    if hidden_poison:
        poison_hidden_slots(req, alloc, kc, vc)
    ws = _ws(P, req)
    st = StagedRequests(req)
    got_alloc = gpu_alloc(P, ws, st)
    assert_alloc_equal(got_alloc, alloc)
    out = torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    fn = P.verify_attn if impl == "tensor" else P.verify_attn_simt
    fn(ws, qp.cuda(), kc.cuda(), vc.cuda(), st.block_table, SCALE, out)
    torch.cuda.synchronize()
    assert ws.status() == 0
    ref = oracle_attn(req, alloc, kc, vc, qp)
    ok, max_abs, worst = attn_close(out, ref)
    assert ok, f"{impl}: max|d|={max_abs} worst at (row, head, d)={worst}"
    m_live = 8 * req["n_live"]
    assert (out[m_live:].float() == 0).all()
    return max_abs


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_tiny(P, impl):
    _attn_parity(P, impl, CONFIGS["tiny"])
    _attn_parity(P, impl, CONFIGS["tiny"], n_bs=7)


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_edge_context_lengths(P, impl):
    # empty context, around page (16) and key-tile (128) boundaries, ragged tails
    ctx = [0, 1, 15, 16, 17, 111, 112, 113, 127, 128, 129, 255, 256, 257, 300, 1000]
    cfg = small_variant(CONFIGS["tiny"], n=len(ctx), seed=11, n_q_heads=8, n_kv_heads=2)
    _attn_parity(P, impl, cfg, ctx_override=ctx)


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_qwen3_4b_layer(P, impl):
    worst = _attn_parity(P, impl, CONFIGS["qwen3_4b_layer"])
    assert worst < 5e-3


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_skewed_lengths(P, impl):
    # window lengths 1 and 15 side by side, short and long contexts
    cfg = small_variant(CONFIGS["skew"], n=8, ctx_lo=40, ctx_hi=2100)
    _attn_parity(P, impl, cfg, n_bs=8)


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_pairs_cut_across_many_ctas(P, impl):
    # two long requests on two kv-heads: every (request, kv-head) pair spans dozens of CTAs of the
    # persistent grid, so the split-KV merge sees many contributors per pair
    cfg = small_variant(CONFIGS["tiny"], n=2, seed=41)
    _attn_parity(P, impl, cfg, ctx_override=[20000, 9000])


@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_attn_full_capacity_of_64_requests(P, impl):
    cfg = small_variant(CONFIGS["tiny"], n=64, seed=43, ctx_lo=0, ctx_hi=300)
    _attn_parity(P, impl, cfg)
    cfg = small_variant(CONFIGS["tiny"], n=37, seed=44, ctx_lo=100, ctx_hi=900)
    _attn_parity(P, impl, cfg, n_bs=64)


@pytest.mark.parametrize("seed", range(12))
def test_attn_random_shapes(P, seed):
    """Seeded sweep over live counts, capacities, head counts and context mixes (short, around
    the 128-key tile boundary, long enough to be cut across CTAs): the tensor-core kernel against
    the oracle, then the CUDA-core kernel against the same oracle on the same inputs."""
    rng = np.random.default_rng(1000 + seed)
    n_bs = int(rng.integers(1, 25))
    n = int(rng.integers(1, n_bs + 1))
    h_kv = int(rng.choice([1, 2, 4, 8]))
    kinds = rng.integers(0, 4, size=n)
    ctx = np.where(kinds == 0, rng.integers(0, 40, size=n),
          np.where(kinds == 1, 128 * rng.integers(1, 4, size=n) + rng.integers(-2, 3, size=n),
          np.where(kinds == 2, rng.integers(200, 1500, size=n), rng.integers(2000, 6000, size=n))))
    if seed % 3 == 0:
        ctx[int(rng.integers(0, n))] = int(rng.integers(12000, 30000))     # one pair over many CTAs
    cfg = small_variant(CONFIGS["tiny"], n=n, seed=500 + seed, n_q_heads=4 * h_kv, n_kv_heads=h_kv)
    for impl in ("tensor", "simt"):
        _attn_parity(P, impl, cfg, n_bs=n_bs, ctx_override=[int(x) for x in ctx])


def test_attn_simt_other_group_sizes(P):
    for hq, hkv in ((4, 4), (8, 4), (8, 1)):
        cfg = small_variant(CONFIGS["tiny"], n_q_heads=hq, n_kv_heads=hkv, seed=21)
        _attn_parity(P, "simt", cfg)


# ------------------------------------------------- padded comparison baseline
@pytest.mark.parametrize("name,n_bs", [("tiny", 4), ("tiny", 6), ("qwen3_4b_layer", 8)])
def test_padded_baseline_matches_unpacked_oracle(P, name, n_bs):
    from oracle import verify_attn as OV
    cfg = CONFIGS[name]
    req, alloc, kc, vc, qu, qp = full_case(cfg, n_bs=n_bs)
    ws = _ws(P, req)
    st = StagedRequests(req)
    gpu_alloc(P, ws, st)                                  # the baseline takes N from the workspace
    out = torch.full(qu.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    P.verify_attn_padded(ws, qu.cuda(), kc.cuda(), vc.cuda(), st.block_table, st.ctx_len, SCALE, out)
    torch.cuda.synchronize()
    assert ws.status() == 0
    ref = OV.verify_attn_padded(qu.float().numpy(), kc.float().numpy(), vc.float().numpy(),
                                req["block_table"], req["ctx_len"], req["n_live"], cfg.n_q_heads,
                                cfg.n_kv_heads, SCALE)
    ok, max_abs, worst = attn_close(out, ref)
    assert ok, f"padded: max|d|={max_abs} worst at {worst}"
    assert (out[req["n_live"]:].float() == 0).all()


# -------------------------------------------------------------- graph replay
@pytest.mark.parametrize("impl", ["simt", "tensor"])
def test_one_captured_graph_replays_at_any_mix_of_lengths(P, impl):
    base = small_variant(CONFIGS["tiny"], vocab=4096, ctx_lo=30, ctx_hi=400)
    n_bs = 8
    steps = [make_requests(small_variant(base, n=n, seed=s), n_bs=n_bs)
             for n, s in ((8, 1), (3, 2), (6, 3))]
    max_pages = max(r["max_pages"] for r in steps)
    num_pages = max(r["num_pages"] for r in steps)
    for r in steps:                                   # same shapes at every replay
        bt = np.full((n_bs, max_pages), -1, dtype=np.int32)
        bt[:, : r["max_pages"]] = r["block_table"]
        r["block_table"], r["max_pages"], r["num_pages"] = bt, max_pages, num_pages
    cfg = steps[0]["cfg"]
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads)
    st = StagedRequests(steps[0])
    shape_kv = (num_pages, cfg.n_kv_heads, 16, 128)
    kc = torch.zeros(shape_kv, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    q = torch.zeros((8 * n_bs, cfg.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    logits = torch.zeros((8 * n_bs, cfg.vocab), dtype=torch.float32, device="cuda")
    o = dict(accept_len=torch.zeros(n_bs, dtype=torch.int32, device="cuda"),
             next_anchor=torch.zeros(n_bs, dtype=torch.int32, device="cuda"),
             out_tokens=torch.zeros((n_bs, 16), dtype=torch.int32, device="cuda"),
             out_len=torch.zeros(n_bs, dtype=torch.int32, device="cuda"))
    fn = P.verify_attn if impl == "tensor" else P.verify_attn_simt

    def step():
        P.alloc_verify(ws, st.n_live, st.scores, st.draft, st.ctx_len, st.block_table, num_pages)
        fn(ws, q, kc, vc, st.block_table, SCALE, out)
        P.accept(ws, logits, cfg.vocab, o["accept_len"], o["next_anchor"], o["out_tokens"],
                 o["out_len"], None)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                         # warm-up outside capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()

    from dscale_inputs import make_kv_layer, make_q_unpacked
    for r in steps:
        alloc = oracle_alloc(r)
        k_cpu, v_cpu = make_kv_layer(r, 0)
        pad = num_pages - k_cpu.shape[0]
        qp = rows_to_packed(make_q_unpacked(r, 0), alloc["k"], alloc["offset"], r["n_live"], 8 * n_bs)
        lp = rows_to_packed(make_logits_unpacked(r), alloc["k"], alloc["offset"], r["n_live"],
                            8 * n_bs)
        st.load(r)
        kc.fill_(float("nan")); vc.fill_(float("nan"))
        kc[: k_cpu.shape[0]].copy_(k_cpu); vc[: v_cpu.shape[0]].copy_(v_cpu)
        q.copy_(qp); logits.copy_(lp)
        graph.replay()
        torch.cuda.synchronize()
        assert ws.status() == 0
        for f in ALLOC_FIELDS:
            np.testing.assert_array_equal(ws.field(f).cpu().numpy(), alloc[f], err_msg=f)
        ref = oracle_attn(r, alloc, k_cpu, v_cpu, qp)
        ok, max_abs, worst = attn_close(out, ref)
        assert ok, f"replay N={r['n_live']}: max|d|={max_abs} at {worst}"
        exp = oracle_accept(r, alloc, lp)
        for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
            np.testing.assert_array_equal(o[f].cpu().numpy(), exp[f], err_msg=f)
        truth = planted_expectation(r, alloc["k"])
        np.testing.assert_array_equal(o["accept_len"].cpu().numpy(), truth["accept_len"])
        assert pad >= 0
