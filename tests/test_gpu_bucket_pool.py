"""Graph pool over request capacities (Eq. 13, Algorithm 2): bucket choice, sentinel-heavy
replays, one captured graph per bucket, results against the oracle."""
import ctypes as C

import numpy as np
import pytest
import torch

from dscale_inputs import (CONFIGS, make_kv_layer, make_logits_unpacked, make_q_unpacked,
                           make_requests, planted_expectation, rows_to_packed, small_variant)
from gpu_case import ALLOC_FIELDS, SCALE, attn_close, oracle_accept, oracle_alloc, oracle_attn


def test_bucket_choice_is_the_smallest_that_fits():
    import paper_2609_37532_b200 as P
    arr = (C.c_int32 * 4)(16, 4, 32, 8)
    pick = lambda n: P.lib.dscale_select_bucket(arr, 4, n)
    assert [pick(n) for n in (1, 4, 5, 8, 9, 16, 17, 32)] == [4, 4, 8, 8, 16, 16, 32, 32]
    assert pick(33) == -5 and pick(0) == -1
    assert P.lib.dscale_select_bucket(arr, 0, 3) == -1


@pytest.mark.gpu
def test_pool_replays_each_step_in_its_bucket():
    import paper_2609_37532_b200 as P
    base = small_variant(CONFIGS["tiny"], vocab=2048, ctx_lo=20, ctx_hi=500)
    steps = [(3, 11), (8, 12), (5, 13), (1, 14), (7, 15)]          # (N, seed): buckets 4, 8, 8, 4, 8
    reqs = {}
    for n, seed in steps:
        b = 4 if n <= 4 else 8
        reqs[(n, seed)] = make_requests(small_variant(base, n=n, seed=seed), n_bs=b)
    max_pages = max(r["max_pages"] for r in reqs.values())
    num_pages = max(r["num_pages"] for r in reqs.values())
    cfg = base
    kc = torch.zeros((num_pages, cfg.n_kv_heads, 16, 128), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    pool = P.VerifyGraphPool([8, 4], cfg.n_q_heads, cfg.n_kv_heads, max_pages, [(kc, vc)],
                             cfg.vocab, SCALE)
    assert pool.select(3) == 4 and pool.select(5) == 8
    for (n, seed) in steps:
        r = reqs[(n, seed)]
        n_bs = r["n_bs"]
        alloc = oracle_alloc(r)
        k_cpu, v_cpu = make_kv_layer(r, 0)
        qp = rows_to_packed(make_q_unpacked(r, 0), alloc["k"], alloc["offset"], n, 8 * n_bs)
        lp = rows_to_packed(make_logits_unpacked(r), alloc["k"], alloc["offset"], n, 8 * n_bs)
        t = pool.slot(n)
        assert t["ws"].n_bs == n_bs
        kc.fill_(float("nan")); vc.fill_(float("nan"))
        kc[: k_cpu.shape[0]].copy_(k_cpu); vc[: v_cpu.shape[0]].copy_(v_cpu)
        bt = np.full((n_bs, max_pages), -1, dtype=np.int32)
        bt[:, : r["max_pages"]] = r["block_table"]
        t["n_live"].fill_(n)
        t["scores"].copy_(torch.as_tensor(r["scores"])); t["draft"].copy_(torch.as_tensor(r["draft_tokens"]))
        t["ctx_len"].copy_(torch.as_tensor(r["ctx_len"])); t["block_table"].copy_(torch.as_tensor(bt))
        t["q"][0].copy_(qp); t["logits"].copy_(lp)
        t["out"][0].fill_(float("nan"))
        pool.replay(n)
        torch.cuda.synchronize()
        assert t["ws"].status() == 0
        for f in ALLOC_FIELDS:
            np.testing.assert_array_equal(t["ws"].field(f).cpu().numpy(), alloc[f], err_msg=f)
        ok, max_abs, worst = attn_close(t["out"][0], oracle_attn(r, alloc, k_cpu, v_cpu, qp))
        assert ok, f"N={n}: max|d|={max_abs} at {worst}"
        assert (t["out"][0][8 * n:].float() == 0).all()            # sentinel rows
        exp = oracle_accept(r, alloc, lp)
        for f in ("accept_len", "next_anchor", "out_tokens", "out_len"):
            np.testing.assert_array_equal(t[f].cpu().numpy(), exp[f], err_msg=f)
        truth = planted_expectation(r, alloc["k"])
        np.testing.assert_array_equal(t["accept_len"].cpu().numpy(), truth["accept_len"])
