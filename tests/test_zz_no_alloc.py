"""dscale_accept_static: the acceptance entry point for callers that cannot
allocate device memory (a serving loop where cudaMalloc would stall the
device, a plug-in that only gets input / output pointers).  Its scratch is a
fixed array inside the library, so the checks that matter are that it returns
exactly what the workspace-based dscale_accept returns and what the CPU oracle's
sequential acceptance loop returns, on calls in a row (every call after the
first finds the previous call's leftovers in the shared scratch), also when the
lengths come from an allocation under another budget or block width.

This file is collected last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, make_logits_unpacked, make_requests, rows_to_packed, small_variant
from gpu_case import StagedRequests, gpu_accept, gpu_alloc, oracle_accept, oracle_alloc

pytestmark = pytest.mark.gpu


def _one_case(P, cfg, n_bs, budget=None, block_width=16):
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req, budget=budget, block_width=block_width)
    ws = P.VerifyWorkspace(req["n_bs"], cfg.n_q_heads, cfg.n_kv_heads)
    st = StagedRequests(req)
    gpu_alloc(P, ws, st, budget=budget, block_width=block_width)
    lp_cpu = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], req["n_live"],
                            8 * req["n_bs"])
    lp = lp_cpu.cuda()
    want = gpu_accept(P, ws, lp, cfg.vocab, req["n_bs"])          # existing entry point
    exp = oracle_accept(req, alloc, lp_cpu)                        # the oracle's sequential loop

    outs = [torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
            torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
            torch.full((n_bs, 16), -9, dtype=torch.int32, device="cuda"),
            torch.full((n_bs,), -9, dtype=torch.int32, device="cuda")]
    ptr = lambda t: C.c_void_p(t.data_ptr())
    rc = P.lib.dscale_accept_static(                                # straight through the C ABI
        n_bs, ptr(st.n_live), ptr(ws.field("k")), ptr(ws.field("offset")), ptr(ws.field("tokens")),
        ptr(lp), lp.stride(0), cfg.vocab, ptr(outs[0]), ptr(outs[1]), ptr(outs[2]), ptr(outs[3]),
        C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    torch.cuda.synchronize()
    for name, got in zip(("accept_len", "next_anchor", "out_tokens", "out_len"), outs):
        np.testing.assert_array_equal(got.cpu().numpy(), want[name], err_msg=name)
        np.testing.assert_array_equal(got.cpu().numpy(), exp[name], err_msg=name + " (oracle)")


def test_static_scratch_accept_matches_workspace_accept_twice_in_a_row():
    import paper_2609_37532_b200 as P
    # two different problems back to back: different sizes, vocabularies and lengths
    _one_case(P, small_variant(CONFIGS["qwen3_4b_layer"], vocab=151936), n_bs=11)
    _one_case(P, small_variant(CONFIGS["tiny"], vocab=40000, n=4, seed=6), n_bs=4)


def test_static_scratch_accept_under_other_budgets_and_block_widths():
    """Lengths from dscale_alloc_verify_ex: 13 rows per request (more live rows than 8 N, which
    a row count derived from N alone would cut short), 3 rows per request after a larger call
    (the scratch then still holds target tokens of rows that are no longer live), and an
    8-slot block."""
    import paper_2609_37532_b200 as P
    cfg = small_variant(CONFIGS["tiny"], vocab=30000, n=4, seed=8)
    _one_case(P, cfg, n_bs=8, budget=13 * 4)
    _one_case(P, cfg, n_bs=8, budget=3 * 4)
    _one_case(P, small_variant(cfg, seed=9), n_bs=6, block_width=8)
    _one_case(P, small_variant(cfg, seed=10), n_bs=7, budget=29, block_width=8)


def test_static_scratch_accept_gives_sentinel_outputs_for_rows_outside_the_live_range():
    """Caller-made lengths that point outside the live packed rows must not be followed."""
    import paper_2609_37532_b200 as P
    n_bs, vocab = 4, 4096
    ptr = lambda t: C.c_void_p(t.data_ptr())
    dev = lambda a: torch.tensor(a, dtype=torch.int32, device="cuda")
    n_live = dev([3])
    k = dev([4, 30, 5, 0])                       # request 1: a length no block has
    offset = dev([0, 4, 9, 14, 14])              # request 2 would end at 14 = offset[N]: fine
    tokens = torch.randint(0, vocab, (8 * n_bs,), dtype=torch.int32, device="cuda")
    lg = torch.randn((8 * n_bs, vocab), dtype=torch.float32, device="cuda")
    outs = [torch.full((n_bs,), -9, dtype=torch.int32, device="cuda") for _ in range(2)]
    outs += [torch.full((n_bs, 16), -9, dtype=torch.int32, device="cuda"),
             torch.full((n_bs,), -9, dtype=torch.int32, device="cuda")]
    rc = P.lib.dscale_accept_static(n_bs, ptr(n_live), ptr(k), ptr(offset), ptr(tokens), ptr(lg), vocab,
                                    vocab, ptr(outs[0]), ptr(outs[1]), ptr(outs[2]), ptr(outs[3]),
                                    C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    torch.cuda.synchronize()
    top1 = lg.argmax(dim=1).cpu().numpy()
    a_len, nxt, _, o_len = [t.cpu().numpy() for t in outs]
    assert o_len[1] == 0 and nxt[1] == -1 and o_len[3] == 0 and nxt[3] == -1
    for i, (oi, ki) in ((0, (0, 4)), (2, (9, 5))):
        tk = tokens.cpu().numpy()
        a = 0
        while a < ki - 1 and top1[oi + a] == tk[oi + a + 1]:
            a += 1
        assert a_len[i] == a and nxt[i] == top1[oi + a] and o_len[i] == a + 1


def test_static_scratch_accept_rejects_sizes_beyond_its_capacity():
    import paper_2609_37532_b200 as P
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    lg = torch.zeros((8, 8), dtype=torch.float32, device="cuda")
    ptr = lambda t: C.c_void_p(t.data_ptr())
    rc = P.lib.dscale_accept_static(65, ptr(z), ptr(z), ptr(z), ptr(z), ptr(lg), 8, 8, ptr(z),
                                    ptr(z), ptr(z), ptr(z), C.c_void_p(0))
    assert rc == -5
    torch.cuda.synchronize()
