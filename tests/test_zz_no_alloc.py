"""dscale_accept_static: the acceptance entry point for callers that cannot
allocate device memory (a serving loop where cudaMalloc would stall the
device, a plug-in that only gets input / output pointers).  Its scratch is a
fixed array inside the library, so the check that matters is that it returns
exactly what the workspace-based dscale_accept returns, on two calls in a row
(the second call finds the first call's leftovers in the shared scratch).

This file is collected last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, make_logits_unpacked, make_requests, rows_to_packed, small_variant
from gpu_case import StagedRequests, gpu_accept, gpu_alloc, oracle_alloc

pytestmark = pytest.mark.gpu


def _one_case(P, cfg, n_bs):
    req = make_requests(cfg, n_bs=n_bs)
    alloc = oracle_alloc(req)
    ws = P.VerifyWorkspace(req["n_bs"], cfg.n_q_heads, cfg.n_kv_heads)
    st = StagedRequests(req)
    gpu_alloc(P, ws, st)
    lp = rows_to_packed(make_logits_unpacked(req), alloc["k"], alloc["offset"], req["n_live"],
                        8 * req["n_bs"]).cuda()
    want = gpu_accept(P, ws, lp, cfg.vocab, req["n_bs"])          # existing entry point

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


def test_static_scratch_accept_matches_workspace_accept_twice_in_a_row():
    import paper_2609_37532_b200 as P
    # two different problems back to back: different sizes, vocabularies and lengths
    _one_case(P, small_variant(CONFIGS["qwen3_4b_layer"], vocab=151936), n_bs=11)
    _one_case(P, small_variant(CONFIGS["tiny"], vocab=40000, n=4, seed=6), n_bs=4)


def test_static_scratch_accept_rejects_sizes_beyond_its_capacity():
    import paper_2609_37532_b200 as P
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    lg = torch.zeros((8, 8), dtype=torch.float32, device="cuda")
    ptr = lambda t: C.c_void_p(t.data_ptr())
    rc = P.lib.dscale_accept_static(65, ptr(z), ptr(z), ptr(z), ptr(z), ptr(lg), 8, 8, ptr(z),
                                    ptr(z), ptr(z), ptr(z), C.c_void_p(0))
    assert rc == -5
    torch.cuda.synchronize()
