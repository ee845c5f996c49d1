"""A bounded device-side wait that runs out, made to happen without any GPU fault.

Every wait inside the attention kernel (mbarrier waits of the copy, MMA and softmax warps)
has a time limit; when one runs out the CTA raises its abort flag, all of its warps leave
their loops, the copy warps wait (bounded) for the copies still in flight, the MMA warp waits
(bounded) for the products still in flight, tensor memory is released and the kernel returns
with DSCALE_STATUS_TIMEOUT set in the workspace.  Nothing traps and nothing spins without limit.

The path is exercised with the wait-limit test build of the library
(libdscale_waittest.so: the same sources, every limit at about 1 ms, plus a hook that leaves
out the copies of one key tile of one CTA while the tile's barrier stays armed), loaded here
beside the product library.  After the timed-out call the workspace is re-initialised, as the
header prescribes for a sticky status, and the same call must match the oracle again.
"""
import ctypes as C
import os

import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, make_requests, small_variant
from gpu_case import ALLOC_FIELDS, SCALE, attn_close, dev, full_case, oracle_attn

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LIB_PATH = os.path.join(ROOT, "paper_2609_37532_b200", "libdscale_waittest.so")


@pytest.fixture(scope="module")
def wlib():
    import paper_2609_37532_b200  # noqa: F401  (builds both libraries if they are stale)
    lib = C.CDLL(LIB_PATH)
    lib.dscale_workspace_bytes.restype = C.c_size_t
    lib.dscale_ws_field.restype = C.c_void_p
    lib.dscale_ws_field.argtypes = [C.c_void_p, C.c_int, C.c_int]
    return lib


def _vp(t):
    return C.c_void_p(t.data_ptr())


def test_a_wait_that_runs_out_sets_the_status_and_the_kernel_returns(wlib):
    # two long pairs on two kv-heads: every CTA of the grid has a slice of a few key tiles
    cfg = small_variant(CONFIGS["tiny"], n=2, seed=41)
    req, alloc, kc, vc, qu, qp = full_case(cfg, ctx_override=[20000, 9000])
    n_bs, hq, hkv = req["n_bs"], cfg.n_q_heads, cfg.n_kv_heads
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nbytes = wlib.dscale_workspace_bytes(n_bs, hq, hkv, 128, sms)
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    ws = buf.data_ptr() + (-buf.data_ptr()) % 256
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)

    n_live = dev(np.array([req["n_live"]], dtype=np.int32))
    scores, draft = dev(req["scores"]), dev(req["draft_tokens"])
    ctx, bt = dev(req["ctx_len"]), dev(req["block_table"])
    q_d, k_d, v_d = qp.cuda(), kc.cuda(), vc.cuda()
    out = torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")

    def status():
        addr = wlib.dscale_ws_field(C.c_void_p(ws), n_bs, 0)
        off = addr - buf.data_ptr()
        return int(buf[off:off + 4].view(torch.int32).item())

    def init_and_alloc():
        assert wlib.dscale_workspace_init(C.c_void_p(ws), C.c_size_t(nbytes), n_bs, hq, hkv, 128, sms, stream) == 0
        assert wlib.dscale_alloc_verify(C.c_void_p(ws), n_bs, _vp(n_live), _vp(scores), 0, _vp(draft), _vp(ctx),
                                        _vp(bt), req["max_pages"], req["num_pages"], stream) == 0

    def attention():
        rc = wlib.dscale_verify_attn(C.c_void_p(ws), n_bs, _vp(q_d), _vp(k_d), _vp(v_d), _vp(bt), req["max_pages"],
                                     req["num_pages"], hq, hkv, C.c_float(SCALE), _vp(out), stream)
        assert rc == 0
        torch.cuda.synchronize()          # returns: the kernel ended by itself

    init_and_alloc()
    torch.cuda.synchronize()
    for f, fid in (("k", 1), ("offset", 2)):
        addr = wlib.dscale_ws_field(C.c_void_p(ws), n_bs, fid)
        off = addr - buf.data_ptr()
        got = buf[off:off + 4 * len(alloc[f])].view(torch.int32).cpu().numpy()
        np.testing.assert_array_equal(got, alloc[f], err_msg=f)

    # 1. CTA 5 never gets the K copies of its second key tile: the waits behind it run out
    assert wlib.dscale_test_drop_copy(5, 1) == 0
    attention()
    assert status() & 8, "DSCALE_STATUS_TIMEOUT was not set"
    assert status() & ~8 == 0

    # 2. the status is sticky, and the pair whose contributor gave up never completed its
    #    ticket count: the workspace is initialised again, as the header prescribes
    assert wlib.dscale_test_drop_copy(-1, -1) == 0
    init_and_alloc()
    out.fill_(float("nan"))
    attention()
    assert status() == 0
    ok, max_abs, worst = attn_close(out, oracle_attn(req, alloc, kc, vc, qp))
    assert ok, f"after re-initialisation: max|d|={max_abs} at {worst}"

    # 3. and once more without re-initialising: the tickets of a clean launch reset themselves
    out.fill_(float("nan"))
    attention()
    assert status() == 0
    ok, max_abs, worst = attn_close(out, oracle_attn(req, alloc, kc, vc, qp))
    assert ok, f"second clean launch: max|d|={max_abs} at {worst}"
    assert wlib.dscale_workspace_destroy(C.c_void_p(ws)) == 0


def test_predictor_stream_wait_runs_out_and_the_call_returns(wlib):
    """The same for the predictor's stream kernel: one CTA never gets the logit boxes of its second
    sub-tile, its compute warps run into the wait limit, raise the abort flag, the copy warp waits
    (bounded) for what is in flight, the CTA returns, the tail kernel behind it runs on whatever
    records there are, and the call ends with DSCALE_STATUS_TIMEOUT.  After re-initialisation the
    same call gives the product library's result again."""
    import paper_2609_37532_b200 as P
    from dscale_inputs import make_predictor_inputs
    cfg = small_variant(CONFIGS["tiny"], vocab=20480, n=3, seed=83)
    req = make_requests(cfg, n_bs=4)
    n_bs, hq, hkv = 4, cfg.n_q_heads, cfg.n_kv_heads
    d = {k: (v.cuda().contiguous() if torch.is_tensor(v) else v) for k, v in make_predictor_inputs(req, 64).items()}
    n_live = dev(np.array([req["n_live"]], dtype=np.int32))
    # the product library's answer
    pws = P.VerifyWorkspace(n_bs, hq, hkv)
    want = torch.zeros((n_bs, 15), dtype=torch.float32, device="cuda")
    P.predict_scores(pws, n_live, d["draft_logits"], cfg.vocab, d["draft_hidden"], d["p_hidden"], d["p_logit"],
                     d["w1"], d["b1"], d["w2"], d["b2"], want)
    torch.cuda.synchronize()

    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nbytes = wlib.dscale_workspace_bytes(n_bs, hq, hkv, 128, sms)
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    ws = buf.data_ptr() + (-buf.data_ptr()) % 256
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    got = torch.zeros((n_bs, 15), dtype=torch.float32, device="cuda")

    def status():
        off = wlib.dscale_ws_field(C.c_void_p(ws), n_bs, 0) - buf.data_ptr()
        return int(buf[off:off + 4].view(torch.int32).item())

    def init():
        assert wlib.dscale_workspace_init(C.c_void_p(ws), C.c_size_t(nbytes), n_bs, hq, hkv, 128, sms, stream) == 0

    def predict():
        rc = wlib.dscale_predict_scores(
            C.c_void_p(ws), n_bs, _vp(n_live), _vp(d["draft_logits"]), C.c_int64(d["draft_logits"].shape[2]),
            cfg.vocab, _vp(d["draft_hidden"]), 64, _vp(d["p_hidden"]), _vp(d["p_logit"]), _vp(d["w1"]), _vp(d["b1"]),
            _vp(d["w2"]), _vp(d["b2"]), _vp(got), C.c_void_p(None), stream)
        assert rc == 0
        torch.cuda.synchronize()          # returns: the kernels ended by themselves

    init()
    assert wlib.dscale_test_drop_pred_copy(0, 1) == 0
    predict()
    assert status() & 8, "DSCALE_STATUS_TIMEOUT was not set"
    assert status() & ~8 == 0
    assert wlib.dscale_test_drop_pred_copy(-1, -1) == 0
    init()
    got.zero_()
    predict()
    assert status() == 0
    np.testing.assert_array_equal(got.cpu().numpy(), want.cpu().numpy())
    assert wlib.dscale_workspace_destroy(C.c_void_p(ws)) == 0


def test_lm_head_wait_runs_out_and_the_call_returns(wlib):
    """The same for the one-CTA-per-tile LM-head kernel: one CTA never gets the weight box of its
    second k step; its MMA warp runs into the wait limit, waits (bounded) for the products it has
    issued, the copy warp waits (bounded) for the copies it has armed, the epilogue warps leave,
    tensor memory is released and the kernel returns with DSCALE_STATUS_TIMEOUT.  After
    re-initialisation the same call gives the product library's outputs."""
    import paper_2609_37532_b200 as P
    from dscale_inputs import make_lm_head_unpacked, rows_to_packed
    from gpu_case import StagedRequests, gpu_alloc, oracle_alloc
    cfg = small_variant(CONFIGS["tiny"], vocab=20000, n=7, seed=85)
    req = make_requests(cfg, n_bs=8)
    n_bs, n, hq, hkv, H = 8, req["n_live"], cfg.n_q_heads, cfg.n_kv_heads, 512
    alloc = oracle_alloc(req)
    weight, hid_unpacked = make_lm_head_unpacked(req, H)
    hidden = rows_to_packed(hid_unpacked, alloc["k"], alloc["offset"], n, 8 * n_bs).cuda().contiguous()
    weight = weight.cuda().contiguous()

    def outputs():
        return [torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
                torch.full((n_bs,), -9, dtype=torch.int32, device="cuda"),
                torch.full((n_bs, 16), -9, dtype=torch.int32, device="cuda"),
                torch.full((n_bs,), -9, dtype=torch.int32, device="cuda")]

    # the product library's answer
    pws = P.VerifyWorkspace(n_bs, hq, hkv)
    gpu_alloc(P, pws, StagedRequests(req))
    want = outputs()
    P.lm_head_accept(pws, hidden, weight, want[0], want[1], want[2], want[3])
    torch.cuda.synchronize()
    assert pws.status() == 0

    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nbytes = wlib.dscale_workspace_bytes(n_bs, hq, hkv, 128, sms)
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    ws = buf.data_ptr() + (-buf.data_ptr()) % 256
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    n_live = dev(np.array([n], dtype=np.int32))
    scores, draft = dev(req["scores"]), dev(req["draft_tokens"])
    ctx, bt = dev(req["ctx_len"]), dev(req["block_table"])

    def status():
        off = wlib.dscale_ws_field(C.c_void_p(ws), n_bs, 0) - buf.data_ptr()
        return int(buf[off:off + 4].view(torch.int32).item())

    def init_and_alloc():
        assert wlib.dscale_workspace_init(C.c_void_p(ws), C.c_size_t(nbytes), n_bs, hq, hkv, 128, sms, stream) == 0
        assert wlib.dscale_alloc_verify(C.c_void_p(ws), n_bs, _vp(n_live), _vp(scores), 0, _vp(draft), _vp(ctx),
                                        _vp(bt), req["max_pages"], req["num_pages"], stream) == 0

    def lm_head(o):
        rc = wlib.dscale_lm_head_accept(C.c_void_p(ws), n_bs, _vp(hidden), _vp(weight), H, cfg.vocab, _vp(o[0]),
                                        _vp(o[1]), _vp(o[2]), _vp(o[3]), C.c_void_p(None), C.c_void_p(None), stream)
        assert rc == 0
        torch.cuda.synchronize()          # returns: the kernel ended by itself

    init_and_alloc()
    assert wlib.dscale_test_drop_lm_copy(0, 1) == 0
    lm_head(outputs())
    assert status() & 8, "DSCALE_STATUS_TIMEOUT was not set"
    assert status() & ~8 == 0
    assert wlib.dscale_test_drop_lm_copy(-1, -1) == 0
    init_and_alloc()
    got = outputs()
    lm_head(got)
    assert status() == 0
    for g, w in zip(got, want):
        np.testing.assert_array_equal(g.cpu().numpy(), w.cpu().numpy())
    assert wlib.dscale_workspace_destroy(C.c_void_p(ws)) == 0
