"""ctypes binding of include/dscale.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdscale.so")

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2609_37532_b200.build` "
        "(there is no fallback path)")

lib = C.CDLL(_LIB_PATH)

_vp, _i, _i64, _f, _sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t
lib.dscale_workspace_bytes.restype = _sz
lib.dscale_workspace_bytes.argtypes = [_i, _i, _i, _i, _i]
lib.dscale_workspace_init.restype = _i
lib.dscale_workspace_init.argtypes = [_vp, _sz, _i, _i, _i, _i, _i, _vp]
lib.dscale_workspace_destroy.restype = _i
lib.dscale_workspace_destroy.argtypes = [_vp]
lib.dscale_alloc_verify.restype = _i
lib.dscale_alloc_verify.argtypes = [_vp, _i, _vp, _vp, _i, _vp, _vp, _vp, _i, _i, _vp]
lib.dscale_alloc_verify_ex.restype = _i
lib.dscale_alloc_verify_ex.argtypes = [_vp, _i, _vp, _vp, _i, _vp, _vp, _vp, _i, _i, _i, _vp, _vp]
for _name in ("dscale_verify_attn", "dscale_verify_attn_simt"):
    getattr(lib, _name).restype = _i
    getattr(lib, _name).argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _f, _vp, _vp]
lib.dscale_accept.restype = _i
lib.dscale_accept.argtypes = [_vp, _i, _vp, _i64, _i, _vp, _vp, _vp, _vp, _vp, _vp]


class LayerPtrs(C.Structure):
    _fields_ = [("q", _vp), ("k_cache", _vp), ("v_cache", _vp), ("out", _vp)]


lib.dscale_step_staging_bytes.restype = _sz
lib.dscale_step_staging_bytes.argtypes = [_i, _i]
lib.dscale_verify_step_host.restype = _i
lib.dscale_verify_step_host.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _vp, _i, _i, _vp,
                                        C.POINTER(LayerPtrs), _i, _i, _i, _f, _vp, _i64, _i,
                                        _vp, _vp, _vp, _vp, _vp]
lib.dscale_verify_step_host_graph.restype = _i
lib.dscale_verify_step_host_graph.argtypes = lib.dscale_verify_step_host.argtypes
lib.dscale_verify_attn_padded.restype = _i
lib.dscale_verify_attn_padded.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _i, _i, _vp, _i, _i, _f, _vp, _vp]
lib.dscale_accept_static.restype = _i
lib.dscale_accept_static.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _i64, _i, _vp, _vp, _vp, _vp, _vp]
lib.dscale_predict_scores.restype = _i
lib.dscale_predict_scores.argtypes = [_vp, _i, _vp, _vp, C.c_int64, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.dscale_lm_head_accept.restype = _i
lib.dscale_lm_head_accept.argtypes = [_vp, _i, _vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.dscale_accept_sampling.restype = _i
lib.dscale_accept_sampling.argtypes = [_vp, _i, _vp, _i64, _i, _f, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.dscale_select_bucket.restype = _i
lib.dscale_select_bucket.argtypes = [_vp, _i, _i]
lib.dscale_ws_field.restype = _vp
lib.dscale_ws_field.argtypes = [_vp, _i, _i]
lib.dscale_launches_per_call.restype = _i
lib.dscale_launches_per_call.argtypes = [_i]

WS_FIELDS = dict(status=0, k=1, offset=2, q_start=3, q_end=4, tokens=5, positions=6, kv_refs=7,
                 row_req=8, top1=9, k0=10, n_live=11)
_ERR = {-1: "invalid argument", -2: "unsupported shape", -3: "CUDA error", -4: "workspace",
        -5: "size beyond the built-in capacity"}


class DScaleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {_ERR.get(code, 'error')} ({code})")
        self.code = code


def _check(rc: int, where: str):
    if rc != 0:
        raise DScaleError(rc, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _need(t: torch.Tensor, dtype, name: str):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")


class VerifyWorkspace:
    """The fixed-address workspace of one captured capacity n_bs."""

    def __init__(self, n_bs: int, n_q_heads: int, n_kv_heads: int, head_dim: int = 128,
                 device=None):
        device = torch.device("cuda" if device is None else device)
        self.n_bs, self.n_q_heads, self.n_kv_heads, self.head_dim = n_bs, n_q_heads, n_kv_heads, head_dim
        self.num_sms = torch.cuda.get_device_properties(device).multi_processor_count
        nbytes = lib.dscale_workspace_bytes(n_bs, n_q_heads, n_kv_heads, head_dim, self.num_sms)
        if nbytes == 0:
            raise DScaleError(-2, "dscale_workspace_bytes")
        self.nbytes = nbytes
        self.buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        with torch.cuda.device(device):
            _check(lib.dscale_workspace_init(C.c_void_p(self.ptr), nbytes, n_bs, n_q_heads,
                                             n_kv_heads, head_dim, self.num_sms, _stream()),
                   "dscale_workspace_init")

    def close(self):
        """Forget the workspace in the library (registry entry, cached step graph, tensor
        maps) and release its memory.  No work on it may be in flight."""
        if self.ptr:
            lib.dscale_workspace_destroy(C.c_void_p(self.ptr))
            self.ptr, self.buf = 0, None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def field(self, name: str) -> torch.Tensor:
        """int32 view of a workspace section (shares memory with the workspace)."""
        n_bs = self.n_bs
        sizes = dict(status=1, n_live=1, k=n_bs, k0=n_bs, offset=n_bs + 1, q_start=n_bs,
                     q_end=n_bs, tokens=8 * n_bs, positions=8 * n_bs, kv_refs=8 * n_bs,
                     row_req=8 * n_bs, top1=8 * n_bs)
        addr = lib.dscale_ws_field(C.c_void_p(self.ptr), n_bs, WS_FIELDS[name])
        start = (addr - self.buf.data_ptr())
        return self.buf[start:start + 4 * sizes[name]].view(torch.int32)

    def status(self) -> int:
        return int(self.field("status").item())


def alloc_verify(ws: VerifyWorkspace, n_live, scores, draft_tokens, ctx_len, block_table,
                 num_pages: int, scores_are_logits: bool = False, budget_rows=None, block_width: int = 16):
    """DVL allocation; a budget_rows tensor (device int32[1]) or a block width other than 16
    goes through dscale_alloc_verify_ex."""
    _need(n_live, torch.int32, "n_live"); _need(scores, torch.float32, "scores")
    _need(draft_tokens, torch.int32, "draft_tokens"); _need(ctx_len, torch.int32, "ctx_len")
    _need(block_table, torch.int32, "block_table")
    assert scores.shape == (ws.n_bs, 15) and draft_tokens.shape == (ws.n_bs, 16)
    assert ctx_len.shape == (ws.n_bs,) and block_table.shape[0] == ws.n_bs
    if budget_rows is not None or block_width != 16:
        if budget_rows is not None:
            _need(budget_rows, torch.int32, "budget_rows")
        _check(lib.dscale_alloc_verify_ex(C.c_void_p(ws.ptr), ws.n_bs, _ptr(n_live), _ptr(scores),
                                          int(scores_are_logits), _ptr(draft_tokens), _ptr(ctx_len),
                                          _ptr(block_table), block_table.shape[1], num_pages, int(block_width),
                                          _ptr(budget_rows), _stream()),
               "dscale_alloc_verify_ex")
        return
    _check(lib.dscale_alloc_verify(C.c_void_p(ws.ptr), ws.n_bs, _ptr(n_live), _ptr(scores),
                                   int(scores_are_logits), _ptr(draft_tokens), _ptr(ctx_len),
                                   _ptr(block_table), block_table.shape[1], num_pages, _stream()),
           "dscale_alloc_verify")


def _attn(fn, name, ws, q, k_cache, v_cache, block_table, sm_scale, out):
    _need(q, torch.bfloat16, "q"); _need(k_cache, torch.bfloat16, "k_cache")
    _need(v_cache, torch.bfloat16, "v_cache"); _need(out, torch.bfloat16, "out")
    _need(block_table, torch.int32, "block_table")
    assert q.shape == (8 * ws.n_bs, ws.n_q_heads, 128) and out.shape == q.shape
    assert k_cache.shape[1:] == (ws.n_kv_heads, 16, 128) and v_cache.shape == k_cache.shape
    _check(fn(C.c_void_p(ws.ptr), ws.n_bs, _ptr(q), _ptr(k_cache), _ptr(v_cache),
              _ptr(block_table), block_table.shape[1], k_cache.shape[0], ws.n_q_heads,
              ws.n_kv_heads, float(sm_scale), _ptr(out), _stream()), name)


def verify_attn(ws, q, k_cache, v_cache, block_table, sm_scale, out):
    _attn(lib.dscale_verify_attn, "dscale_verify_attn", ws, q, k_cache, v_cache, block_table,
          sm_scale, out)


def verify_attn_simt(ws, q, k_cache, v_cache, block_table, sm_scale, out):
    _attn(lib.dscale_verify_attn_simt, "dscale_verify_attn_simt", ws, q, k_cache, v_cache,
          block_table, sm_scale, out)


def accept(ws, logits, vocab: int, accept_len, next_anchor, out_tokens, out_len,
           ctx_len_inout=None):
    _need(logits, torch.float32, "logits")
    for n, t in (("accept_len", accept_len), ("next_anchor", next_anchor),
                 ("out_tokens", out_tokens), ("out_len", out_len)):
        _need(t, torch.int32, n)
    assert logits.shape[0] == 8 * ws.n_bs and out_tokens.shape == (ws.n_bs, 16)
    _check(lib.dscale_accept(C.c_void_p(ws.ptr), ws.n_bs, _ptr(logits), logits.stride(0), vocab,
                             _ptr(accept_len), _ptr(next_anchor), _ptr(out_tokens), _ptr(out_len),
                             _ptr(ctx_len_inout), _stream()), "dscale_accept")


class HostStep:
    """Whole verify step from pinned host buffers (dscale_verify_step_host).

    Holds the pinned input / output buffers, the device staging scratch and
    the per-layer pointer table; `run()` enqueues one step on the current
    stream and returns without synchronising."""

    def __init__(self, ws: VerifyWorkspace, max_pages: int, num_pages: int, layers, logits,
                 vocab: int, sm_scale: float, pinned: bool = True):
        n_bs = ws.n_bs
        self.ws, self.max_pages, self.num_pages = ws, max_pages, num_pages
        self.vocab, self.sm_scale, self.logits = vocab, float(sm_scale), logits
        pin = dict(pin_memory=pinned)       # pageable buffers take the library's copy path
        self.h_n_live = torch.zeros(1, dtype=torch.int32, **pin)
        self.h_scores = torch.zeros((n_bs, 15), dtype=torch.float32, **pin)
        self.h_draft = torch.zeros((n_bs, 16), dtype=torch.int32, **pin)
        self.h_ctx_len = torch.zeros(n_bs, dtype=torch.int32, **pin)
        self.h_block_table = torch.zeros((n_bs, max_pages), dtype=torch.int32, **pin)
        self.h_accept_len = torch.zeros(n_bs, dtype=torch.int32, **pin)
        self.h_next_anchor = torch.zeros(n_bs, dtype=torch.int32, **pin)
        self.h_out_tokens = torch.zeros((n_bs, 16), dtype=torch.int32, **pin)
        self.h_out_len = torch.zeros(n_bs, dtype=torch.int32, **pin)
        nbytes = lib.dscale_step_staging_bytes(n_bs, max_pages)
        self.staging = torch.empty(nbytes + 256, dtype=torch.uint8, device=ws.buf.device)
        self.staging_ptr = self.staging.data_ptr() + (-self.staging.data_ptr()) % 256
        self._keep = layers
        self.table = (LayerPtrs * len(layers))()
        for x, (q, kc, vc, out) in enumerate(layers):
            _need(q, torch.bfloat16, "q"); _need(kc, torch.bfloat16, "k_cache")
            _need(vc, torch.bfloat16, "v_cache"); _need(out, torch.bfloat16, "out")
            self.table[x] = LayerPtrs(q.data_ptr(), kc.data_ptr(), vc.data_ptr(), out.data_ptr())
        self.h2d_bytes = 4 + n_bs * (15 + 16 + 1 + max_pages) * 4
        self.d2h_bytes = n_bs * (1 + 1 + 16 + 1) * 4

    def run(self, graph: bool = False):
        """Enqueue one step; graph=True goes through dscale_verify_step_host_graph."""
        ws = self.ws
        fn = lib.dscale_verify_step_host_graph if graph else lib.dscale_verify_step_host
        _check(fn(
            C.c_void_p(ws.ptr), ws.n_bs, _ptr(self.h_n_live), _ptr(self.h_scores),
            _ptr(self.h_draft), _ptr(self.h_ctx_len), _ptr(self.h_block_table), self.max_pages,
            self.num_pages, C.c_void_p(self.staging_ptr), self.table, len(self.table),
            ws.n_q_heads, ws.n_kv_heads, self.sm_scale, _ptr(self.logits),
            self.logits.stride(0), self.vocab, _ptr(self.h_accept_len), _ptr(self.h_next_anchor),
            _ptr(self.h_out_tokens), _ptr(self.h_out_len), _stream()), "dscale_verify_step_host")


def accept_static(n_bs: int, n_live, k, offset, tokens, logits, vocab: int, accept_len,
                  next_anchor, out_tokens, out_len):
    """dscale_accept_static: acceptance without a workspace and without any
    allocation (the scratch is a fixed array inside the library).  For callers
    that cannot call cudaMalloc on their hot path.  Calls on one GPU must not
    overlap; make the first call on a device outside stream capture."""
    _need(logits, torch.float32, "logits")
    for n, t in (("n_live", n_live), ("k", k), ("offset", offset), ("tokens", tokens),
                 ("accept_len", accept_len), ("next_anchor", next_anchor),
                 ("out_tokens", out_tokens), ("out_len", out_len)):
        _need(t, torch.int32, n)
    _check(lib.dscale_accept_static(n_bs, _ptr(n_live), _ptr(k), _ptr(offset), _ptr(tokens),
                                    _ptr(logits), logits.stride(0), vocab, _ptr(accept_len),
                                    _ptr(next_anchor), _ptr(out_tokens), _ptr(out_len), _stream()),
           "dscale_accept_static")


def verify_attn_padded(ws, q_unpacked, k_cache, v_cache, block_table, ctx_len, sm_scale, out_unpacked):
    """The comparison baseline: unpacked W = 16, one 128-row tile per (request, q-head)."""
    _need(q_unpacked, torch.bfloat16, "q_unpacked"); _need(out_unpacked, torch.bfloat16, "out_unpacked")
    _need(k_cache, torch.bfloat16, "k_cache"); _need(v_cache, torch.bfloat16, "v_cache")
    _need(block_table, torch.int32, "block_table"); _need(ctx_len, torch.int32, "ctx_len")
    assert q_unpacked.shape == (ws.n_bs, 16, ws.n_q_heads, 128) and out_unpacked.shape == q_unpacked.shape
    _check(lib.dscale_verify_attn_padded(C.c_void_p(ws.ptr), ws.n_bs, _ptr(q_unpacked), _ptr(k_cache),
                                         _ptr(v_cache), _ptr(block_table), block_table.shape[1],
                                         k_cache.shape[0], _ptr(ctx_len), ws.n_q_heads, ws.n_kv_heads,
                                         float(sm_scale), _ptr(out_unpacked), _stream()),
           "dscale_verify_attn_padded")


class VerifyGraphPool:
    """Fixed-address graph capture and replay over a set of request capacities
    (Algorithm 2): one workspace, one set of fixed-address tensors and one
    captured CUDA graph `[alloc -> attention x L -> accept]` per bucket; a step
    picks the smallest bucket that holds the live requests (Eq. 13), writes its
    inputs into that bucket's tensors and replays its graph.  Requests beyond N
    in the bucket are sentinels.

    The KV cache (one (k, v) pair per layer) is shared by all buckets; Q, logits
    and outputs are per bucket because their shapes depend on the capacity."""

    def __init__(self, buckets, n_q_heads: int, n_kv_heads: int, max_pages: int, kv_layers,
                 vocab: int, sm_scale: float, device=None):
        self.device = torch.device("cuda" if device is None else device)
        self.buckets = sorted(int(b) for b in buckets)
        self._barr = (C.c_int32 * len(self.buckets))(*self.buckets)
        self.kv_layers, self.vocab, self.sm_scale = kv_layers, vocab, float(sm_scale)
        self.max_pages, self.num_pages = max_pages, kv_layers[0][0].shape[0]
        self.slots = {}
        for b in self.buckets:
            self.slots[b] = self._capture(b, n_q_heads, n_kv_heads)

    def _capture(self, n_bs, n_q_heads, n_kv_heads):
        dev, L = self.device, len(self.kv_layers)
        i32 = dict(dtype=torch.int32, device=dev)
        t = dict(
            ws=VerifyWorkspace(n_bs, n_q_heads, n_kv_heads, device=dev),
            n_live=torch.ones(1, **i32), scores=torch.zeros((n_bs, 15), dtype=torch.float32, device=dev),
            draft=torch.zeros((n_bs, 16), **i32), ctx_len=torch.zeros(n_bs, **i32),
            block_table=torch.zeros((n_bs, self.max_pages), **i32),
            q=[torch.zeros((8 * n_bs, n_q_heads, 128), dtype=torch.bfloat16, device=dev) for _ in range(L)],
            out=[torch.zeros((8 * n_bs, n_q_heads, 128), dtype=torch.bfloat16, device=dev) for _ in range(L)],
            logits=torch.zeros((8 * n_bs, self.vocab), dtype=torch.float32, device=dev),
            accept_len=torch.zeros(n_bs, **i32), next_anchor=torch.zeros(n_bs, **i32),
            out_tokens=torch.zeros((n_bs, 16), **i32), out_len=torch.zeros(n_bs, **i32))

        def step():
            alloc_verify(t["ws"], t["n_live"], t["scores"], t["draft"], t["ctx_len"], t["block_table"],
                         self.num_pages)
            for l, (kc, vc) in enumerate(self.kv_layers):
                verify_attn(t["ws"], t["q"][l], kc, vc, t["block_table"], self.sm_scale, t["out"][l])
            accept(t["ws"], t["logits"], self.vocab, t["accept_len"], t["next_anchor"], t["out_tokens"],
                   t["out_len"], None)

        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            step()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step()
        torch.cuda.synchronize()
        t["graph"] = g
        return t

    def select(self, n_live: int) -> int:
        b = lib.dscale_select_bucket(self._barr, len(self.buckets), int(n_live))
        if b < 0:
            raise DScaleError(b, "dscale_select_bucket")
        return b

    def slot(self, n_live: int):
        """The fixed-address tensors of the bucket a batch of n_live requests uses."""
        return self.slots[self.select(n_live)]

    def replay(self, n_live: int):
        self.slots[self.select(n_live)]["graph"].replay()


def accept_sampling(ws, logits, vocab: int, temperature: float, u_accept, u_draw, accept_len,
                    next_anchor, out_tokens, out_len, p_draft=None):
    """Prefix verification under a sampling target policy (dscale_accept_sampling)."""
    _need(logits, torch.float32, "logits"); _need(u_accept, torch.float32, "u_accept")
    _need(u_draw, torch.float32, "u_draw")
    for n, t in (("accept_len", accept_len), ("next_anchor", next_anchor),
                 ("out_tokens", out_tokens), ("out_len", out_len)):
        _need(t, torch.int32, n)
    assert u_accept.shape == (8 * ws.n_bs,) and u_draw.shape == (ws.n_bs,)
    _check(lib.dscale_accept_sampling(C.c_void_p(ws.ptr), ws.n_bs, _ptr(logits), logits.stride(0), vocab,
                                      float(temperature), _ptr(u_accept), _ptr(u_draw), _ptr(accept_len),
                                      _ptr(next_anchor), _ptr(out_tokens), _ptr(out_len), _ptr(p_draft),
                                      _stream()), "dscale_accept_sampling")


def lm_head_accept(ws, hidden, weight, accept_len, next_anchor, out_tokens, out_len,
                   ctx_len_inout=None, row_max=None):
    """Fused LM head + argmax + greedy acceptance (dscale_lm_head_accept)."""
    _need(hidden, torch.bfloat16, "hidden"); _need(weight, torch.bfloat16, "weight")
    for n, t in (("accept_len", accept_len), ("next_anchor", next_anchor),
                 ("out_tokens", out_tokens), ("out_len", out_len)):
        _need(t, torch.int32, n)
    assert hidden.shape[0] == 8 * ws.n_bs and hidden.shape[1] == weight.shape[1]
    _check(lib.dscale_lm_head_accept(C.c_void_p(ws.ptr), ws.n_bs, _ptr(hidden), _ptr(weight), hidden.shape[1],
                                     weight.shape[0], _ptr(accept_len), _ptr(next_anchor), _ptr(out_tokens),
                                     _ptr(out_len), _ptr(ctx_len_inout), _ptr(row_max), _stream()),
           "dscale_lm_head_accept")


def predict_scores(ws, n_live, draft_logits, vocab, draft_hidden, p_hidden, p_logit, w1, b1, w2, b2,
                   pred_logits, features_out=None):
    """Predictor front end (dscale_predict_scores): drafter logits / hidden states -> predLogits."""
    _need(n_live, torch.int32, "n_live"); _need(draft_logits, torch.float32, "draft_logits")
    _need(draft_hidden, torch.bfloat16, "draft_hidden"); _need(p_hidden, torch.bfloat16, "p_hidden")
    _need(p_logit, torch.bfloat16, "p_logit"); _need(pred_logits, torch.float32, "pred_logits")
    for n, t in (("w1", w1), ("b1", b1), ("w2", w2), ("b2", b2)):
        _need(t, torch.float32, n)
    assert draft_logits.shape[:2] == (ws.n_bs, 15) and draft_hidden.shape[:2] == (ws.n_bs, 15)
    assert w1.shape == (64, 1735) and w2.shape == (15, 64) and pred_logits.shape == (ws.n_bs, 15)
    _check(lib.dscale_predict_scores(C.c_void_p(ws.ptr), ws.n_bs, _ptr(n_live), _ptr(draft_logits),
                                     draft_logits.shape[2], vocab, _ptr(draft_hidden), draft_hidden.shape[2],
                                     _ptr(p_hidden), _ptr(p_logit), _ptr(w1), _ptr(b1), _ptr(w2), _ptr(b2),
                                     _ptr(pred_logits), _ptr(features_out), _stream()),
           "dscale_predict_scores")
