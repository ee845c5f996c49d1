"""Helpers shared by the GPU parity tests: stage a seeded case on the device,
run the library through its C ABI, run the oracle on the same inputs."""
from __future__ import annotations

import numpy as np
import torch

from dscale_inputs import (make_kv_layer, make_logits_unpacked, make_q_unpacked, make_requests,
                           rows_to_packed)
from oracle import accept as OC
from oracle import dvl_alloc as OA
from oracle import verify_attn as OV

SCALE = 1.0 / float(np.sqrt(128.0))
ALLOC_FIELDS = ("k", "k0", "offset", "q_start", "q_end", "tokens", "positions", "kv_refs",
                "row_req")


def dev(x, dtype=None):
    t = torch.as_tensor(x)
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


class StagedRequests:
    """Device copies of one step's staged inputs (fixed addresses)."""

    def __init__(self, req):
        self.req = req
        self.n_live = dev(np.array([req["n_live"]], dtype=np.int32))
        self.scores = dev(req["scores"])
        self.draft = dev(req["draft_tokens"])
        self.ctx_len = dev(req["ctx_len"])
        self.block_table = dev(req["block_table"])

    def load(self, req):
        """Overwrite in place (same addresses) with another step's inputs."""
        self.req = req
        self.n_live.copy_(torch.as_tensor(np.array([req["n_live"]], dtype=np.int32)))
        self.scores.copy_(torch.as_tensor(req["scores"]))
        self.draft.copy_(torch.as_tensor(req["draft_tokens"]))
        self.ctx_len.copy_(torch.as_tensor(req["ctx_len"]))
        self.block_table.copy_(torch.as_tensor(req["block_table"]))


def oracle_alloc(req, logits_mode=False, budget=None, block_width=16):
    W = block_width
    return OA.dvl_alloc(req["n_bs"], req["n_live"], req["scores"][:, : W - 1], req["draft_tokens"][:, :W],
                        req["ctx_len"], req["block_table"], logits_mode=logits_mode, W=W, budget=budget,
                        capacity=8 * req["n_bs"])


def gpu_alloc(P, ws, st: StagedRequests, logits_mode=False, budget=None, block_width=16):
    b = None if budget is None else torch.tensor([budget], dtype=torch.int32, device="cuda")
    P.alloc_verify(ws, st.n_live, st.scores, st.draft, st.ctx_len, st.block_table,
                   st.req["num_pages"], scores_are_logits=logits_mode, budget_rows=b, block_width=block_width)
    torch.cuda.synchronize()
    return {f: ws.field(f).cpu().numpy().copy() for f in ALLOC_FIELDS}


def assert_alloc_equal(got, exp):
    for f in ALLOC_FIELDS:
        np.testing.assert_array_equal(got[f], exp[f], err_msg=f"allocation field {f}")


def oracle_attn(req, alloc, kc, vc, qp, dtype=np.float32):
    cfg = req["cfg"]
    return OV.verify_attn(qp.float().numpy(), kc.float().numpy(), vc.float().numpy(),
                          req["block_table"], req["ctx_len"], alloc["k"], alloc["offset"],
                          req["n_live"], cfg.n_q_heads, cfg.n_kv_heads, SCALE, dtype=dtype)


ROW_REL_L2 = 8e-3      # per (row, head) output vector: ||gpu - ref||_2 <= ROW_REL_L2 ||ref||_2 + ROW_ABS_L2
ROW_ABS_L2 = 2e-4


def attn_stats(got: np.ndarray, ref: np.ndarray) -> dict:
    """Error figures of an attention output against the oracle: max abs, max rel over
    |ref| > 1e-2, ||d||_2 / ||ref||_2 over everything, and the worst per-(row, head) vector."""
    err = np.abs(got - ref)
    big = np.abs(ref) > 1e-2
    num = np.sqrt((err.astype(np.float64) ** 2).sum(axis=-1))
    den = np.sqrt((ref.astype(np.float64) ** 2).sum(axis=-1))
    row_excess = num - (ROW_REL_L2 * den + ROW_ABS_L2)
    return dict(max_abs=float(err.max()),
                max_rel=float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0,
                rel_l2=float(np.sqrt((num ** 2).sum() / max((den ** 2).sum(), 1e-300))),
                worst_row_rel_l2=float((num / np.maximum(den, 1e-30))[den > 1e-3].max()) if (den > 1e-3).any() else 0.0,
                row_excess=row_excess)


def attn_close(got_bf16: torch.Tensor, ref: np.ndarray, atol=1e-2, rtol=1e-2):
    """The parity bar for bf16 attention outputs.  Per element: |gpu - ref| <= max(atol, rtol |ref|)
    (1e-2 absolute or 1e-2 relative, whichever is larger: tighter than the sum of the two).
    Per (row, head) output vector: ||gpu - ref||_2 <= 8e-3 ||ref||_2 + 2e-4.  The vector bound is the
    sharp one: with N(0,1) inputs and thousands of keys an output element is a few 1e-2, bf16
    rounding of the probabilities and of the result costs about 2e-3 of the vector's norm, while a
    dropped 16-key page shifts a vector by several per cent of its norm.
    Returns (ok, max_abs, worst_index) so a failure can say where."""
    got = got_bf16.float().cpu().numpy()
    if not np.isfinite(got).all():
        bad = np.argwhere(~np.isfinite(got))[0]
        return False, float("nan"), tuple(bad)
    err = np.abs(got - ref)
    lim = np.maximum(atol, rtol * np.abs(ref))
    st = attn_stats(got, ref)
    if (st["row_excess"] > 0).any():
        worst = np.unravel_index(np.argmax(st["row_excess"]), st["row_excess"].shape)
        return False, float(err.max()), tuple(int(x) for x in worst) + (-1,)
    worst = np.unravel_index(np.argmax(err - lim), err.shape)
    return bool((err <= lim).all()), float(err.max()), tuple(int(x) for x in worst)


def full_case(cfg, n_bs=None, layer=0, poison=True, valid_extra=None, ctx_override=None):
    """Requests + oracle allocation + one layer of K/V/Q (CPU tensors)."""
    req = make_requests(cfg, n_bs=n_bs, ctx_override=ctx_override)
    alloc = oracle_alloc(req)
    if valid_extra is None:
        kc, vc = make_kv_layer(req, layer, poison=poison)
    else:
        kc, vc = make_kv_layer(req, layer, poison=poison, valid_extra=valid_extra)
    qu = make_q_unpacked(req, layer)
    qp = rows_to_packed(qu, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"])
    return req, alloc, kc, vc, qu, qp


def poison_hidden_slots(req, alloc, kc, vc):
    """NaN every cache slot at logical position >= ctx_i + k_i (what the packed
    path may never touch, even though the window's 16 slots were written)."""
    for i in range(req["n_live"]):
        first_hidden = int(req["ctx_len"][i]) + int(alloc["k"][i])
        for t in range(first_hidden, int(req["ctx_len"][i]) + 16):
            pg = int(req["block_table"][i, t // 16])
            kc[pg, :, t % 16, :] = float("nan")
            vc[pg, :, t % 16, :] = float("nan")


def oracle_accept(req, alloc, logits_packed: torch.Tensor, with_ctx=False):
    cfg = req["cfg"]
    return OC.accept(logits_packed.numpy(), cfg.vocab, alloc["tokens"], alloc["k"],
                     alloc["offset"], req["n_live"], req["n_bs"],
                     ctx_len=req["ctx_len"] if with_ctx else None)


def gpu_accept(P, ws, logits_dev, vocab, n_bs, ctx_len_dev=None):
    outs = dict(accept_len=torch.full((n_bs,), -7, dtype=torch.int32, device="cuda"),
                next_anchor=torch.full((n_bs,), -7, dtype=torch.int32, device="cuda"),
                out_tokens=torch.full((n_bs, 16), -7, dtype=torch.int32, device="cuda"),
                out_len=torch.full((n_bs,), -7, dtype=torch.int32, device="cuda"))
    P.accept(ws, logits_dev, vocab, outs["accept_len"], outs["next_anchor"], outs["out_tokens"],
             outs["out_len"], ctx_len_dev)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in outs.items()}
    res["top1"] = ws.field("top1").cpu().numpy().copy()
    return res
