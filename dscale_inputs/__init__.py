"""Seeded synthetic inputs for the DScale verify step.

This module only *draws inputs*: request shapes, predictor scores, draft
tokens, paged K/V, queries and target logits with a planted acceptance
length.  It contains none of the method's arithmetic (no allocation, no
attention, no argmax) and is the one module that both the CUDA path's
tests/benchmark and the CPU oracle's tests may import.

The five named workloads stand in for the serving traces the paper measured
on (which are not available): they keep the shapes that matter for the
verify path -- W = 16 slots per request, a budget of 8 per request, Qwen3
head geometry (head_dim 128, GQA group 4), 16-token KV pages, vocabulary
151936, concurrency 4-32 -- with N(0,1) tensors and acceptance lengths from
a truncated geometric law.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

W = 16
PAGE = 16
HEAD_DIM = 128


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    n: int                    # live requests (the paper's N, "B" in the workload text)
    n_q_heads: int
    n_kv_heads: int
    vocab: int
    ctx_lo: int
    ctx_hi: int
    layers: int
    seed: int
    accept_mean: float = 4.0
    ctx_mode: str = "uniform"      # "uniform" | "bimodal" (half ctx_lo, half ctx_hi)
    score_mode: str = "uniform"    # "uniform": q_i ~ U(0.5, 0.95) | "bimodal": q_i in {0.3, 0.97}
    head_dim: int = HEAD_DIM


CONFIGS = {
    "tiny": VerifyConfig("tiny", 4, 8, 2, 1024, 64, 256, 1, 0),
    "qwen3_4b_layer": VerifyConfig("qwen3_4b_layer", 8, 32, 8, 151936, 512, 2048, 1, 1),
    "qwen3_8b_layer": VerifyConfig("qwen3_8b_layer", 16, 32, 8, 151936, 1024, 4096, 1, 2,
                                   accept_mean=5.0),
    "qwen3_8b_step": VerifyConfig("qwen3_8b_step", 32, 32, 8, 151936, 2048, 8192, 36, 3),
    "skew": VerifyConfig("skew", 32, 32, 8, 151936, 256, 16384, 1, 4,
                         ctx_mode="bimodal", score_mode="bimodal"),
}


def small_variant(cfg: VerifyConfig, **kw) -> VerifyConfig:
    return replace(cfg, **kw)


def _streams(seed: int, n: int):
    return [np.random.Generator(np.random.PCG64(s)) for s in np.random.SeedSequence(seed).spawn(n)]


def make_requests(cfg: VerifyConfig, n_bs: int | None = None, ctx_override=None) -> dict:
    """Per-request state for one step: scores, draft tokens, context lengths,
    block table, planted acceptance.  Rows n..n_bs-1 are unused capacity and
    hold harmless defaults."""
    n = cfg.n
    n_bs = n if n_bs is None else n_bs
    assert n_bs >= n
    r_ctx, r_q, r_tok, r_acc, r_perm, r_next, r_shuf = _streams(cfg.seed, 7)

    if ctx_override is not None:
        ctx = np.asarray(ctx_override, dtype=np.int64)
    elif cfg.ctx_mode == "uniform":
        ctx = r_ctx.integers(cfg.ctx_lo, cfg.ctx_hi + 1, size=n)
    else:
        ctx = np.array([cfg.ctx_lo] * (n // 2) + [cfg.ctx_hi] * (n - n // 2))
        r_shuf.shuffle(ctx)

    if cfg.score_mode == "uniform":
        qi = r_q.uniform(0.5, 0.95, size=n)
    else:
        qi = np.array([0.3] * (n // 2) + [0.97] * (n - n // 2))
        r_q.shuffle(qi)
    j = np.arange(1, W)
    scores = np.zeros((n_bs, W - 1), dtype=np.float32)
    scores[:n] = (qi[:, None] ** j[None, :]).astype(np.float32)

    draft = np.zeros((n_bs, W), dtype=np.int32)
    draft[:n] = r_tok.integers(0, cfg.vocab, size=(n, W))

    # planted accepted-candidate count: truncated geometric on 0..15
    if cfg.score_mode == "uniform":
        p_cont = np.full(n, cfg.accept_mean / (1.0 + cfg.accept_mean))
    else:
        p_cont = qi
    planted_a = np.zeros(n_bs, dtype=np.int32)
    planted_a[:n] = np.minimum(r_acc.geometric(1.0 - p_cont) - 1, W - 1)
    # the token the target emits after the accepted prefix: any token that is
    # not the candidate in slot a+1
    planted_next = np.zeros(n_bs, dtype=np.int32)
    for i in range(n):
        t = int(r_next.integers(0, cfg.vocab))
        a = int(planted_a[i])
        if a + 1 < W and t == draft[i, a + 1]:
            t = (t + 1) % cfg.vocab
        planted_next[i] = t

    pages_per_req = (ctx + W + PAGE - 1) // PAGE
    max_pages = int(-(-int(pages_per_req.max()) // 4) * 4)
    num_pages = int(pages_per_req.sum()) + 8
    perm = r_perm.permutation(num_pages)
    block_table = np.full((n_bs, max_pages), -1, dtype=np.int32)
    cur = 0
    for i in range(n):
        block_table[i, : pages_per_req[i]] = perm[cur: cur + pages_per_req[i]]
        cur += int(pages_per_req[i])
    ctx_len = np.zeros(n_bs, dtype=np.int32)
    ctx_len[:n] = ctx
    return dict(cfg=cfg, n_bs=n_bs, n_live=n, scores=scores, draft_tokens=draft,
                ctx_len=ctx_len, block_table=block_table, max_pages=max_pages,
                num_pages=num_pages, planted_a=planted_a, planted_next=planted_next,
                spare_pages=perm[cur:].copy())


def make_kv_layer(req: dict, layer: int, device: str = "cpu", poison: bool = True,
                  valid_extra: int = W):
    """K and V of one layer, bf16 [num_pages, H_kv, PAGE, D], N(0,1).

    Slots that no request owns (beyond ctx_i + valid_extra in its last pages,
    and the spare pages) are NaN when `poison` is set, so that any read past
    the visible keys shows up in the result."""
    cfg = req["cfg"]
    shape = (req["num_pages"], cfg.n_kv_heads, PAGE, cfg.head_dim)
    g = torch.Generator(device=device)
    out = []
    for which in (0, 1):
        g.manual_seed(cfg.seed * 1_000_003 + layer * 2 + which + 17)
        if device == "cpu":
            t = torch.empty(shape, dtype=torch.bfloat16)
            step = 2048
            for p0 in range(0, shape[0], step):
                p1 = min(shape[0], p0 + step)
                t[p0:p1] = torch.randn((p1 - p0,) + shape[1:], generator=g,
                                       dtype=torch.float32).to(torch.bfloat16)
        else:
            t = torch.randn(shape, generator=g, dtype=torch.bfloat16, device=device)
        out.append(t)
    if poison:
        bt = req["block_table"]
        nan = float("nan")
        for t in out:
            for i in range(req["n_live"]):
                n_valid = int(req["ctx_len"][i]) + valid_extra
                n_pages = (int(req["ctx_len"][i]) + W + PAGE - 1) // PAGE
                for p in range(n_valid // PAGE, n_pages):
                    lo = max(0, n_valid - p * PAGE)
                    if lo < PAGE:
                        t[int(bt[i, p]), :, lo:, :] = nan
            if len(req["spare_pages"]):
                t[torch.as_tensor(req["spare_pages"], dtype=torch.long, device=t.device)] = nan
    return out[0], out[1]


def make_q_unpacked(req: dict, layer: int, device: str = "cpu") -> torch.Tensor:
    """Query rows of every slot, bf16 [n_bs, W, H_q, D], N(0,1)."""
    cfg = req["cfg"]
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + 7919 * (layer + 1))
    shape = (req["n_bs"], W, cfg.n_q_heads, cfg.head_dim)
    return torch.randn(shape, generator=g, dtype=torch.float32, device=device).to(torch.bfloat16)


def make_logits_unpacked(req: dict, device: str = "cpu") -> torch.Tensor:
    """Target logits of every slot, fp32 [n_bs, W, vocab]: N(0,1) noise with
    the planted acceptance.  Slot j's row predicts slot j+1: for j < a_i the
    candidate of slot j+1 is boosted by 8, at j = a_i the planted successor
    is.  Afterwards each planted token is checked to be the strict row
    maximum and lifted above it if the noise happened to win."""
    cfg = req["cfg"]
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + 104729)
    n_bs = req["n_bs"]
    logits = torch.randn((n_bs, W, cfg.vocab), generator=g, dtype=torch.float32, device=device)
    draft = req["draft_tokens"]
    for i in range(req["n_live"]):
        a = int(req["planted_a"][i])
        for j in range(a + 1):
            tok = int(draft[i, j + 1]) if j < a else int(req["planted_next"][i])
            row = logits[i, j]
            row[tok] += 8.0
            others = row.clone()
            others[tok] = float("-inf")
            top_other = float(others.max())
            if not float(row[tok]) > top_other:
                row[tok] = top_other + 1.0
    return logits


def make_lm_head_unpacked(req: dict, hidden_dim: int, device: str = "cpu"):
    """Inputs of the LM head: (weight bf16 [vocab, hidden_dim], hidden bf16
    [n_bs, W, hidden_dim]).  Weights are N(0,1); every slot's final hidden
    state is N(0, 0.25 / hidden_dim) noise (logits of standard deviation
    0.5), and the slots that carry the planted acceptance (the same ones
    make_logits_unpacked boosts) additionally point
    along the weight row of their planted token, scaled so that token's logit
    is about 8 while all others stay below about 3."""
    cfg = req["cfg"]
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + 130363)
    n_bs = req["n_bs"]
    weight = torch.randn((cfg.vocab, hidden_dim), generator=g, dtype=torch.float32,
                         device=device).to(torch.bfloat16)
    hidden = (0.5 / hidden_dim ** 0.5) * torch.randn((n_bs, W, hidden_dim), generator=g, dtype=torch.float32, device=device)
    draft = req["draft_tokens"]
    for i in range(req["n_live"]):
        a = int(req["planted_a"][i])
        for j in range(a + 1):
            tok = int(draft[i, j + 1]) if j < a else int(req["planted_next"][i])
            w = weight[tok].float()
            hidden[i, j] += 8.0 * w / float(w @ w)
    return weight, hidden.to(torch.bfloat16)


def make_predictor_inputs(req: dict, hidden_dim: int, device: str = "cpu") -> dict:
    """Inputs of the acceptance-predictor front end, shape-faithful with seeded
    random parameters (the trained predictor and the fixed projections are not
    published).  Drafter logits fp32 [n_bs, 15, ld] (ld = vocab rounded up to a
    multiple of 4, padding NaN): N(-3, 2^2) with the drafted token of each
    position lifted by 6, so it is the drafter's top-1 as in the paper's
    deterministic drafter; drafter hidden states bf16 [n_bs, 15, hidden_dim]
    N(0,1); fixed projections bf16, N(0, 1/hidden_dim) and N(0, 1/vocab) with a
    common offset of 0.5/vocab (so the centring term matters); perceptron
    weights fp32 with fan-in scaling, biases N(0, 0.25)."""
    cfg = req["cfg"]
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + 15485863)
    n_bs, V = req["n_bs"], cfg.vocab
    ld = (V + 3) // 4 * 4
    kw = dict(generator=g, dtype=torch.float32, device=device)
    logits = torch.full((n_bs, W - 1, ld), float("nan"), dtype=torch.float32, device=device)
    logits[:, :, :V] = torch.randn((n_bs, W - 1, V), **kw) * 2.0 - 3.0
    draft = torch.as_tensor(req["draft_tokens"]).to(device).long()
    idx = draft[:, 1:].unsqueeze(-1)                                   # candidate of slot p + 1
    logits.scatter_add_(2, idx, torch.full(idx.shape, 6.0, dtype=torch.float32, device=device))
    hidden = torch.randn((n_bs, W - 1, hidden_dim), **kw).to(torch.bfloat16)
    p_hidden = (torch.randn((64, hidden_dim), **kw) / hidden_dim ** 0.5).to(torch.bfloat16)
    p_logit = (torch.randn((32, V), **kw) / V ** 0.5 + 0.5 / V).to(torch.bfloat16)
    w1 = torch.randn((64, 1735), **kw) / 1735 ** 0.5
    b1 = torch.randn((64,), **kw) * 0.5
    w2 = torch.randn((15, 64), **kw) / 8.0
    b2 = torch.randn((15,), **kw) * 0.5
    return dict(draft_logits=logits, draft_hidden=hidden, p_hidden=p_hidden, p_logit=p_logit,
                w1=w1, b1=b1, w2=w2, b2=b2, ld=ld)


def rows_to_packed(unpacked: torch.Tensor, k, offset, n_live: int, m_bs: int,
                   fill: float = 0.0) -> torch.Tensor:
    """Lay the first k_i slot rows of each request at rows offset_i .. of a
    [m_bs, ...] tensor: how the upstream model hands rows to the verify path."""
    out = torch.full((m_bs,) + tuple(unpacked.shape[2:]), fill, dtype=unpacked.dtype,
                     device=unpacked.device)
    for i in range(int(n_live)):
        ki, oi = int(k[i]), int(offset[i])
        out[oi:oi + ki] = unpacked[i, :ki]
    return out


def planted_expectation(req: dict, k) -> dict:
    """What acceptance must return for lengths k, from the planted truth:
    a_out = min(a_planted, k_i - 1); the successor is the next candidate if
    the window was cut before the planted rejection, else the planted token."""
    n_bs, n = req["n_bs"], req["n_live"]
    accept_len = np.zeros(n_bs, dtype=np.int32)
    next_anchor = np.full(n_bs, -1, dtype=np.int32)
    for i in range(n):
        a_pl = int(req["planted_a"][i])
        a = min(a_pl, int(k[i]) - 1)
        accept_len[i] = a
        next_anchor[i] = req["draft_tokens"][i, a + 1] if a < a_pl else req["planted_next"][i]
    return dict(accept_len=accept_len, next_anchor=next_anchor)
