"""GPU needle tests for the packed verify attention (Eq. 15 and the sentence after it).

One key is given a huge dot product with the query of one output row (k = 8 q, score about
90 against N(0,1) for every other key) and a recognisable value row (linspace(-2, 2)).  If that
key is visible to the row, the row's output must be that value row; if it is the first hidden
key, the row must come out as in the run without the needle (to a few bf16 ulps).  A mask that is off by
one, a dropped page or key tile, or a partial that a split-KV merge loses fails by O(1), also at
contexts of thousands of keys where an element-wise tolerance on N(0,1) data cannot see it.

Needles sit at key 0, at the last visible key ctx + j, at the first hidden key ctx + j + 1 (inside
the window, and just beyond the request's last key), on both sides of page edges, and on both
sides of EVERY 128-key tile edge of a long (request, kv-head) pair.  The persistent grid cuts the
tile list into one slice per CTA, a few tiles each for these sizes, so the sweep crosses every
cut between two CTAs and every partial of the in-kernel merge, whatever the schedule is.
Several needles share one launch: each has its own target row, and a foreign needle reaches a
row with a score of about N(0, 8^2), e^-60 of its own.
"""
import numpy as np
import pytest
import torch

from dscale_inputs import CONFIGS, small_variant
from gpu_case import SCALE, StagedRequests, assert_alloc_equal, attn_close, full_case, gpu_alloc, oracle_attn

pytestmark = pytest.mark.gpu

V_NEEDLE = np.linspace(-2.0, 2.0, 128).astype(np.float32)
CTX = [4100, 20500, 137]          # 33, 161 and 2 key tiles per pair


@pytest.fixture(scope="module")
def P():
    import paper_2609_37532_b200 as pkg
    return pkg


@pytest.fixture(scope="module")
def case():
    cfg = small_variant(CONFIGS["tiny"], n=len(CTX), seed=91, n_q_heads=8, n_kv_heads=2)
    req, alloc, kc, vc, qu, qp = full_case(cfg, n_bs=4, ctx_override=CTX, poison=True)
    return req, alloc, kc, vc, qp


def _run(P, impl, req, alloc, kc, vc, qp):
    cfg = req["cfg"]
    ws = P.VerifyWorkspace(req["n_bs"], cfg.n_q_heads, cfg.n_kv_heads)
    st = StagedRequests(req)
    assert_alloc_equal(gpu_alloc(P, ws, st), alloc)
    out = torch.full(qp.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    fn = P.verify_attn if impl == "tensor" else P.verify_attn_simt
    fn(ws, qp.cuda(), kc.cuda(), vc.cuda(), st.block_table, SCALE, out)
    torch.cuda.synchronize()
    assert ws.status() == 0
    return out.float().cpu().numpy()


def _plant(req, kc, vc, qp, alloc, i, g, t, j, h):
    """Key t of request i, kv-head g, becomes the needle of row j, q-head h."""
    pg = int(req["block_table"][i, t // 16])
    kc[pg, g, t % 16, :] = (qp[int(alloc["offset"][i]) + j, h].float() * 8.0).to(torch.bfloat16)
    vc[pg, g, t % 16, :] = torch.from_numpy(V_NEEDLE).to(torch.bfloat16)


def _visible_needles(P, impl, case, i, g, positions):
    """Plant the needles of `positions` (key indices of request i, kv-head g) in as few launches
    as the pair has rows, each for a target row that sees it; every target row must return the
    needle's value row, and the whole output must match the oracle on the same planted cache."""
    req, alloc, kc0, vc0, qp = case
    G = req["cfg"].n_q_heads // req["cfg"].n_kv_heads
    ki, oi, ci = int(alloc["k"][i]), int(alloc["offset"][i]), int(req["ctx_len"][i])
    positions = list(positions)
    while positions:
        kc, vc = kc0.clone(), vc0.clone()
        planted = []
        free_rows = [(j, h) for j in range(ki) for h in range(g * G, (g + 1) * G)]
        rest = []
        for t in positions:
            row = next(((j, h) for (j, h) in free_rows if t <= ci + j), None)
            if row is None:
                rest.append(t)
                continue
            free_rows.remove(row)
            _plant(req, kc, vc, qp, alloc, i, g, t, *row)
            planted.append((t, row))
        assert planted, f"no row of request {i} sees keys {positions}"
        positions = rest
        got = _run(P, impl, req, alloc, kc, vc, qp)
        for t, (j, h) in planted:
            err = np.abs(got[oi + j, h] - V_NEEDLE)
            assert (err <= 1e-2 + 1e-2 * np.abs(V_NEEDLE)).all(), \
                f"{impl}: needle at key {t} (tile {t // 128}, request {i}, head {g}) not returned by row " \
                f"({j}, {h}): max|d|={err.max():.3f}"
        ok, max_abs, worst = attn_close(torch.from_numpy(got), oracle_attn(req, alloc, kc, vc, qp))
        assert ok, f"{impl}: max|d|={max_abs} at {worst} with needles {planted}"


@pytest.mark.parametrize("impl", ["tensor", "simt"])
def test_needle_at_key_zero_last_visible_key_and_page_edges(P, case, impl):
    req, alloc, _, _, _ = case
    for i in range(len(CTX)):
        ki, ci = int(alloc["k"][i]), int(req["ctx_len"][i])
        edges = [0, 15, 16, ci - 1, ci, ci + ki - 1]                      # first key, first page edge, window
        edges += [t for t in (16 * 131 - 1, 16 * 131, 16 * 1277 - 1, 16 * 1277) if t < ci]    # deep page edges
        edges += [ci + j for j in range(ki)]                              # every row's own last visible key
        for g in range(2):
            _visible_needles(P, impl, case, i, g, sorted(set(edges)))


def test_needle_on_both_sides_of_every_tile_edge_of_a_long_pair(P, case):
    """161 key tiles of one pair, spread over dozens of CTAs: both sides of each of the 160 tile
    edges (and so of every cut between two CTAs' slices) on one kv-head, every fourth edge on
    the other."""
    req, alloc, _, _, _ = case
    i = 1
    n_tiles = (int(req["ctx_len"][i]) + int(alloc["k"][i]) + 127) // 128
    assert n_tiles >= 161
    edges = [128 * t + d for t in range(1, n_tiles) for d in (-1, 0)]
    _visible_needles(P, "tensor", case, i, 1, edges)
    _visible_needles(P, "tensor", case, i, 0, edges[::8] + edges[1::8])
    _visible_needles(P, "tensor", case, 0, 0, [128 * t + d for t in range(1, 33) for d in (-1, 0)])
    _visible_needles(P, "simt", case, i, 1, edges[::4] + edges[1::4])


@pytest.mark.parametrize("impl", ["tensor", "simt"])
def test_needle_at_the_first_hidden_key_changes_nothing(P, case, impl):
    req, alloc, kc0, vc0, qp = case
    ref = _run(P, impl, req, alloc, kc0, vc0, qp)
    G = req["cfg"].n_q_heads // req["cfg"].n_kv_heads
    for i in range(len(CTX)):
        ki, oi, ci = int(alloc["k"][i]), int(alloc["offset"][i]), int(req["ctx_len"][i])
        for g in range(2):
            for j in sorted({0, ki // 2, ki - 1}):
                h = g * G + (j % G)
                kc, vc = kc0.clone(), vc0.clone()
                # ctx + j + 1 is inside the window for j < k_i - 1 (loaded, masked for row j) and
                # the first key beyond the request's last one for j = k_i - 1 (never to be read)
                _plant(req, kc, vc, qp, alloc, i, g, ci + j + 1, j, h)
                got = _run(P, impl, req, alloc, kc, vc, qp)
                # (the order in which a cut pair's partials are folded may differ between two
                # launches, hence a few bf16 ulps and not bit equality; a leak is O(1))
                np.testing.assert_allclose(got[oi:oi + j + 1, g * G:(g + 1) * G], ref[oi:oi + j + 1, g * G:(g + 1) * G],
                                           rtol=2.0 ** -6, atol=1e-4,
                                           err_msg=f"{impl}: hidden key {ci + j + 1} of request {i} head {g} leaked "
                                                   f"into rows <= {j}")
                # the rows after j do see it: the whole output against the oracle on the planted cache
                ok, max_abs, worst = attn_close(torch.from_numpy(got), oracle_attn(req, alloc, kc, vc, qp))
                assert ok, f"{impl}: max|d|={max_abs} at {worst}"
