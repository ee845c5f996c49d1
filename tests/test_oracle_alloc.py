"""Pins for oracle/dvl_alloc.py (CPU only).

Each test fixes the oracle to something other than itself: numbers the paper
prints, closed forms, exhaustive enumeration, or an independent sort-based
formulation of the greedy loop.
"""
import itertools

import numpy as np
import pytest

from conftest import read_golden
from dscale_inputs import CONFIGS, make_requests
from oracle import dvl_alloc as O

F32 = np.float32


def _scores_from_q(q, W=16):
    j = np.arange(1, W)
    return (np.asarray(q, dtype=np.float64)[:, None] ** j[None, :]).astype(np.float32)


def _dummy_fields(n_bs, max_pages=4, ctx=5):
    draft = np.arange(n_bs * 16, dtype=np.int32).reshape(n_bs, 16) + 100
    ctx_len = np.full(n_bs, ctx, dtype=np.int32)
    bt = (np.arange(n_bs * max_pages, dtype=np.int32).reshape(n_bs, max_pages) * 7 + 3) % (n_bs * max_pages)
    return draft, ctx_len, bt


# ---------------------------------------------------------------- Eq. 6 / 7
def test_seed_worked_example_from_paper():
    g = read_golden("eq7_seed_example.txt")
    # six ones and one 0.2 sum to 6.2
    s = [1.0] * 6 + [0.2] + [0.0] * 8
    q = O.prefix_scores(s)
    assert abs(float(sum(q[1:])) - g["l_hat"][0]) < 1e-6
    assert O.seed_length(q) == g["k0"][0]


@pytest.mark.parametrize("q,k0", [(0.3, 1), (0.5, 1), (0.7, 2), (0.8, 4), (0.9, 7),
                                  (0.95, 10), (0.97, 12)])
def test_seed_closed_form_geometric_scores(q, k0):
    # l_hat = q (1 - q^15) / (1 - q) for p_j = q^j; the rounding is far from .5
    closed = q * (1 - q ** 15) / (1 - q)
    assert min(16, max(1, int(np.floor(closed + 0.5)))) == k0
    row = _scores_from_q([q])[0]
    assert O.seed_length(O.prefix_scores(row)) == k0


def test_seed_clipping():
    assert O.seed_length(O.prefix_scores([0.0] * 15)) == 1          # never below the anchor
    assert O.seed_length(O.prefix_scores([1.0] * 15)) == 15         # 15 draft scores -> 15, not 16
    assert O.seed_length(O.prefix_scores([0.49] + [0.0] * 14)) == 1
    assert O.seed_length(O.prefix_scores([0.5] + [0.0] * 14)) == 1  # floor(0.5+0.5)=1
    assert O.seed_length(O.prefix_scores([1.0, 0.5] + [0.0] * 13)) == 2  # 1.5 rounds half up


def test_round_half_up_not_half_even():
    # l_hat = 2.5 exactly -> 3 (half-even would give 2)
    q = O.prefix_scores([1.0, 1.0, 0.5] + [0.0] * 12)
    assert O.seed_length(q) == 3


def test_cummin_on_non_monotone_scores():
    s = [0.9, 0.95, 0.4, 0.8, 0.1] + [0.5] * 10
    q = O.prefix_scores(s)
    hand = [1.0, 0.9, 0.9, 0.4, 0.4] + [0.1] * 11
    np.testing.assert_array_equal(q, np.asarray(hand, dtype=np.float32))
    assert all(q[j] >= q[j + 1] for j in range(15))


def test_sigmoid_pins():
    assert O.sigmoid_f32(0.0) == F32(0.5)
    for x in (0.3, 1.7, 5.0, 11.0):
        assert abs(float(O.sigmoid_f32(x)) + float(O.sigmoid_f32(-x)) - 1.0) < 2e-7
    assert O.sigmoid_f32(40.0) == F32(1.0)
    assert float(O.sigmoid_f32(-40.0)) < 1e-17
    # logits mode is sigmoid then the same path
    x = np.array([2.0, 1.0, 3.0, -1.0] + [0.0] * 11)
    q = O.prefix_scores(x, logits_mode=True)
    p = 1 / (1 + np.exp(-x))
    np.testing.assert_allclose(q[1:], np.minimum.accumulate(p), rtol=1e-6)


# ------------------------------------------------------- worked allocation
def _fig5_scores():
    rows = [
        [1, 1, 1, 1, 0.8, 0.2],              # sum 5  -> k0 5, next-slot score q_5 = 0.8
        [1] * 9 + [0.6, 0.4],                # sum 10 -> k0 10, q_10 = 0.6
        [1] * 6 + [0.7, 0.3],                # sum 7  -> k0 7,  q_7 = 0.7
        [1] * 8 + [0.5, 0.5],                # sum 9  -> k0 9,  q_9 = 0.5
    ]
    s = np.zeros((4, 15), dtype=np.float32)
    for i, r in enumerate(rows):
        s[i, : len(r)] = r
    return s


def test_fig5_worked_allocation():
    g = read_golden("fig5_allocation_example.txt")
    s = _fig5_scores()
    draft, ctx_len, bt = _dummy_fields(4)
    r = O.dvl_alloc(4, 4, s, draft, ctx_len, bt)
    assert list(r["k0"]) == g["k0"]
    assert r["m_live"] == g["budget"][0]
    assert list(r["k"]) == g["k"]
    assert list(r["offset"][:4]) == g["offset"]
    assert r["offset"][4] == g["end"][0]
    assert r["n_updates"] == 1


def test_challenge3_boundaries():
    g = read_golden("challenge3_boundaries.txt")
    assert O.offsets_of(g["k_a"])[:-1] == g["offset_a"]
    assert O.offsets_of(g["k_b"])[:-1] == g["offset_b"]
    assert O.offsets_of(g["k_a"])[-1] == O.offsets_of(g["k_b"])[-1] == g["total"][0]


# ------------------------------------------------------------- invariants
def _random_scores(rng, n, monotone):
    if monotone:
        return _scores_from_q(rng.uniform(0.05, 0.995, size=n))
    return rng.uniform(0, 1, size=(n, 15)).astype(np.float32)


@pytest.mark.parametrize("seed", range(12))
def test_budget_and_pack_invariants(seed):
    rng = np.random.default_rng(seed)
    n_bs = int(rng.integers(1, 40))
    n = int(rng.integers(1, n_bs + 1))
    s = _random_scores(rng, n_bs, monotone=bool(seed % 2))
    draft, _, _ = _dummy_fields(n_bs)
    max_pages = 8
    ctx_len = rng.integers(0, max_pages * 16 - 16, size=n_bs).astype(np.int32)
    bt = rng.permutation(n_bs * max_pages).astype(np.int32).reshape(n_bs, max_pages)
    r = O.dvl_alloc(n_bs, n, s, draft, ctx_len, bt)
    k, off = r["k"], r["offset"]
    assert k[:n].sum() == 8 * n                                   # Eq. 3
    assert ((k[:n] >= 1) & (k[:n] <= 16)).all()
    assert r["n_updates"] == abs(8 * n - int(r["k0"].sum())) <= 7 * n   # Prop. 1, update bound
    assert off[0] == 0 and off[n] == 8 * n
    assert (np.diff(off[: n + 1]) == k[:n]).all()
    assert (k[n:] == 0).all() and (off[n + 1:] == 8 * n).all()   # sentinels
    # every live slot hit exactly once, fields are the first k_i entries
    seen = np.zeros(8 * n_bs, dtype=int)
    for i in range(n):
        for j in range(k[i]):
            sl = off[i] + j
            seen[sl] += 1
            assert r["tokens"][sl] == draft[i, j]
            assert r["positions"][sl] == ctx_len[i] + j
            t = ctx_len[i] + j
            assert r["kv_refs"][sl] == bt[i, t // 16] * 16 + t % 16
            assert r["row_req"][sl] == i
    assert (seen[: 8 * n] == 1).all() and (seen[8 * n:] == 0).all()
    # tail placeholders: token 0, position 0, request 0's first KV ref
    first_ref = bt[0, ctx_len[0] // 16] * 16 + ctx_len[0] % 16
    assert (r["tokens"][8 * n:] == 0).all() and (r["positions"][8 * n:] == 0).all()
    assert (r["kv_refs"][8 * n:] == first_ref).all() and (r["row_req"][8 * n:] == -1).all()
    assert (r["q_start"] == off[:-1]).all() and (r["q_end"] == off[:-1] + k).all()


# -------------------------------------------------- Proposition 1, brute force
def _brute_best(Q, k0, budget, W, grow):
    n = len(k0)
    best = -1.0
    for ks in itertools.product(range(1, W + 1), repeat=n):
        if sum(ks) != budget:
            continue
        if grow and any(ks[i] < k0[i] for i in range(n)):
            continue
        if (not grow) and any(ks[i] > k0[i] for i in range(n)):
            continue
        best = max(best, O.prefix_objective(Q, ks))
    return best


@pytest.mark.parametrize("seed", range(10))
def test_prop1_bruteforce_other_budgets(seed):
    """Eq. 9 for totals other than (W/2) N: the greedy result is optimal among all allocations
    reachable by only growing (or only shrinking) the seeds, for every budget in [N, W N]."""
    rng = np.random.default_rng(900 + seed)
    W, n = 5, 4
    s = np.sort(rng.uniform(0, 1, size=(n, W - 1)), axis=1)[:, ::-1].astype(np.float32)
    if seed % 2 == 0:
        s = np.round(s * 4) / 4
    Q = np.stack([O.prefix_scores(s[i], W=W) for i in range(n)])
    k0 = [O.seed_length(Q[i], W=W) for i in range(n)]
    for budget in range(n, W * n + 1):
        k, upd = O.budget_adjust(Q, k0, budget, W=W)
        assert sum(k) == budget and upd == abs(budget - sum(k0)) and all(1 <= x <= W for x in k)
        d0 = budget - sum(k0)
        if d0 == 0:
            assert k == k0
        else:
            best = _brute_best(Q, k0, budget, W, grow=d0 > 0)
            assert abs(O.prefix_objective(Q, k) - best) < 1e-9


@pytest.mark.parametrize("seed", range(10))
def test_prop1_bruteforce_small_W(seed):
    rng = np.random.default_rng(100 + seed)
    W, n = 6, 4
    s = np.sort(rng.uniform(0, 1, size=(n, W - 1)), axis=1)[:, ::-1].astype(np.float32)
    if seed % 3 == 0:                       # plateaus and cross-request ties
        s = np.round(s * 4) / 4
    Q = np.stack([O.prefix_scores(s[i], W=W) for i in range(n)])
    k0 = [O.seed_length(Q[i], W=W) for i in range(n)]
    budget = (W // 2) * n
    k, upd = O.budget_adjust(Q, k0, budget, W=W)
    assert sum(k) == budget and upd == abs(budget - sum(k0))
    d0 = budget - sum(k0)
    if d0 == 0:
        assert k == k0
    else:
        best = _brute_best(Q, k0, budget, W, grow=d0 > 0)
        assert abs(O.prefix_objective(Q, k) - best) < 1e-9
        for i in range(n):
            assert (k[i] >= k0[i]) if d0 > 0 else (k[i] <= k0[i])


@pytest.mark.parametrize("seed", range(4))
def test_prop1_bruteforce_full_W_three_requests(seed):
    rng = np.random.default_rng(200 + seed)
    qs = rng.uniform(0.3, 0.99, size=3)
    if seed == 3:
        qs = np.array([0.99, 0.985, 0.98])        # seeds 14-15 each: forces the shrink branch
    s = _scores_from_q(qs)
    Q = np.stack([O.prefix_scores(s[i]) for i in range(3)])
    k0 = [O.seed_length(Q[i]) for i in range(3)]
    k, _ = O.budget_adjust(Q, k0, 24)
    d0 = 24 - sum(k0)
    if seed == 3:
        assert d0 < 0
    if d0 != 0:
        best = _brute_best(Q, k0, 24, 16, grow=d0 > 0)
        assert abs(O.prefix_objective(Q, k) - best) < 1e-9


# ------------------------------------- independent formulation: rank select
def _rank_select(Q, k0, budget, W=16):
    """The greedy loop restated as a selection from one sorted list: growing
    takes the first delta of {(i,j): k0_i <= j < W} in (q desc, i asc, j asc)
    order; shrinking removes the first |delta| of {(i,j): 1 <= j < k0_i} in
    (q asc, i asc, j desc) order.  Written with numpy lexsort only."""
    n = len(k0)
    d = budget - sum(k0)
    k = list(k0)
    if d > 0:
        c = [(i, j) for i in range(n) for j in range(k0[i], W)]
        keys = np.lexsort(([j for _, j in c], [i for i, _ in c], [-float(Q[i][j]) for i, j in c]))
        for t in keys[:d]:
            k[c[t][0]] += 1
    elif d < 0:
        c = [(i, j) for i in range(n) for j in range(1, k0[i])]
        keys = np.lexsort(([-j for _, j in c], [i for i, _ in c], [float(Q[i][j]) for i, j in c]))
        for t in keys[:-d]:
            k[c[t][0]] -= 1
    return k


@pytest.mark.parametrize("seed", range(30))
def test_serial_loop_equals_rank_select(seed):
    rng = np.random.default_rng(300 + seed)
    n = int(rng.integers(1, 65))
    mode = seed % 4
    if mode == 0:
        s = _scores_from_q(rng.uniform(0.05, 0.995, size=n))
    elif mode == 1:
        s = _scores_from_q(rng.choice([0.3, 0.97, 0.99], size=n))       # heavy ties
    elif mode == 2:
        s = (np.round(rng.uniform(0, 1, size=(n, 15)) * 8) / 8).astype(np.float32)
    else:
        s = _scores_from_q(rng.uniform(0.96, 0.999, size=n))              # shrink
    Q = np.stack([O.prefix_scores(s[i]) for i in range(n)])
    k0 = [O.seed_length(Q[i]) for i in range(n)]
    k, _ = O.budget_adjust(Q, k0, 8 * n)
    assert k == _rank_select(Q, k0, 8 * n)


# ----------------------------------------------------------- special cases
def test_all_equal_scores_round_robin_by_index():
    # all scores 0.5 -> every q_j = 0.5, seed floor(7.5+0.5)=8 -> delta 0
    s = np.full((5, 15), 0.5, dtype=np.float32)
    Q = np.stack([O.prefix_scores(r) for r in s])
    assert [O.seed_length(q) for q in Q] == [8] * 5
    # with equal scores and a surplus of 3 slots the lowest index takes all three
    # (its next-slot score stays tied and index 0 keeps winning)
    k, upd = O.budget_adjust(Q, [7, 8, 8, 8, 6], 40)
    assert k == [10, 8, 8, 8, 6] and upd == 3
    k, upd = O.budget_adjust(Q, [9, 9, 9, 8, 8], 40)
    assert k == [6, 9, 9, 8, 8] and upd == 3


def test_skew_workload_closed_form():
    # q in {0.3, 0.97}: seeds 1 and 12 (sum 208 at N=32), surplus 48 = 16 * 3 goes
    # to the sixteen 0.97-requests because 0.97^15 > 0.3: they end at 15, others at 1
    req = make_requests(CONFIGS["skew"])
    r = O.dvl_alloc(32, 32, req["scores"], req["draft_tokens"], req["ctx_len"], req["block_table"])
    hi = req["scores"][:, 0] > 0.5
    assert hi.sum() == 16
    assert (r["k0"][hi] == 12).all() and (r["k0"][~hi] == 1).all()
    assert (r["k"][hi] == 15).all() and (r["k"][~hi] == 1).all()
    assert r["k"].sum() == 256


def test_forced_shrink_branch():
    s = _scores_from_q([0.99, 0.99, 0.2, 0.99])
    draft, ctx_len, bt = _dummy_fields(4)
    r = O.dvl_alloc(4, 4, s, draft, ctx_len, bt)
    assert list(r["k0"]) == [14, 14, 1, 14] and r["k"].sum() == 32
    # 11 removals, always the smallest last-slot score, lowest index first among
    # equals: the three 0.99-requests are trimmed in turn 0,1,3,0,1,3,...
    assert list(r["k"]) == [10, 10, 1, 11]
    assert r["n_updates"] == 11


def test_sentinel_requests_ignored():
    rng = np.random.default_rng(7)
    s = _random_scores(rng, 8, True)
    draft, ctx_len, bt = _dummy_fields(8)
    a = O.dvl_alloc(8, 5, s, draft, ctx_len, bt)
    s2 = s.copy()
    s2[5:] = 0.123                                  # capacity rows must not matter
    b = O.dvl_alloc(8, 5, s2, draft, ctx_len, bt)
    for key in ("k", "offset", "tokens", "positions", "kv_refs", "row_req"):
        np.testing.assert_array_equal(a[key], b[key])
