"""Pins for oracle/predictor.py (CPU only): closed forms, invariants and explicit loops,
none of which go through the oracle's own expressions."""
import math

import numpy as np

from oracle import predictor as OP


def test_sizes_are_the_papers():
    # 15 x 18 = 270, 15 x 64 = 960, 15 x 32 = 480, 25: 1735 ("Acceptance predictor" paragraph)
    assert OP.CONF == 18 and OP.N_POS * OP.CONF == 270
    assert OP.N_POS * OP.HID_PROJ == 960 and OP.N_POS * OP.LOGIT_PROJ == 480
    assert OP.N_FEATURES == 1735
    # 1735-64-15 with biases is the "112K-parameter predictor"
    params = 1735 * 64 + 64 + 64 * 15 + 15
    assert params == 112079 and round(params / 1000) == 112


def test_uniform_logits_closed_form():
    V = 1000
    c = OP.confidence_features(np.full(V, 2.5))
    assert c[0] == 2.5
    np.testing.assert_allclose(c[1:16], 0.0, atol=0)                # all gaps vanish
    np.testing.assert_allclose(c[16], -math.log(V), rtol=1e-13)      # log-probability of the top
    np.testing.assert_allclose(c[17], math.log(V), rtol=1e-13)       # entropy of the uniform law


def test_two_level_distribution_closed_form():
    """One logit a, the other V - 1 equal to b: softmax, entropy and gaps by hand."""
    V, a, b = 50, 3.0, -1.0
    z = np.full(V, b); z[17] = a
    c = OP.confidence_features(z)
    zsum = math.exp(a) + (V - 1) * math.exp(b)
    p_top, p_rest = math.exp(a) / zsum, math.exp(b) / zsum
    assert c[0] == a
    np.testing.assert_allclose(c[1:16], a - b, rtol=1e-15)
    np.testing.assert_allclose(c[16], math.log(p_top), rtol=1e-13)
    np.testing.assert_allclose(c[17], -(p_top * math.log(p_top) + (V - 1) * p_rest * math.log(p_rest)), rtol=1e-13)


def test_gaps_follow_the_sorted_ranks():
    z = np.array([0.5, 9.0, 7.5, -2.0, 8.0] + [float(-10 - i) for i in range(20)])
    c = OP.confidence_features(z)
    want = [9.0 - 8.0, 9.0 - 7.5, 9.0 - 0.5, 9.0 + 2.0] + [9.0 + 10 + i for i in range(11)]
    np.testing.assert_allclose(c[1:16], want, rtol=0, atol=0)
    assert (np.diff(c[1:16]) >= 0).all()


def test_shift_invariance():
    """Adding a constant to the logits moves only the top logit."""
    rng = np.random.default_rng(3)
    z = rng.normal(size=400) * 3
    p_l = rng.normal(size=(OP.LOGIT_PROJ, 400))
    c0, c1 = OP.confidence_features(z), OP.confidence_features(z + 7.25)
    np.testing.assert_allclose(c1[0], c0[0] + 7.25, rtol=1e-14)
    np.testing.assert_allclose(c1[1:], c0[1:], rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(OP.logit_projection(z + 7.25, p_l), OP.logit_projection(z, p_l), atol=1e-9)


def test_permutation_invariance_of_confidence():
    rng = np.random.default_rng(4)
    z = rng.normal(size=300)
    np.testing.assert_allclose(OP.confidence_features(z[rng.permutation(300)]), OP.confidence_features(z),
                               rtol=1e-12, atol=1e-13)


def test_entropy_against_scipy():
    from scipy.special import logsumexp
    from scipy.stats import entropy
    rng = np.random.default_rng(5)
    z = rng.normal(size=2000) * 2
    c = OP.confidence_features(z)
    np.testing.assert_allclose(c[17], entropy(np.exp(z - logsumexp(z))), rtol=1e-11)
    np.testing.assert_allclose(c[16], z.max() - logsumexp(z), rtol=1e-12)


def test_projections_by_explicit_loops():
    rng = np.random.default_rng(6)
    V, H = 37, 11
    z, h = rng.normal(size=V), rng.normal(size=H)
    p_l, p_h = rng.normal(size=(OP.LOGIT_PROJ, V)), rng.normal(size=(OP.HID_PROJ, H))
    mean = sum(z) / V
    lp = [sum(p_l[j, v] * (z[v] - mean) for v in range(V)) for j in range(OP.LOGIT_PROJ)]
    hp = [sum(p_h[j, d] * h[d] for d in range(H)) for j in range(OP.HID_PROJ)]
    np.testing.assert_allclose(OP.logit_projection(z, p_l), lp, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(OP.hidden_projection(h, p_h), hp, rtol=1e-11, atol=1e-12)


def test_feature_layout_and_batch_context():
    rng = np.random.default_rng(7)
    n, V, H = 3, 64, 8
    z, h = rng.normal(size=(n, 15, V)), rng.normal(size=(n, 15, H))
    p_h, p_l = rng.normal(size=(64, H)), rng.normal(size=(32, V))
    f = OP.features(z, h, p_h, p_l, n)
    assert f.shape == (n, 1735)
    i, p = 2, 9
    np.testing.assert_allclose(f[i, 18 * p], z[i, p].max())                            # confidence, draft order
    np.testing.assert_allclose(f[i, 270 + 64 * p: 270 + 64 * (p + 1)], p_h @ h[i, p])  # then hidden projection
    np.testing.assert_allclose(f[i, 1230 + 32 * p: 1230 + 32 * (p + 1)], p_l @ (z[i, p] - z[i, p].mean()))
    ctx = f[i, 1710:]
    assert ctx.shape == (25,) and ctx[0] == n and ctx[3] == 1.0
    assert np.count_nonzero(ctx) == 2


def test_mlp_by_explicit_loops_and_relu():
    rng = np.random.default_rng(8)
    f = rng.normal(size=(2, 1735))
    w1, b1 = rng.normal(size=(64, 1735)) * 0.05, rng.normal(size=64)
    w2, b2 = rng.normal(size=(15, 64)), rng.normal(size=15)
    out = OP.mlp(f, w1, b1, w2, b2)
    for r in range(2):
        hid = [max(0.0, sum(w1[j, x] * f[r, x] for x in range(1735)) + b1[j]) for j in range(64)]
        ref = [sum(w2[o, j] * hid[j] for j in range(64)) + b2[o] for o in range(15)]
        np.testing.assert_allclose(out[r], ref, rtol=1e-10, atol=1e-10)
    # a hidden unit that is negative everywhere contributes nothing
    w1n, b1n = -np.abs(w1), -np.abs(b1) - 1.0
    np.testing.assert_allclose(OP.mlp(np.abs(f), w1n, b1n, w2, b2), np.tile(b2, (2, 1)), atol=0)


def test_predict_zero_rows_for_dead_requests():
    rng = np.random.default_rng(9)
    n_bs, n, V, H = 4, 2, 40, 8
    z, h = rng.normal(size=(n_bs, 15, V)), rng.normal(size=(n_bs, 15, H))
    r = OP.predict(z, h, rng.normal(size=(64, H)), rng.normal(size=(32, V)), rng.normal(size=(64, 1735)) * 0.02,
                   np.zeros(64), rng.normal(size=(15, 64)), np.zeros(15), n, n_bs)
    assert r["pred_logits"].shape == (n_bs, 15) and (r["pred_logits"][n:] == 0).all()
    assert r["features"].shape == (n, 1735)
