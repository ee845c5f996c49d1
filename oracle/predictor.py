"""Oracle: acceptance-predictor front end (features and MLP), by the definition.

TEST INFRASTRUCTURE ONLY -- see the package docstring.

"Acceptance predictor" paragraph, Eq. 4 (features) and Eq. 5 (predictor).  Per
request, the 15 new draft positions each contribute 18 confidence values
computed from the drafter's logits z at that position, in this order:

    [ top logit,
      top - (rank-r logit) for r = 2..16            (15 gaps, >= 0),
      log-probability of the top token  = top - logsumexp(z),
      entropy = - sum_v p_v ln p_v,  p = softmax(z) ]

(270 values, position-major: "in draft order").  A fixed 64 x H matrix maps
each position's hidden-state vector to 64 values (960), a fixed 32 x V matrix
maps each position's mean-centred logit vector z - mean(z) to 32 values (480),
and the 25-value batch context holds the live count N in entry 0 and the
initial-state flag 1 in entry 3.  Concatenated in the order confidence,
hidden projection, logit projection, batch context: 1735 features.  The
predictor is a 1735-64-15 perceptron with ReLU and biases (112,079
parameters, the paper's "112K"); its 15 outputs are the predLogits that
Algorithm 1 turns into scores with a sigmoid.

All arithmetic is binary64 on the given inputs, one position at a time.
"""
from __future__ import annotations

import numpy as np

N_POS = 15            # new draft positions per request (W - 1)
N_TOP = 16            # ranks that enter the confidence features
CONF = 1 + (N_TOP - 1) + 1 + 1          # 18
HID_PROJ = 64
LOGIT_PROJ = 32
BATCH_CTX = 25
N_FEATURES = N_POS * CONF + N_POS * HID_PROJ + N_POS * LOGIT_PROJ + BATCH_CTX   # 1735
MLP_HIDDEN = 64


def confidence_features(z: np.ndarray) -> np.ndarray:
    """The 18 confidence values of one position from its logits z [V]."""
    z = np.asarray(z, dtype=np.float64)
    order = np.sort(z)[::-1]                       # descending
    top = order[0]
    gaps = top - order[1:N_TOP]
    lse = top + np.log(np.sum(np.exp(z - top)))
    p = np.exp(z - lse)
    nz = p > 0
    entropy = -np.sum(p[nz] * (z[nz] - lse))
    return np.concatenate([[top], gaps, [top - lse], [entropy]])


def logit_projection(z: np.ndarray, p_logit: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    return np.asarray(p_logit, dtype=np.float64) @ (z - z.mean())


def hidden_projection(h: np.ndarray, p_hidden: np.ndarray) -> np.ndarray:
    return np.asarray(p_hidden, dtype=np.float64) @ np.asarray(h, dtype=np.float64)


def batch_context(n_live: int) -> np.ndarray:
    c = np.zeros(BATCH_CTX)
    c[0] = float(n_live)
    c[3] = 1.0
    return c


def features(logits: np.ndarray, hidden: np.ndarray, p_hidden, p_logit, n_live: int) -> np.ndarray:
    """features_i for every live request: logits [n, 15, V], hidden [n, 15, H] -> [n, 1735]."""
    n = int(n_live)
    out = np.zeros((n, N_FEATURES))
    for i in range(n):
        conf = [confidence_features(logits[i, p]) for p in range(N_POS)]
        hp = [hidden_projection(hidden[i, p], p_hidden) for p in range(N_POS)]
        lp = [logit_projection(logits[i, p], p_logit) for p in range(N_POS)]
        out[i] = np.concatenate(conf + hp + lp + [batch_context(n)])
    return out


def mlp(feat: np.ndarray, w1, b1, w2, b2) -> np.ndarray:
    """predLogits = W2 relu(W1 f + b1) + b2 for every row of feat."""
    f = np.asarray(feat, dtype=np.float64)
    h = np.maximum(f @ np.asarray(w1, dtype=np.float64).T + np.asarray(b1, dtype=np.float64), 0.0)
    return h @ np.asarray(w2, dtype=np.float64).T + np.asarray(b2, dtype=np.float64)


def predict(logits, hidden, p_hidden, p_logit, w1, b1, w2, b2, n_live: int, n_bs: int):
    """Returns dict(features [n_live, 1735], pred_logits [n_bs, 15]); rows of dead
    requests are zero."""
    f = features(np.asarray(logits), np.asarray(hidden), p_hidden, p_logit, n_live)
    pl = np.zeros((n_bs, N_POS))
    pl[: int(n_live)] = mlp(f, w1, b1, w2, b2)
    return dict(features=f, pred_logits=pl)
