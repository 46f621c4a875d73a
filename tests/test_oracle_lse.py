"""Pins for the oracle's one-sweep scoring route (Eq. 2 from Eq. 1's log-denominators).

``window_lse`` is fixed by a closed form (zero keys), the hand-worked three-key case
(tests/golden/softmax_handworked.txt: ln 6) and torch's logsumexp on a causal mask built here;
``window_scores_from_lse`` by a closed form, by the scaling law of its definition, by the hand-worked
case, and by agreeing with the row-normalising route of ``window_scores`` (different arithmetic: that
one divides by a sum it forms itself, this one subtracts a logarithm it is given).
"""
import math
import os

import numpy as np
import torch

from oracle import dynamickv as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "softmax_handworked.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, v = line.split()
                vals[name] = float(v)
    return vals


def test_lse_zero_keys_closed_form():
    # K == 0: row r sees P + r + 1 logits equal to 0, so its log-denominator is ln(P + r + 1).
    ws, G, P, D = 5, 3, 11, 8
    q = _rand((2, 2 * G, ws, D), 0)
    k = np.zeros((2, 2, P + ws, D))
    lse = O.window_lse(q, k, ws)
    expect = np.log(np.arange(P + 1, P + ws + 1, dtype=np.float64))
    assert np.allclose(lse, expect[None, None, :], rtol=0, atol=1e-14)
    out = O.window_scores_from_lse(q, k, lse, ws, pool=3)
    assert np.allclose(out["score"], G * sum(1.0 / (P + r + 1) for r in range(ws)), rtol=1e-14)


def test_hand_worked_three_keys():
    g = _golden()
    q = np.array([[[[math.sqrt(2.0), 0.0]]]])
    k = np.array([[[[math.log(j + 1.0), 0.0] for j in range(3)]]])
    lse = O.window_lse(q, k, 1)
    assert lse.shape == (1, 1, 1) and abs(lse[0, 0, 0] - g["lse"]) < 1e-15
    assert abs(g["lse"] - math.log(6.0)) < 1e-15
    out = O.window_scores_from_lse(q, k, lse, 1, pool=1)
    assert np.allclose(out["raw"][0, 0], [g["raw0"], g["raw1"]], rtol=1e-15)


def test_lse_against_torch_logsumexp():
    ws, G, Hkv, P, D = 6, 4, 3, 40, 16
    q = _rand((2, Hkv * G, ws, D), 1) * 1.5
    k = _rand((2, Hkv, P + ws, D), 2) * 1.5
    lse = O.window_lse(q, k, ws)
    tq, tk = torch.from_numpy(q), torch.from_numpy(k).repeat_interleave(G, dim=1)
    logits = torch.einsum("bhrd,bhsd->bhrs", tq, tk) / math.sqrt(D)
    hidden = torch.arange(P + ws)[None, :] > (P + torch.arange(ws))[:, None]
    ref = torch.logsumexp(logits.masked_fill(hidden, float("-inf")), dim=-1).numpy()
    assert np.allclose(lse, ref, rtol=1e-13, atol=1e-13)


def test_from_lse_equals_the_normalising_route():
    ws, G, Hkv, P, D = 6, 4, 3, 70, 16
    q = _rand((2, Hkv * G, ws, D), 3) * 2
    k = _rand((2, Hkv, P + ws, D), 4) * 2
    a = O.window_scores(q, k, ws, 5)
    b = O.window_scores_from_lse(q, k, O.window_lse(q, k, ws), ws, 5)
    assert np.allclose(a["raw"], b["raw"], rtol=1e-12, atol=0)
    assert np.allclose(a["score"], b["score"], rtol=1e-12, atol=0)
    for kind, mean in ((1, False), (0, True), (1, True)):
        a = O.window_scores(q, k, ws, 5, pool_kind=kind, window_mean=mean)
        b = O.window_scores_from_lse(q, k, O.window_lse(q, k, ws), ws, 5, pool_kind=kind, window_mean=mean)
        assert np.allclose(a["score"], b["score"], rtol=1e-12, atol=0)


def test_scaling_law_and_row_independence():
    # exp(s - (lse + c)) = exp(-c) exp(s - lse): shifting every normaliser by ln 2 halves every score;
    # shifting one row's normaliser to +inf removes exactly that row's probabilities.
    ws, G, P, D = 3, 2, 20, 8
    q = _rand((1, G, ws, D), 5)
    k = _rand((1, 1, P + ws, D), 6)
    lse = O.window_lse(q, k, ws)
    base = O.window_scores_from_lse(q, k, lse, ws, 1)["raw"]
    half = O.window_scores_from_lse(q, k, lse + math.log(2.0), ws, 1)["raw"]
    assert np.allclose(half, base / 2, rtol=1e-14)
    lse2 = lse.copy()
    lse2[0, 1, 2] = np.inf
    dropped = O.window_scores_from_lse(q, k, lse2, ws, 1)["raw"]
    row = O.softmax_rows_causal(q[0, 1], k[0, 0], P)[2, :P]
    assert np.allclose(base - dropped, row[None, None, :], rtol=1e-11, atol=1e-15)
