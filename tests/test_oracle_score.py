"""Pins for the oracle's scoring (Eq. 1-2, Algorithm 1's scoring statement).

Each test fixes the oracle to something other than itself: a closed form, a conservation law,
a hand-worked case (tests/golden/softmax_handworked.txt), an independent torch route, or a
symmetry.  Together they are meant to catch a dropped 1/sqrt(d_k), a transposed operand, a
wrong causal extent, a wrong group mapping, a sum/mean mix-up and an off-by-one in pooling.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import dynamickv as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_zero_keys_closed_form():
    # K == 0: every visible key gets 1/(P+r+1) from window row r, so raw[j] = G * sum_r 1/(P+r+1).
    ws, G, P, D = 2, 1, 3, 4
    q = _rand((1, G, ws, D), 0)
    k = np.zeros((1, 1, P + ws, D))
    out = O.window_scores(q, k, ws, pool=1)
    assert np.allclose(out["raw"], 1 / 4 + 1 / 5, rtol=0, atol=1e-15)
    ws, G, P, D = 5, 3, 11, 8
    q = _rand((2, 2 * G, ws, D), 1)
    k = np.zeros((2, 2, P + ws, D))
    expect = G * sum(1.0 / (P + r + 1) for r in range(ws))
    out = O.window_scores(q, k, ws, pool=3)
    assert np.allclose(out["score"], expect, rtol=1e-14)


def test_zero_queries_closed_form():
    ws, G, P, D = 4, 2, 9, 8
    q = np.zeros((1, G, ws, D))
    k = _rand((1, 1, P + ws, D), 2)
    expect = G * sum(1.0 / (P + r + 1) for r in range(ws))
    assert np.allclose(O.window_scores(q, k, ws, 1)["raw"], expect, rtol=1e-14)


def test_probability_mass_is_conserved():
    ws, G, Hkv, P, D = 6, 4, 3, 50, 16
    q = _rand((2, Hkv * G, ws, D), 3) * 2
    k = _rand((2, Hkv, P + ws, D), 4) * 2
    out = O.window_scores(q, k, ws, 5)
    total = out["raw"].sum(-1) + out["window_mass"]
    assert np.allclose(total, ws * G, rtol=1e-13)
    # the causal block is not empty: row r puts mass on r+1 window columns
    assert (out["window_mass"] > 0).all()


def test_hand_worked_three_keys():
    vals = {}
    with open(os.path.join(GOLDEN, "softmax_handworked.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, v = line.split()
            vals[name] = float(v)
    q = np.array([[[[math.sqrt(2.0), 0.0]]]])
    k = np.array([[[[math.log(1.0), 0.0], [math.log(2.0), 0.0], [math.log(3.0), 0.0]]]])
    out = O.window_scores(q, k, ws=1, pool=1)
    assert out["raw"][0, 0, 0] == pytest.approx(vals["raw0"], rel=1e-14)
    assert out["raw"][0, 0, 1] == pytest.approx(vals["raw1"], rel=1e-14)
    assert out["window_mass"][0, 0] == pytest.approx(vals["window_mass"], rel=1e-14)


def test_scale_is_one_over_sqrt_dk():
    # two prefix keys + the window key itself, d_k = 16: logit gap must be (a-b)/4, not (a-b).
    D, a = 16, 3.0
    q = np.zeros((1, 1, 1, D)); q[..., 0] = 1.0
    k = np.zeros((1, 1, 3, D)); k[0, 0, 0, 0] = a
    out = O.window_scores(q, k, ws=1, pool=1)
    e = math.exp(a / 4.0)
    assert out["raw"][0, 0, 0] == pytest.approx(e / (e + 2.0), rel=1e-14)
    assert out["raw"][0, 0, 1] == pytest.approx(1.0 / (e + 2.0), rel=1e-14)


def test_one_hot_key_takes_all_mass_and_pooling_spreads_it():
    ws, G, P, D, pool = 3, 2, 20, 8, 5
    rng = np.random.default_rng(5)
    qdir = rng.standard_normal(D); qdir /= np.linalg.norm(qdir)
    q = np.broadcast_to(qdir * 4.0, (1, G, ws, D)).copy()
    k = np.zeros((1, 1, P + ws, D))
    jstar = 9
    k[0, 0, jstar] = qdir * 200.0
    out = O.window_scores(q, k, ws, pool)
    assert out["raw"][0, 0, jstar] == pytest.approx(ws * G, rel=1e-12)
    s = out["score"][0, 0]
    assert np.allclose(s[jstar - 2:jstar + 3], ws * G, rtol=1e-12)
    assert (s[:jstar - 2] < 1e-6).all() and (s[jstar + 3:] < 1e-6).all()


def test_against_torch_softmax_and_max_pool():
    # Independent route: full causal attention matrix with torch.softmax over ALL S rows, last ws
    # rows sliced afterwards; pooling with F.max_pool1d (pads with -inf).
    ws, G, Hkv, P, D, pool = 8, 2, 2, 70, 16, 7
    S = P + ws
    q = _rand((1, Hkv * G, ws, D), 6)
    k = _rand((1, Hkv, S, D), 7)
    out = O.window_scores(q, k, ws, pool)
    tq, tk = torch.from_numpy(q), torch.from_numpy(k)
    for h in range(Hkv):
        acc = torch.zeros(P, dtype=torch.float64)
        for g in range(G):
            qfull = torch.zeros(S, D, dtype=torch.float64)
            qfull[P:] = tq[0, h * G + g]
            logits = qfull @ tk[0, h].T / math.sqrt(D)
            mask = torch.ones(S, S, dtype=torch.bool).tril()
            A = torch.softmax(logits.masked_fill(~mask, float("-inf")), dim=-1)
            acc += A[P:, :P].sum(0)
        pooled = torch.nn.functional.max_pool1d(acc[None, None], pool, 1, pool // 2)[0, 0]
        assert np.allclose(out["raw"][0, h], acc.numpy(), rtol=1e-12)
        assert np.allclose(out["score"][0, h], pooled.numpy(), rtol=1e-12)


def test_prefix_permutation_equivariance():
    ws, G, P, D = 4, 2, 33, 8
    q = _rand((1, G, ws, D), 8)
    k = _rand((1, 1, P + ws, D), 9)
    perm = np.random.default_rng(10).permutation(P)
    k2 = k.copy(); k2[0, 0, :P] = k[0, 0, perm]
    a = O.window_scores(q, k, ws, 1)["raw"][0, 0]
    b = O.window_scores(q, k2, ws, 1)["raw"][0, 0]
    assert np.allclose(b, a[perm], rtol=1e-12)


def test_group_mapping_uses_consecutive_query_heads():
    # KV head h is scored by query heads hG .. hG+G-1: making exactly those heads' queries zero must
    # turn head h's scores into the uniform closed form and leave the other head untouched.
    ws, G, Hkv, P, D = 3, 2, 2, 12, 8
    q = _rand((1, Hkv * G, ws, D), 11)
    k = _rand((1, Hkv, P + ws, D), 12)
    base = O.window_scores(q, k, ws, 1)["raw"]
    q2 = q.copy(); q2[0, 2:4] = 0
    out = O.window_scores(q2, k, ws, 1)["raw"]
    assert np.allclose(out[0, 0], base[0, 0])
    assert np.allclose(out[0, 1], G * sum(1.0 / (P + r + 1) for r in range(ws)))


def test_causal_extent_inside_window():
    # A huge key at window position P+1 must not change row 0 (which cannot see it) but must drain
    # rows 1.. of their prefix mass.
    ws, P, D = 3, 5, 4
    q = np.ones((1, 1, ws, D))
    k = np.zeros((1, 1, P + ws, D))
    k[0, 0, P + 1] = 100.0
    out = O.window_scores(q, k, ws, 1)
    # row 0 sees P+1 keys, all logit 0 -> 1/(P+1) each; rows 1,2 put ~all mass on the big key.
    assert np.allclose(out["raw"][0, 0], 1.0 / (P + 1), rtol=1e-12)


def test_max_pool_small_cases():
    x = np.array([1.0, 5.0, 2.0, 0.0, 0.0, 3.0])
    assert O.max_pool_same(x, 1).tolist() == x.tolist()
    assert O.max_pool_same(x, 3).tolist() == [5, 5, 5, 2, 3, 3]
    assert O.max_pool_same(x, 5).tolist() == [5, 5, 5, 5, 3, 3]
    assert O.max_pool_same(np.array([2.0, 1.0]), 7).tolist() == [2, 2]
    with pytest.raises(ValueError):
        O.max_pool_same(x, 4)
