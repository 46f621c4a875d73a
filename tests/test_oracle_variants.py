"""Pins for the oracle's alternative readings (window mean, average pool, pro-rata budget, min-max
normalisation).  Hand-worked budget cases (tests/golden/rebudget_variants_handworked.txt), closed forms
and an independent torch route; each variant must also leave the default untouched."""
import os

import numpy as np
import pytest
import torch

from oracle import dynamickv as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    out = []
    with open(os.path.join(GOLDEN, "rebudget_variants_handworked.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = [p.strip() for p in line.split("|")]
            ints = lambda s: [int(x) for x in s.split(",")]
            out.append(dict(case=int(parts[0]), variant=parts[1], N=int(parts[2]), Bl=int(parts[3]), L=int(parts[4]),
                            cnt=ints(parts[5]), Z=ints(parts[6]), Zp=ints(parts[7])))
    return out


@pytest.mark.parametrize("c", _cases(), ids=lambda c: f"case{c['case']}-{c['variant']}")
def test_budget_variants_hand_worked(c):
    zz = O.budget_from_counts(c["cnt"], c["Bl"], c["N"], c["L"], prorata="prorata" in c["variant"],
                              minmax="minmax" in c["variant"])
    assert zz["Z"] == c["Z"] and zz["Zp"] == c["Zp"]


def test_prorata_equals_default_at_the_last_update():
    cnt = [9, 4, 4, 1]
    a = O.budget_from_counts(cnt, 16, 5, 4)
    b = O.budget_from_counts(cnt, 16, 5, 4, prorata=True)
    assert a == b                                   # l == L: the two budgets coincide


def test_minmax_zeroes_the_least_hit_layer_and_keeps_the_maximum():
    rng = np.random.default_rng(0)
    for _ in range(20):
        cnt = rng.integers(1, 50, size=6).tolist()
        if max(cnt) == min(cnt):
            continue
        zz = O.budget_from_counts(cnt, 32, 8, 6, minmax=True)
        assert zz["Z"][int(np.argmin(cnt))] == 0 and max(zz["Z"]) == 32


def test_rebudget_passes_the_variants_through():
    hist = []
    for i, n in enumerate([6, 2]):
        a = np.full((1, 40), 0.001)
        a[0, 3:3 + n] = 1.0 + 0.01 * i
        hist.append(a)
    res = O.rebudget(hist, [8, 8], N=4, Bl=8, L=4, prorata=True)
    assert res["cnt"] == [6, 2] and res["Zp"] == [6, 1] and res["counts"] == [6, 1]
    res = O.rebudget(hist, [8, 8], N=4, Bl=8, L=4)
    assert res["Zp"] == [12, 3] and res["counts"] == [8, 3]


def test_avg_pool_small_cases_and_torch():
    x = np.array([1.0, 5.0, 2.0, 0.0, 0.0, 3.0])
    assert O.avg_pool_same(x, 1).tolist() == x.tolist()
    assert np.allclose(O.avg_pool_same(x, 3), [3.0, 8 / 3, 7 / 3, 2 / 3, 1.0, 1.5])
    assert np.allclose(O.avg_pool_same(np.array([2.0, 1.0]), 7), [1.5, 1.5])
    rng = np.random.default_rng(1)
    y = rng.random((3, 57))
    for k in (3, 5, 9):
        ref = torch.nn.functional.avg_pool1d(torch.from_numpy(y)[None], k, 1, k // 2, count_include_pad=False)[0]
        assert np.allclose(O.avg_pool_same(y, k), ref.numpy(), rtol=1e-13)
    with pytest.raises(ValueError):
        O.avg_pool_same(x, 2)


def test_window_mean_closed_form_and_scaling():
    # K == 0: the mean over the ws * G rows of 1 / (P + r + 1)
    ws, G, P, D = 4, 2, 9, 8
    q = np.random.default_rng(2).standard_normal((1, G, ws, D))
    k = np.zeros((1, 1, P + ws, D))
    out = O.window_scores(q, k, ws, 1, window_mean=True)
    assert np.allclose(out["raw"], sum(1.0 / (P + r + 1) for r in range(ws)) / ws, rtol=1e-14)
    # on random inputs the mean is the sum divided by ws * G, before pooling, for both pools
    k = np.random.default_rng(3).standard_normal((1, 1, P + ws, D))
    for kind in (0, 1):
        a = O.window_scores(q, k, ws, 3, pool_kind=kind)["score"]
        b = O.window_scores(q, k, ws, 3, pool_kind=kind, window_mean=True)["score"]
        assert np.allclose(b * (ws * G), a, rtol=1e-13)


def test_avg_pool_conserves_mass_away_from_the_borders():
    ws, G, P, D, pool = 3, 1, 40, 8, 5
    rng = np.random.default_rng(4)
    q = rng.standard_normal((1, G, ws, D))
    k = rng.standard_normal((1, 1, P + ws, D))
    raw = O.window_scores(q, k, ws, 1)["raw"][0, 0]
    pooled = O.window_scores(q, k, ws, pool, pool_kind=1)["score"][0, 0]
    # interior positions: a plain moving average of the raw scores
    for j in range(2, P - 2):
        assert pooled[j] == pytest.approx(raw[j - 2:j + 3].mean(), rel=1e-13)
    assert pooled[0] == pytest.approx(raw[:3].mean(), rel=1e-13)


def test_pass_with_variants_differs_only_where_expected():
    # pro-rata tightens the intermediate updates, so final counts are never larger than the default's
    rng = np.random.default_rng(5)
    L, Hq, Hkv, D, S, ws = 4, 2, 1, 8, 60, 4

    def layer_fn(l):
        r = np.random.default_rng(100 + l)
        q = r.standard_normal((1, Hq, ws, D)); k = r.standard_normal((1, Hkv, S, D)) * (1 + l)
        rows = (r.integers(0, 1 << 16, size=(1, Hkv, S, D))).astype(np.uint16)
        return {"q": q, "k": k, "k_rows": rows, "v_rows": rows}

    a = O.run_prefill_pass(layer_fn, L, ws=ws, pool=3, N=6, Bl=12, m=2)
    b = O.run_prefill_pass(layer_fn, L, ws=ws, pool=3, N=6, Bl=12, m=2, prorata=True)
    assert (b["counts"] <= a["counts"]).all()
    assert a["updates"][0][1][0]["cnt"] == b["updates"][0][1][0]["cnt"]      # same scores, same hits
    assert b["counts"].sum() <= 6 * L
