"""Pins for the oracle's selection and budget steps (Eq. 3-6, Update_Buffer_Length).

Brute-force subset enumeration fixes the per-head top-k and its tie rule; hand-worked cases
(tests/golden/rebudget_handworked.txt) fix the integer budget arithmetic; a from-scratch
Python sort fixes the global count; invariants cover the rest.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import dynamickv as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _brute_force_topk(score, keep):
    best, best_set = None, None
    for subset in itertools.combinations(range(len(score)), keep):       # lexicographic order
        tot = sum(score[i] for i in subset)
        if best is None or tot > best:                                    # strict: first (smallest) set wins ties
            best, best_set = tot, subset
    return list(best_set)


@pytest.mark.parametrize("seed", range(6))
def test_select_matches_subset_enumeration(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.integers(5, 12))
    keep = int(rng.integers(1, P))
    # few distinct dyadic values => many exact ties and exact sums
    score = rng.integers(0, 4, size=P).astype(np.float64) / 4.0
    sel = O.select_topk(score, keep)
    assert sel["idx"].tolist() == _brute_force_topk(score.tolist(), keep)


def test_select_all_equal_keeps_lowest_indices():
    sel = O.select_topk(np.full(10, 0.25), 4)
    assert sel["idx"].tolist() == [0, 1, 2, 3]
    assert sel["rank"].tolist() == [0, 1, 2, 3]


def test_select_rank_is_the_score_order():
    score = np.array([0.1, 0.9, 0.5, 0.9, 0.2, 0.7])
    sel = O.select_topk(score, 4)
    assert sel["idx"].tolist() == [1, 2, 3, 5]
    assert sel["rank"].tolist() == [0, 3, 1, 2]          # 0.9@1, 0.9@3, 0.7@5, 0.5@2


def test_select_invariants_and_clamp():
    rng = np.random.default_rng(3)
    score = rng.random(200)
    sel = O.select_topk(score, 64)
    idx, rank = sel["idx"], sel["rank"]
    assert (np.diff(idx) > 0).all() and idx.min() >= 0 and idx.max() < 200
    assert sorted(rank.tolist()) == list(range(64))
    by_rank = idx[np.argsort(rank)]
    assert (np.diff(score[by_rank]) <= 0).all()
    assert score[idx].min() >= np.delete(score, idx).max()
    sel = O.select_topk(score[:10], 64)                  # Bl >= P keeps everything
    assert sel["idx"].tolist() == list(range(10))


def test_select_is_nested():
    # top-k' of top-k equals top-k' of everything: what makes truncation by rank valid.
    rng = np.random.default_rng(4)
    score = np.round(rng.random(300), 2)                  # ties
    big = O.select_topk(score, 100)
    for k2 in (1, 17, 99):
        small = O.select_topk(score, k2)
        assert small["idx"].tolist() == big["idx"][big["rank"] < k2].tolist()


def _golden_cases():
    cases = []
    with open(os.path.join(GOLDEN, "rebudget_handworked.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = [p.strip() for p in line.split("|")]
            ints = lambda s: [int(x) for x in s.split(",")]
            cases.append(dict(case=int(parts[0]), N=int(parts[1]), Bl=int(parts[2]), L=int(parts[3]),
                              cnt=ints(parts[4]), Z=ints(parts[5]), Zp=ints(parts[6]), counts=ints(parts[7])))
    return cases


@pytest.mark.parametrize("c", _golden_cases(), ids=lambda c: f"case{c['case']}")
def test_budget_hand_worked(c):
    zz = O.budget_from_counts(c["cnt"], c["Bl"], c["N"], c["L"])
    assert zz["Z"] == c["Z"] and zz["Zp"] == c["Zp"]
    # the same case through the whole update, with scores built to give exactly these counts
    l, P = len(c["cnt"]), 40
    k = c["N"] * 1 * l
    assert sum(c["cnt"]) == k
    hist = []
    for i, n in enumerate(c["cnt"]):
        a = np.full((1, P), 0.001)
        a[0, 3:3 + n] = 1.0 + 0.01 * i
        hist.append(a)
    res = O.rebudget(hist, [c["Bl"]] * c["L"], c["N"], c["Bl"], c["L"])
    assert res["cnt"] == c["cnt"] and res["Zp"] == c["Zp"]
    assert res["counts"][:l] == c["counts"] and res["counts"][l:] == [c["Bl"]] * (c["L"] - l)


def test_global_counts_ties_go_to_lower_layers():
    hist = [np.full((1, 4), 0.5), np.full((1, 4), 0.5)]
    assert O.global_topk_counts(hist, 4).tolist() == [4, 0]
    assert O.global_topk_counts(hist, 6).tolist() == [4, 2]
    hist = [np.full((2, 3), 0.5), np.full((2, 3), 0.5)]          # two heads: head-major inside a layer
    assert O.global_topk_counts(hist, 7).tolist() == [6, 1]


def test_global_counts_against_python_sort():
    rng = np.random.default_rng(7)
    l, H, P = 5, 3, 37
    hist = [np.round(rng.random((H, P)), 1) for _ in range(l)]      # heavy ties
    k = 111
    triples = [(-hist[i][h, p], (i * H + h) * P + p, i) for i in range(l) for h in range(H) for p in range(P)]
    triples.sort()
    expect = [0] * l
    for t in triples[:k]:
        expect[t[2]] += 1
    assert O.global_topk_counts(hist, k).tolist() == expect


def test_rebudget_invariants():
    rng = np.random.default_rng(8)
    L, H, P, N, Bl = 8, 2, 300, 16, 48
    hist = [rng.random((H, P)) * (1 + i % 3) for i in range(L)]
    counts = [Bl] * L
    prev = counts
    for l in (2, 4, 6, 8):
        res = O.rebudget(hist[:l], prev, N, Bl, L)
        assert sum(res["cnt"]) == N * H * l
        assert max(res["Z"]) == Bl
        B = N * L
        assert B - l < sum(res["Zp"]) <= B
        assert all(a <= b for a, b in zip(res["counts"], prev))
        assert all(c <= Bl for c in res["counts"])
        prev = res["counts"]
    assert sum(prev) <= N * L


def test_rebudget_k_clamped_to_population():
    hist = [np.random.default_rng(9).random((1, 5)) for _ in range(2)]
    res = O.rebudget(hist, [8, 8], N=100, Bl=200, L=2)
    assert res["cnt"] == [5, 5]


def test_shrink_keeps_rank_below_count_in_position_order():
    rng = np.random.default_rng(10)
    P, ws, D, Bl = 60, 4, 3, 20
    full = rng.integers(0, 1 << 16, size=(P + ws, D)).astype(np.uint16)
    score = np.round(rng.random(P), 1)
    sel = O.select_topk(score, Bl)
    buf = O.gather_rows(full, sel["idx"], ws)
    assert buf.shape == (Bl + ws, D)
    assert (buf[:Bl] == full[sel["idx"]]).all() and (buf[Bl:] == full[P:]).all()
    rows, idx2, rank2 = O.shrink_rows(buf, sel["idx"], sel["rank"], Bl, 7, ws)
    direct = O.select_topk(score, 7)
    assert idx2.tolist() == direct["idx"].tolist() and rank2.tolist() == direct["rank"].tolist()
    assert (rows[:7] == full[direct["idx"]]).all() and (rows[7:] == full[P:]).all()
    # shrinking to more than is held changes nothing
    rows3, idx3, _ = O.shrink_rows(buf, sel["idx"], sel["rank"], Bl, 500, ws)
    assert (rows3 == buf).all() and idx3.tolist() == sel["idx"].tolist()
