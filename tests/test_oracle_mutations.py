"""Plausible mistakes planted in the ORACLE (on the CPU) must be caught by its pins.

Each mutant replaces one oracle function by a wrong variant (a dropped 1/sqrt(d_k), a mean instead of a
sum, a wrong causal extent, an off-by-one pooling window, ties broken the wrong way, a rounding instead
of a floor, a total taken over l instead of L, counts allowed to grow).  The checks below are the closed
forms / hand cases the other oracle tests use; the real oracle passes all of them, every mutant fails one.
"""
import math
import types

import numpy as np
import pytest

from oracle import dynamickv as O


def _checks(o):
    """List of (name, bool) pins evaluated on an oracle-like namespace."""
    out = []
    # scale: two prefix keys + the window key, d_k = 16
    D, a = 16, 3.0
    q = np.zeros((1, 1, 1, D)); q[..., 0] = 1.0
    k = np.zeros((1, 1, 3, D)); k[0, 0, 0, 0] = a
    e = math.exp(a / 4.0)
    out.append(("scale", abs(o.window_scores(q, k, 1, 1)["raw"][0, 0, 0] - e / (e + 2.0)) < 1e-12))
    # sum over window rows and group: zero keys closed form
    ws, G, P = 3, 2, 7
    q = np.ones((1, G, ws, 4)); k = np.zeros((1, 1, P + ws, 4))
    want = G * sum(1.0 / (P + r + 1) for r in range(ws))
    out.append(("sum", np.allclose(o.window_scores(q, k, ws, 1)["raw"], want, rtol=1e-13)))
    # causal extent: a huge key inside the window must not touch row 0
    q = np.ones((1, 1, 3, 4)); k = np.zeros((1, 1, 8, 4)); k[0, 0, 6] = 100.0
    out.append(("causal", np.allclose(o.window_scores(q, k, 3, 1)["raw"][0, 0], 1.0 / 6 + 0.0, atol=1e-9)))
    # pooling window
    x = np.array([1.0, 5.0, 2.0, 0.0, 0.0, 3.0])
    out.append(("pool", o.max_pool_same(x, 3).tolist() == [5, 5, 5, 2, 3, 3]))
    # ties: lowest index first
    out.append(("ties", o.select_topk(np.full(6, 0.5), 2)["idx"].tolist() == [0, 1]))
    # budget: hand-worked case 2 and 3
    zz = o.budget_from_counts([10, 3, 2, 1], 8, 4, 4)
    out.append(("floor", zz["Z"] == [8, 2, 1, 0] and zz["Zp"] == [11, 2, 1, 0]))
    zz = o.budget_from_counts([6, 2], 8, 4, 4)
    out.append(("total", zz["Zp"] == [12, 3]))
    # counts never grow
    hist = [np.full((1, 10), 1.0), np.full((1, 10), 0.5)]
    res = o.rebudget(hist, [3, 3], 4, 8, 2)
    out.append(("shrink_only", res["counts"] == [3, 0]))
    # global ties to the lower layer
    out.append(("global_ties", o.global_topk_counts([np.full((1, 4), 0.5)] * 2, 4).tolist() == [4, 0]))
    # decode step: the hand-worked 3-key case (d_k = 4, probabilities 1/6, 2/6, 3/6), padding never read
    qd = np.zeros((1, 4, 1, 4)); qd[0, :, 0, 0] = 2.0               # four query heads on two KV heads
    kd = np.zeros((2, 5, 4)); vd = np.zeros((2, 5, 4))
    for j in range(3):
        kd[:, j, 0] = math.log(j + 1.0)
        vd[0, j] = [6.0 * (j + 1), 1.0, -(j + 1.0), 0.0]
        vd[1, j] = [1.0, 0.0, 0.0, 0.0]
    kd[:, 3:] = 50.0; vd[:, 3:] = 1e6
    got = o.decode_attention(qd, [kd], [vd], [3])
    out.append(("decode", np.allclose(got[0, 0, 0], [14.0, 1.0, -7.0 / 3.0, 0.0], rtol=1e-12, atol=1e-12)
                and np.allclose(got[0, 1, 0], [14.0, 1.0, -7.0 / 3.0, 0.0], rtol=1e-12, atol=1e-12)
                and np.allclose(got[0, 2, 0], [1.0, 0.0, 0.0, 0.0], atol=1e-12)
                and np.allclose(got[0, 3, 0], [1.0, 0.0, 0.0, 0.0], atol=1e-12)))
    # policies: floors towards minus infinity, first positions then the most recent
    out.append(("pyramid", o.policy_counts("pyramid", 5, 10) == [15, 12, 10, 7, 5]))
    out.append(("sinks", o.positions_sinks_recent(10, 2, 3).tolist() == [0, 1, 7, 8, 9]))
    return out


def _mutant(**overrides):
    ns = types.SimpleNamespace(**{n: getattr(O, n) for n in dir(O) if not n.startswith("_")})
    for name, fn in overrides.items():
        setattr(ns, name, fn)
    # functions that call other oracle functions must see the overrides too
    def window_scores(q_win, k, ws, pool):
        Bt, Hq, _, D = q_win.shape
        Hkv, S = k.shape[1], k.shape[2]
        G, P = Hq // Hkv, S - ws
        raw = np.zeros((Bt, Hkv, P))
        for b in range(Bt):
            for h in range(Hkv):
                for g in range(G):
                    A = ns.softmax_rows_causal(q_win[b, h * G + g], k[b, h], P)
                    raw[b, h] += ns.reduce_rows(A[:, :P])
        return {"raw": raw, "score": ns.max_pool_same(raw, pool)}
    def rebudget(history, counts, N, Bl, L):
        l = len(history); H, P = np.asarray(history[0]).shape
        cnt = ns.global_topk_counts(history, min(N * H * l, l * H * P))
        zz = ns.budget_from_counts(cnt, Bl, N, L)
        new = [int(x) for x in counts]
        for i in range(l):
            new[i] = ns.clamp(new[i], zz["Zp"][i])
        return {"counts": new, "cnt": list(cnt), **zz}
    if "reduce_rows" not in overrides:
        ns.reduce_rows = lambda A: A.sum(axis=0)
    if "clamp" not in overrides:
        ns.clamp = min
    if {"softmax_rows_causal", "reduce_rows", "max_pool_same"} & set(overrides):
        ns.window_scores = window_scores
    if {"global_topk_counts", "budget_from_counts", "clamp"} & set(overrides):
        ns.rebudget = rebudget
    return ns


def _softmax_no_scale(q_rows, keys, P):
    return O.softmax_rows_causal(q_rows * math.sqrt(q_rows.shape[1]), keys, P)


def _softmax_no_causal(q_rows, keys, P):
    return O.softmax_rows_causal(q_rows, keys, keys.shape[0])          # every row sees every key


def _pool_off_by_one(x, kernel):
    return O.max_pool_same(x, kernel + 2)


def _select_high_index(score, Bl):
    n = len(score)
    r = O.select_topk(np.asarray(score)[::-1], Bl)
    return {"idx": np.sort(n - 1 - r["idx"]), "rank": r["rank"]}


def _budget_round(cnt, Bl, N, L):
    cmax = max(cnt); Z = [round(Bl * t / cmax) for t in cnt]
    tot = sum(Z); return {"Z": Z, "Zp": [round(z * N * L / tot) for z in Z]}


def _budget_prorata(cnt, Bl, N, L):
    return O.budget_from_counts(cnt, Bl, N, len(cnt))


def _global_high_layer(history, k):
    return O.global_topk_counts(list(history)[::-1], k)[::-1]


def _decode_no_scale(q_dec, kb, vb, lengths):
    return O.decode_attention(q_dec * math.sqrt(q_dec.shape[-1]), kb, vb, lengths)


def _decode_wrong_group(q_dec, kb, vb, lengths):                       # query head hq reads KV head hq % Hkv
    Hkv = len(kb[0])
    perm = [(hq % Hkv) * (q_dec.shape[1] // Hkv) + hq // Hkv for hq in range(q_dec.shape[1])]
    return O.decode_attention(q_dec, kb, vb, lengths)[:, perm]


def _decode_reads_padding(q_dec, kb, vb, lengths):
    return O.decode_attention(q_dec, kb, vb, [int(n) + 1 for n in lengths])


def _pyramid_truncating(policy, L, N):
    if policy != "pyramid" or L == 1:
        return O.policy_counts(policy, L, N)
    return [N + int(N * (L - 1 - 2 * i) / (2 * (L - 1))) for i in range(L)]      # rounds towards zero


def _sinks_from_the_end(P, n_sink, n_recent):
    return O.positions_sinks_recent(P, n_recent, n_sink)


MUTANTS = {
    "decode: no 1/sqrt(d_k)": dict(decode_attention=_decode_no_scale),
    "decode: wrong KV head for a query head": dict(decode_attention=_decode_wrong_group),
    "decode: one padding row read": dict(decode_attention=_decode_reads_padding),
    "pyramid: truncation instead of floor": dict(policy_counts=_pyramid_truncating),
    "sinks and recents swapped": dict(positions_sinks_recent=_sinks_from_the_end),
    "no 1/sqrt(d_k)": dict(softmax_rows_causal=_softmax_no_scale),
    "mean over window rows": dict(reduce_rows=lambda A: A.mean(axis=0)),
    "no causal mask in the window": dict(softmax_rows_causal=_softmax_no_causal),
    "pooling two too wide": dict(max_pool_same=_pool_off_by_one),
    "ties to the highest index": dict(select_topk=_select_high_index),
    "round instead of floor": dict(budget_from_counts=_budget_round),
    "total over l instead of L": dict(budget_from_counts=_budget_prorata),
    "counts may grow": dict(clamp=lambda old, new: new),
    "global ties to the higher layer": dict(global_topk_counts=_global_high_layer),
}


def test_the_real_oracle_passes_every_pin():
    assert all(ok for _, ok in _checks(_mutant())), _checks(_mutant())
    assert all(ok for _, ok in _checks(O) if True)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_every_planted_mistake_is_caught(name):
    failed = [n for n, ok in _checks(_mutant(**MUTANTS[name])) if not ok]
    assert failed, f"mutant '{name}' slipped through all pins"
