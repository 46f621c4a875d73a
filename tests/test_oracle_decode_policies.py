"""Pins for the oracle's decode step (Eq. 1 over a compressed, ragged cache; Section 4.3) and for the
fixed-pattern budget policies (the "Baselines" paragraph of Section 5.1).

Decode: a hand-worked 3-key case, torch's masked softmax attention on padded buffers, invariance under a
permutation of the cached rows, special cases (one row, equal keys), the GQA head mapping and the length mask.
Policies: hand-worked schedules, sums and monotonicity; the one-sweep pass equals the two-sweep pass.
"""
import os

import numpy as np
import pytest
import torch

from oracle import dynamickv as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def _hand_case():
    q = np.zeros((1, 1, 1, 4)); q[0, 0, 0, 0] = 2.0
    k = np.zeros((5, 4)); v = np.zeros((5, 4))
    for j in range(3):
        k[j, 0] = np.log(j + 1.0)
        v[j] = [6.0 * (j + 1), 1.0, -(j + 1.0), 0.0]
    k[3:] = np.nan; v[3:] = np.nan                       # padding rows must never be read
    return q, [[k]], [[v]]


def test_decode_hand_worked_case():
    g = _golden("decode_handworked.txt")
    q, kb, vb = _hand_case()
    out = O.decode_attention(q, kb, vb, [3])[0, 0, 0]
    assert np.allclose(out, [g["out0"], g["out1"], g["out2"], g["out3"]], rtol=1e-14, atol=1e-14)
    out = O.decode_attention(q, kb, vb, [2])[0, 0, 0]
    assert np.allclose(out, [g["short0"], g["short1"], g["short2"], g["short3"]], rtol=1e-14, atol=1e-14)


def _random_case(seed, Bt=2, Hq=6, Hkv=2, nq=3, D=16, rows=37):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((Bt, Hq, nq, D))
    kb = rng.standard_normal((Bt, Hkv, rows, D)) * 1.5
    vb = rng.standard_normal((Bt, Hkv, rows, D))
    lengths = rng.integers(1, rows + 1, size=Bt)
    return q, kb, vb, lengths


@pytest.mark.parametrize("seed", range(4))
def test_decode_matches_torch_masked_attention(seed):
    q, kb, vb, lengths = _random_case(seed)
    Bt, Hq, nq, D = q.shape
    G = Hq // kb.shape[1]
    tq = torch.from_numpy(q)
    tk = torch.from_numpy(kb).repeat_interleave(G, dim=1)              # [Bt, Hq, rows, D]
    tv = torch.from_numpy(vb).repeat_interleave(G, dim=1)
    mask = torch.arange(kb.shape[2])[None, :] < torch.from_numpy(lengths)[:, None]       # [Bt, rows]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask[:, None, None, :])
    got = O.decode_attention(q, kb, vb, lengths)
    assert np.allclose(got, want.numpy(), rtol=1e-12, atol=1e-12)


def test_decode_does_not_depend_on_the_order_of_the_cached_rows():
    q, kb, vb, lengths = _random_case(11)
    got = O.decode_attention(q, kb, vb, lengths)
    kb2, vb2 = kb.copy(), vb.copy()
    rng = np.random.default_rng(5)
    for b in range(kb.shape[0]):
        perm = rng.permutation(int(lengths[b]))
        kb2[b, :, :lengths[b]] = kb[b][:, perm]
        vb2[b, :, :lengths[b]] = vb[b][:, perm]
    assert np.allclose(O.decode_attention(q, kb2, vb2, lengths), got, rtol=1e-12, atol=1e-13)


def test_decode_special_cases():
    q, kb, vb, _ = _random_case(3)
    one = O.decode_attention(q, kb, vb, [1, 1])                        # a single row: its value, whatever the query
    G = q.shape[1] // kb.shape[1]
    for hq in range(q.shape[1]):
        assert np.allclose(one[:, hq], vb[:, hq // G, None, 0, :])
    kb_eq = np.repeat(kb[:, :, :1], kb.shape[2], axis=2)               # equal keys: the plain mean of the values
    n = [5, 9]
    avg = O.decode_attention(q, kb_eq, vb, n)
    for b in range(2):
        for hq in range(q.shape[1]):
            assert np.allclose(avg[b, hq], vb[b, hq // G, :n[b]].mean(axis=0)[None, :], rtol=1e-12, atol=1e-13)
    lin = O.decode_attention(q, kb, 2.0 * vb + 1.0, [20, 30])          # affine in the values (weights sum to 1)
    assert np.allclose(lin, 2.0 * O.decode_attention(q, kb, vb, [20, 30]) + 1.0, rtol=1e-12, atol=1e-12)


def _rows(name, kind):
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            f = [x.strip() for x in line.split("|")]
            if (f[0] == "sinks") == (kind == "sinks"):
                yield f


def test_policy_schedules_hand_worked():
    for pol, L, N, counts in _rows("policies_handworked.txt", "counts"):
        assert O.policy_counts(pol, int(L), int(N)) == [int(x) for x in counts.split(",")]
    for _, P, a, b, pos in _rows("policies_handworked.txt", "sinks"):
        assert O.positions_sinks_recent(int(P), int(a), int(b)).tolist() == [int(x) for x in pos.split(",")]


@pytest.mark.parametrize("L,N", [(32, 512), (28, 128), (7, 33), (2, 1)])
def test_policy_invariants(L, N):
    u, p = O.policy_counts("uniform", L, N), O.policy_counts("pyramid", L, N)
    assert sum(u) == N * L
    assert N * L - L < sum(p) <= N * L                                 # every floor loses less than one
    assert all(a >= b for a, b in zip(p, p[1:])) and p[0] == N + N // 2 and min(p) >= 0
    pos = O.positions_sinks_recent(1000, 4, N)
    assert (np.diff(pos) > 0).all() and len(pos) == min(1000, 4 + N)


def test_pass_scored_from_the_log_denominators_equals_the_two_sweep_pass():
    from paper_2412_14838_b200 import synth
    w = synth.Workload("lsepass", 81, L=3, Hq=4, Hkv=2, D=64, Bt=1, S=300, ws=8, pool=3, N=16, Bl=40, m=2, recipe="sink")
    host = [synth.layer_inputs(w, l) for l in range(w.L)]
    fn = lambda l: {"q": synth.bf16_bits_to_f64(host[l]["q"]), "k": synth.bf16_bits_to_f64(host[l]["k"]),
                    "k_rows": host[l]["k"], "v_rows": host[l]["v"]}
    kw = dict(ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    a = O.run_prefill_pass(fn, w.L, **kw)
    b = O.run_prefill_pass(fn, w.L, lse_fn=lambda l: O.window_lse(fn(l)["q"], fn(l)["k"], w.ws), **kw)
    assert (a["counts"] == b["counts"]).all()
    for l in range(w.L):
        assert np.allclose(a["score"][l], b["score"][l], rtol=1e-12)
        for h in range(w.Hkv):
            assert (a["idx"][l][0][h] == b["idx"][l][0][h]).all()
