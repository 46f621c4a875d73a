"""Pins for the oracle's driver loop (Algorithm 1) on small seeded workloads."""
import numpy as np

from oracle import dynamickv as O
from paper_2412_14838_b200 import synth


def _layer_fn(w):
    def fn(l):
        t = synth.layer_inputs(w, l)
        return {"q": synth.bf16_bits_to_f64(t["q"]), "k": synth.bf16_bits_to_f64(t["k"]),
                "k_rows": t["k"], "v_rows": t["v"]}
    return fn


SMALL = synth.WORKLOADS["tiny"].with_(name="tiny_s256", S=256, N=16, Bl=40)


def test_single_layer_rmax1_is_plain_topN():
    # L = 1, r_max = 1: the whole method reduces to one fixed-budget per-head top-N (SnapKV-like).
    w = SMALL.with_(L=1, N=16, Bl=16, m=1)
    res = O.run_prefill_pass(_layer_fn(w), w.L, ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    assert res["counts"].tolist() == [[16]]
    for h in range(w.Hkv):
        direct = O.select_topk(res["score"][0][0, h], 16)["idx"]
        assert res["idx"][0][0][h].tolist() == direct.tolist()


def test_no_update_when_interval_exceeds_depth_except_final():
    # m > L: no intermediate update; the driver still runs one at l = L (L % m != 0).
    w = SMALL.with_(L=3, m=5)
    res = O.run_prefill_pass(_layer_fn(w), w.L, ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    assert [u[0] for u in res["updates"]] == [3]


def test_pass_invariants_and_nestedness():
    w = SMALL
    res = O.run_prefill_pass(_layer_fn(w), w.L, ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    assert [u[0] for u in res["updates"]] == [2, 4]
    counts = res["counts"]
    assert counts.shape == (1, w.L) and (counts <= w.Blc).all() and counts.sum() <= w.N * w.L
    for l in range(w.L):
        t = synth.layer_inputs(w, l)
        for h in range(w.Hkv):
            c = int(counts[0, l])
            idx = res["idx"][l][0][h]
            assert len(idx) == c and (np.diff(idx) > 0).all()
            # final kept set = direct top-count of the full score array (rank truncation is nested)
            direct = O.select_topk(res["score"][l][0, h], c)["idx"]
            assert idx.tolist() == direct.tolist()
            assert set(idx.tolist()) <= set(res["first_idx"][l][0][h].tolist())
            kb, vb = res["kb"][l][0][h], res["vb"][l][0][h]
            assert kb.shape == (c + w.ws, w.D)
            assert (kb[:c] == t["k"][0, h][idx]).all() and (kb[c:] == t["k"][0, h][w.P:]).all()
            assert (vb[:c] == t["v"][0, h][idx]).all() and (vb[c:] == t["v"][0, h][w.P:]).all()


def test_counts_only_shrink_over_updates():
    w = SMALL.with_(L=6, m=2)
    res = O.run_prefill_pass(_layer_fn(w), w.L, ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    prev = [w.Blc] * w.L
    for l_done, trail in res["updates"]:
        cur = trail[0]["counts"]
        assert all(a <= b for a, b in zip(cur[:l_done], prev[:l_done]))
        assert cur[l_done:] == [0] * (w.L - l_done)        # layers not yet processed hold nothing
        prev = cur[:l_done] + [w.Blc] * (w.L - l_done)
