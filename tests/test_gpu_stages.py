"""Stage-by-stage GPU-vs-oracle parity through the C ABI.

Scores are compared within the stated relative tolerance.  The integer stages (per-head top-k,
rebudget, gather, shrink) are fed the SAME float32 scores on both sides (`dkv_set_scores`), so
their outputs must be bit-exact with no near-tie allowance.
"""
import numpy as np
import pytest
import torch

from oracle import dynamickv as O
from paper_2412_14838_b200 import binding as B
from paper_2412_14838_b200 import build, synth
from tests import _util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()


def dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


class Ctx:
    def __init__(self, w):
        self.w = w
        self.h = B.dkv_create(B.config_of(w))

    def __enter__(self):
        return self

    def __exit__(self, *a):
        B.dkv_destroy(self.h)


def gpu_scores(c: Ctx, layer, q_bits, k_bits):
    w = c.w
    out = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
    B.dkv_score(c.h, layer, dev(q_bits), dev(k_bits), out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


# ----------------------------------------------------------------------------------------- score
SHAPES = [
    synth.WORKLOADS["tiny"].with_(L=2),
    # ragged: G = 3, 24 window rows, prefix not a multiple of any tile, D = 128, pool 3
    synth.Workload("rag1", 11, L=1, Hq=6, Hkv=2, D=128, Bt=2, S=1371, ws=8, pool=3, N=8, Bl=16, m=1, recipe="sink"),
    # no pooling, single query head per KV head, prefix shorter than one tile
    synth.Workload("rag2", 12, L=1, Hq=2, Hkv=2, D=64, Bt=1, S=77, ws=5, pool=1, N=4, Bl=8, m=1, recipe="iid"),
    # 256 window rows (the maximum), several tiles and a tail
    synth.Workload("rag3", 13, L=1, Hq=8, Hkv=1, D=128, Bt=1, S=4133, ws=32, pool=7, N=8, Bl=16, m=1, recipe="sink"),
    # pooling wider than the prefix
    synth.Workload("rag4", 14, L=1, Hq=4, Hkv=2, D=64, Bt=1, S=20, ws=16, pool=9, N=2, Bl=4, m=1, recipe="iid"),
    # 16 window rows = a single 16-column chunk in sweep 2 (half of the softmax warps have nothing to read),
    # one head long enough that every CTA reuses its accumulator stages
    # G = 7 (28 query / 4 KV heads scaled down): 224 window rows, not a power of two, two row blocks in sweep 1
    synth.Workload("rag6", 17, L=1, Hq=14, Hkv=2, D=128, Bt=1, S=2500, ws=32, pool=7, N=8, Bl=16, m=1, recipe="sink"),
    synth.Workload("rag5", 16, L=1, Hq=2, Hkv=1, D=64, Bt=1, S=90001, ws=8, pool=3, N=8, Bl=16, m=1, recipe="iid"),
]


@pytest.mark.parametrize("w", SHAPES, ids=lambda w: w.name)
def test_score_matches_oracle(w):
    with Ctx(w) as c:
        for layer in range(w.L):
            t = synth.layer_inputs(w, layer)
            got = gpu_scores(c, layer, t["q"], t["k"])
            ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"]), w.ws, w.pool)["score"]
            U.assert_scores_close(got, ref, f"{w.name} layer {layer}")
            # the history slot holds the same values as the copy-out
            addr, _ = B.dkv_layer_views(c.h, layer)
            hist = np.empty_like(got)
            B.dkv_memcpy_to_host(c.h, hist, addr, hist.nbytes)
            assert (hist == got).all()


def test_score_extreme_logits_do_not_overflow():
    # keys aligned with the queries at 40x scale: logits of several hundred, far beyond exp's fp32 range
    w = synth.Workload("hot", 15, L=1, Hq=2, Hkv=1, D=64, Bt=1, S=300, ws=4, pool=1, N=4, Bl=8, m=1, recipe="iid")
    t = synth.layer_inputs(w, 0)
    q = synth.bf16_bits_to_f32(t["q"])
    k = synth.bf16_bits_to_f32(t["k"])
    k[0, 0, 17] = 40.0 * q[0, 0, 0]
    k[0, 0, 230] = -40.0 * q[0, 1, 2]
    kb = synth.f32_to_bf16_bits(k)
    with Ctx(w) as c:
        got = gpu_scores(c, 0, t["q"], kb)
    ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(kb), w.ws, w.pool)["score"]
    assert np.isfinite(got).all()
    U.assert_scores_close(got, ref, "extreme logits")


def test_score_row_maximum_that_keeps_growing_along_the_prefix():
    # Sweep 1 sums relative to a reference that it raises only when a chunk of keys turns out far above it.  Hot keys
    # of growing strength in different tiles (and one beyond the last full tile) make every window row raise it
    # several times in mid-stream, by tens to hundreds of powers of two; in between come keys far below it.
    w = synth.Workload("grow", 18, L=1, Hq=4, Hkv=2, D=128, Bt=1, S=1500, ws=8, pool=3, N=4, Bl=8, m=1, recipe="iid")
    t = synth.layer_inputs(w, 0)
    q = synth.bf16_bits_to_f32(t["q"])
    k = synth.bf16_bits_to_f32(t["k"])
    for h in range(w.Hkv):
        mean_q = q[0, h * w.G:(h + 1) * w.G].reshape(-1, w.D).mean(axis=0)
        for pos, gain in ((40, 12.0), (300, 30.0), (301, -30.0), (700, 60.0), (1100, 5.0), (1400, 120.0)):
            k[0, h, pos] = gain * mean_q
    kb = synth.f32_to_bf16_bits(k)
    with Ctx(w) as c:
        got = gpu_scores(c, 0, t["q"], kb)
    ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(kb), w.ws, w.pool)["score"]
    assert np.isfinite(got).all()
    U.assert_scores_close(got, ref, "growing maximum")


# ----------------------------------------------------------------------------------------- select
def _inject(c: Ctx, layer, scores_f32):
    B.dkv_set_scores(c.h, layer, torch.from_numpy(scores_f32).cuda())


def _gpu_select(c: Ctx, layer):
    w = c.w
    idx = torch.empty((w.Bt, w.Hkv, w.Blc), dtype=torch.int32, device="cuda")
    rank = torch.empty_like(idx)
    B.dkv_select_topk(c.h, layer, idx, rank)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), rank.cpu().numpy()


SEL_SHAPES = [
    dict(Bt=1, Hkv=8, S=32768, ws=32, N=512, Bl=2048),      # full-size head, 2048 of 32736
    dict(Bt=2, Hkv=3, S=1029, ws=29, N=37, Bl=100),         # ragged, keep not a power of two
    dict(Bt=1, Hkv=2, S=500, ws=20, N=100, Bl=1000),        # Bl >= P: keep everything
    dict(Bt=1, Hkv=1, S=40, ws=8, N=1, Bl=1),               # single survivor, fewer positions than threads
    dict(Bt=1, Hkv=2, S=70000, ws=32, N=4096, Bl=16384),    # maximum budget, P above 65536
]


@pytest.mark.parametrize("kw", SEL_SHAPES, ids=lambda k: f"P{k['S']-k['ws']}_Bl{k['Bl']}")
@pytest.mark.parametrize("ties", [0.0, 0.3])
def test_select_bit_exact(kw, ties):
    w = synth.Workload("sel", 21, L=1, Hq=kw["Hkv"], D=64, pool=7, m=1, recipe="iid", **kw)
    sc = synth.pooled_like_scores((w.Bt, w.Hkv, w.P), w.pool, seed=w.P + w.Bl, tie_fraction=ties)
    with Ctx(w) as c:
        _inject(c, 0, sc)
        idx, rank = _gpu_select(c, 0)
        counts = np.zeros((w.Bt, w.L), dtype=np.int32)
        B.dkv_get_counts(c.h, counts)
    assert (counts == w.Blc).all()
    for b in range(w.Bt):
        for h in range(w.Hkv):
            ref = O.select_topk(sc[b, h].astype(np.float64), w.Bl)
            assert (idx[b, h] == ref["idx"]).all(), f"kept set differs at b={b} h={h}"
            assert (rank[b, h] == ref["rank"]).all(), f"ranks differ at b={b} h={h}"


def test_select_all_equal_and_zero_scores():
    w = synth.Workload("sel0", 22, L=1, Hq=2, Hkv=2, D=64, Bt=1, S=3000, ws=8, pool=1, N=10, Bl=50, m=1, recipe="iid")
    sc = np.zeros((1, 2, w.P), dtype=np.float32)
    sc[0, 1] = 0.125
    sc[0, 1, 2000:2010] = 0.5
    with Ctx(w) as c:
        _inject(c, 0, sc)
        idx, rank = _gpu_select(c, 0)
    assert idx[0, 0].tolist() == list(range(50)) and rank[0, 0].tolist() == list(range(50))
    assert idx[0, 1].tolist() == list(range(40)) + list(range(2000, 2010))
    assert rank[0, 1].tolist() == list(range(10, 50)) + list(range(10))


def test_call_order_is_checked():
    w = synth.WORKLOADS["tiny"]
    with Ctx(w) as c:
        with pytest.raises(B.DkvError) as e:
            B.dkv_select_topk(c.h, 0)
        assert e.value.code == B.DKV_ERR_STATE
        with pytest.raises(B.DkvError) as e:
            B.dkv_rebudget(c.h, 1)
        assert e.value.code == B.DKV_ERR_STATE
        buf = torch.empty((w.Bt, w.Hkv, w.Blc + w.ws, w.D), dtype=torch.int16, device="cuda")
        with pytest.raises(B.DkvError) as e:
            B.dkv_compact(c.h, 0, None, None, buf, buf)
        assert e.value.code == B.DKV_ERR_STATE
        with pytest.raises(B.DkvError) as e:
            B.dkv_score(c.h, 99, buf, buf)
        assert e.value.code == B.DKV_ERR_INVALID_ARG


# ----------------------------------------------------------------------------------------- rebudget
RB_SHAPES = [
    dict(L=32, Hkv=8, Bt=1, S=32768, ws=32, N=512, Bl=2048, m=4),     # full size, 8.4 M scores at the last update
    dict(L=6, Hkv=3, Bt=2, S=1029, ws=29, N=37, Bl=100, m=2),
    dict(L=5, Hkv=2, Bt=1, S=300, ws=10, N=64, Bl=200, m=2),          # L % m != 0
    dict(L=3, Hkv=1, Bt=1, S=50, ws=10, N=100, Bl=400, m=1),          # k clamped to the population
]


@pytest.mark.parametrize("kw", RB_SHAPES, ids=lambda k: f"L{k['L']}_P{k['S']-k['ws']}")
@pytest.mark.parametrize("ties", [0.0, 0.2])
def test_rebudget_bit_exact(kw, ties):
    w = synth.Workload("rb", 31, Hq=kw["Hkv"], D=64, pool=7, recipe="iid", **kw)
    rng = np.random.default_rng(w.L * 1000 + w.P)
    layer_gain = np.exp(rng.standard_normal(w.L)).astype(np.float32)
    hist = [synth.pooled_like_scores((w.Bt, w.Hkv, w.P), w.pool, seed=100 + i, tie_fraction=ties) * layer_gain[i]
            for i in range(w.L)]
    if ties:
        for a in hist:                      # identical values across layers: ties at the global cut
            a[:] = np.round(a * 4096) / 4096 + np.float32(2 ** -12)
    with Ctx(w) as c:
        ref_counts = np.zeros((w.Bt, w.L), dtype=np.int64)
        cnt_a, z_a, zp_a, held_a = B.dkv_budget_views(c.h)
        for l in range(w.L):
            _inject(c, l, hist[l])
            B.dkv_select_topk(c.h, l)
            ref_counts[:, l] = w.Blc
            update = (l + 1) % w.m == 0 or (l + 1 == w.L and w.L % w.m != 0)
            if not update:
                continue
            out = torch.empty((w.Bt, w.L), dtype=torch.int32, device="cuda")
            B.dkv_rebudget(c.h, l + 1, out)
            got = out.cpu().numpy()
            cnt, z, zp = (B.read_device_i32(c.h, a, (w.Bt, w.L)) for a in (cnt_a, z_a, zp_a))
            for b in range(w.Bt):
                ref = O.rebudget([hist[i][b].astype(np.float64) for i in range(l + 1)], ref_counts[b], w.N, w.Bl, w.L)
                assert cnt[b, :l + 1].tolist() == ref["cnt"], f"hits per layer differ after {l+1} layers"
                assert z[b, :l + 1].tolist() == ref["Z"] and zp[b, :l + 1].tolist() == ref["Zp"]
                assert got[b].tolist() == ref["counts"]
                ref_counts[b] = ref["counts"]
        host = np.zeros((w.Bt, w.L), dtype=np.int32)
        B.dkv_get_counts(c.h, host)
        assert (host == ref_counts).all()


# ----------------------------------------------------------------------------------------- gather / shrink
@pytest.mark.parametrize("D", [64, 128])
def test_gather_and_shrink_bytes(D):
    w = synth.Workload("cmp", 41, L=3, Hq=4, Hkv=2, D=D, Bt=2, S=2100, ws=20, pool=5, N=40, Bl=300, m=3, recipe="iid")
    rng = np.random.default_rng(D)
    hist = [synth.pooled_like_scores((w.Bt, w.Hkv, w.P), w.pool, seed=200 + i, tie_fraction=0.1) * (1 + 3 * i)
            for i in range(w.L)]
    kfull = [rng.integers(0, 1 << 16, size=(w.Bt, w.Hkv, w.S, w.D), dtype=np.uint16) for _ in range(w.L)]
    vfull = [rng.integers(0, 1 << 16, size=(w.Bt, w.Hkv, w.S, w.D), dtype=np.uint16) for _ in range(w.L)]
    with Ctx(w) as c:
        kb = [torch.zeros((w.Bt, w.Hkv, w.Blc + w.ws, w.D), dtype=torch.int16, device="cuda") for _ in range(w.L)]
        vb = [torch.zeros_like(kb[0]) for _ in range(w.L)]
        lens = torch.zeros((w.Bt, w.Hkv), dtype=torch.int32, device="cuda")
        sel = []
        for l in range(w.L):
            _inject(c, l, hist[l])
            idx, rank = _gpu_select(c, l)
            sel.append((idx, rank))
            B.dkv_compact(c.h, l, dev(kfull[l]), dev(vfull[l]), kb[l], vb[l], lens)
            torch.cuda.synchronize()
            assert (lens.cpu().numpy() == w.Blc + w.ws).all()
            got_k = kb[l].cpu().numpy().view(np.uint16)
            for b in range(w.Bt):
                for h in range(w.Hkv):
                    first = O.select_topk(hist[l][b, h].astype(np.float64), w.Bl)
                    ref = U.buffer_order(O.gather_rows(kfull[l][b, h], first["idx"], w.ws), first["rank"], w.Blc)
                    assert (got_k[b, h] == ref).all()
        counts = torch.empty((w.Bt, w.L), dtype=torch.int32, device="cuda")
        B.dkv_rebudget(c.h, w.L, counts)
        B.dkv_compact_all(c.h, w.L, kb, vb)
        torch.cuda.synchronize()
        counts = counts.cpu().numpy()
        held = B.read_device_i32(c.h, B.dkv_budget_views(c.h)[3], (w.Bt, w.L))
        assert (held == counts).all()
        assert (counts < w.Blc).any(), "the case should actually shrink something"
        for l in range(w.L):
            got_k = kb[l].cpu().numpy().view(np.uint16)
            got_v = vb[l].cpu().numpy().view(np.uint16)
            _, idx_a = B.dkv_layer_views(c.h, l)
            idx_now = B.read_device_i32(c.h, idx_a, (w.Bt, w.Hkv, w.Blc))
            sorted_dev = torch.zeros((w.Bt, w.Hkv, w.Blc), dtype=torch.int32, device="cuda")
            B.dkv_kept_sorted(c.h, l, sorted_dev)
            torch.cuda.synchronize()
            sorted_now = sorted_dev.cpu().numpy()
            for b in range(w.Bt):
                n = int(counts[b, l])
                for h in range(w.Hkv):
                    first = O.select_topk(hist[l][b, h].astype(np.float64), w.Bl)
                    buf0 = O.gather_rows(kfull[l][b, h], first["idx"], w.ws)
                    rk, ri, rr = O.shrink_rows(buf0, first["idx"], first["rank"], w.Blc, n, w.ws)
                    rv, _, _ = O.shrink_rows(O.gather_rows(vfull[l][b, h], first["idx"], w.ws), first["idx"],
                                             first["rank"], w.Blc, n, w.ws)
                    assert (got_k[b, h, :n + w.ws] == U.buffer_order(rk, rr, n)).all()
                    assert (got_v[b, h, :n + w.ws] == U.buffer_order(rv, rr, n)).all()
                    assert (idx_now[b, h, :n] == ri[np.argsort(rr, kind="stable")]).all()
                    assert (sorted_now[b, h, :n] == ri).all()
        # a second shrink with unchanged counts must leave everything as it is
        before = [t.clone() for t in kb]
        B.dkv_compact_all(c.h, w.L, kb, vb)
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(before, kb))


def test_gather_after_an_update_applies_the_new_count():
    # select two layers, rebudget, and only then gather: the buffers must come out at the new counts
    w = synth.Workload("late", 42, L=2, Hq=2, Hkv=2, D=64, Bt=1, S=800, ws=16, pool=3, N=20, Bl=120, m=2, recipe="iid")
    rng = np.random.default_rng(5)
    hist = [synth.pooled_like_scores((1, 2, w.P), 3, seed=300 + i) * (1 + 9 * i) for i in range(2)]
    kfull = [rng.integers(0, 1 << 16, size=(1, 2, w.S, w.D), dtype=np.uint16) for _ in range(2)]
    with Ctx(w) as c:
        for l in range(2):
            _inject(c, l, hist[l])
            B.dkv_select_topk(c.h, l)
        counts = torch.empty((1, 2), dtype=torch.int32, device="cuda")
        B.dkv_rebudget(c.h, 2, counts)
        counts = counts.cpu().numpy()
        for l in range(2):
            kb = torch.zeros((1, 2, w.Blc + w.ws, w.D), dtype=torch.int16, device="cuda")
            vb = torch.zeros_like(kb)
            B.dkv_compact(c.h, l, dev(kfull[l]), dev(kfull[l]), kb, vb)
            torch.cuda.synchronize()
            n = int(counts[0, l])
            for h in range(2):
                sel_n = O.select_topk(hist[l][0, h].astype(np.float64), n)
                ref = U.buffer_order(O.gather_rows(kfull[l][0, h], sel_n["idx"], w.ws), sel_n["rank"], n)
                assert (kb.cpu().numpy().view(np.uint16)[0, h, :n + w.ws] == ref).all()
