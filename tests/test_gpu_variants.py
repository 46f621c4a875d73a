"""GPU-vs-oracle parity for the alternative readings (dkv_config.flags, pool_kind), through the C ABI:
scores within the relative tolerance, the integer budget arithmetic bit-exact on injected scores, and one
whole pass with every variant switched on."""
import numpy as np
import pytest
import torch

from oracle import dynamickv as O
from paper_2412_14838_b200 import binding as B
from paper_2412_14838_b200 import build, synth
from tests import _util as U
from tests.test_gpu_pass import GpuPass, check_properties, compare_full

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()


def dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


SCORE_SHAPES = [
    synth.WORKLOADS["tiny"].with_(L=1),
    synth.Workload("var1", 51, L=1, Hq=6, Hkv=2, D=128, Bt=2, S=1371, ws=8, pool=5, N=8, Bl=16, m=1, recipe="sink"),
    synth.Workload("var2", 52, L=1, Hq=4, Hkv=2, D=64, Bt=1, S=20, ws=16, pool=9, N=2, Bl=4, m=1, recipe="iid"),
]


@pytest.mark.parametrize("w", SCORE_SHAPES, ids=lambda w: w.name)
@pytest.mark.parametrize("pool_kind,flags", [(1, 0), (0, B.DKV_F_WINDOW_MEAN), (1, B.DKV_F_WINDOW_MEAN)])
def test_score_variants_match_oracle(w, pool_kind, flags):
    t = synth.layer_inputs(w, 0)
    h = B.dkv_create(B.config_of(w, pool_kind, flags))
    try:
        out = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
        B.dkv_score(h, 0, dev(t["q"]), dev(t["k"]), out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
    finally:
        B.dkv_destroy(h)
    ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"]), w.ws, w.pool,
                          pool_kind=pool_kind, window_mean=bool(flags & B.DKV_F_WINDOW_MEAN))["score"]
    U.assert_scores_close(got, ref, f"{w.name} pool_kind={pool_kind} flags={flags}")


def test_score_static_takes_the_variants_too():
    w = SCORE_SHAPES[1]
    t = synth.layer_inputs(w, 0)
    out = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
    B.dkv_score_static(B.config_of(w, 1, B.DKV_F_WINDOW_MEAN), dev(t["q"]), dev(t["k"]), out)
    torch.cuda.synchronize()
    ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"]), w.ws, w.pool, pool_kind=1,
                          window_mean=True)["score"]
    U.assert_scores_close(out.cpu().numpy(), ref, "static, average pool of the window mean")


@pytest.mark.parametrize("flags", [B.DKV_F_PRORATA, B.DKV_F_NORM_MINMAX, B.DKV_F_PRORATA | B.DKV_F_NORM_MINMAX])
@pytest.mark.parametrize("ties", [0.0, 0.2])
def test_rebudget_variants_bit_exact(flags, ties):
    w = synth.Workload("rbv", 53, L=6, Hq=3, Hkv=3, D=64, Bt=2, S=1029, ws=29, pool=7, N=37, Bl=100, m=2, recipe="iid")
    rng = np.random.default_rng(flags * 10 + int(ties * 10))
    gain = np.exp(rng.standard_normal(w.L)).astype(np.float32)
    hist = [synth.pooled_like_scores((w.Bt, w.Hkv, w.P), w.pool, seed=300 + i, tie_fraction=ties) * gain[i]
            for i in range(w.L)]
    if ties:
        for a in hist:
            a[:] = np.round(a * 4096) / 4096 + np.float32(2 ** -12)
    h = B.dkv_create(B.config_of(w, 0, flags))
    try:
        ref_counts = np.zeros((w.Bt, w.L), dtype=np.int64)
        cnt_a, z_a, zp_a, _ = B.dkv_budget_views(h)
        for l in range(w.L):
            B.dkv_set_scores(h, l, torch.from_numpy(hist[l]).cuda())
            B.dkv_select_topk(h, l)
            ref_counts[:, l] = w.Blc
            if (l + 1) % w.m:
                continue
            out = torch.empty((w.Bt, w.L), dtype=torch.int32, device="cuda")
            B.dkv_rebudget(h, l + 1, out)
            got = out.cpu().numpy()
            cnt, z, zp = (B.read_device_i32(h, a, (w.Bt, w.L)) for a in (cnt_a, z_a, zp_a))
            for b in range(w.Bt):
                ref = O.rebudget([hist[i][b].astype(np.float64) for i in range(l + 1)], ref_counts[b], w.N, w.Bl, w.L,
                                 prorata=bool(flags & B.DKV_F_PRORATA), minmax=bool(flags & B.DKV_F_NORM_MINMAX))
                assert cnt[b, :l + 1].tolist() == ref["cnt"]
                assert z[b, :l + 1].tolist() == ref["Z"] and zp[b, :l + 1].tolist() == ref["Zp"]
                assert got[b].tolist() == ref["counts"]
                ref_counts[b] = ref["counts"]
    finally:
        B.dkv_destroy(h)


def test_minmax_with_equal_counts_gives_every_layer_the_maximum():
    # identical score arrays in both layers and k = all of them: cnt_0 == cnt_1, so t_i = 1 for both
    w = synth.Workload("eq", 54, L=2, Hq=1, Hkv=1, D=64, Bt=1, S=60, ws=10, pool=1, N=50, Bl=50, m=2, recipe="iid")
    a = synth.pooled_like_scores((1, 1, w.P), 1, seed=7, tie_fraction=0.0)
    h = B.dkv_create(B.config_of(w, 0, B.DKV_F_NORM_MINMAX))
    try:
        for l in range(2):
            B.dkv_set_scores(h, l, torch.from_numpy(a).cuda())
            B.dkv_select_topk(h, l)
        out = torch.empty((1, 2), dtype=torch.int32, device="cuda")
        B.dkv_rebudget(h, 2, out)
        ref = O.rebudget([a[0].astype(np.float64)] * 2, [50, 50], w.N, w.Bl, w.L, minmax=True)
        assert ref["cnt"] == [50, 50] and out.cpu().numpy()[0].tolist() == ref["counts"]
    finally:
        B.dkv_destroy(h)


@pytest.mark.parametrize("pool_kind,flags", [(1, B.DKV_F_WINDOW_MEAN | B.DKV_F_PRORATA | B.DKV_F_NORM_MINMAX),
                                             (0, B.DKV_F_PRORATA)])
def test_pass_with_variants_matches_oracle(pool_kind, flags):
    w = synth.WORKLOADS["tiny"]
    g = GpuPass(w, pool_kind=pool_kind, flags=flags).run()
    try:
        check_properties(g)
        near = compare_full(g)
        assert near <= 8
    finally:
        g.close()


def test_unknown_flag_bits_and_pool_kinds_are_refused():
    w = synth.WORKLOADS["tiny"]
    with pytest.raises(B.DkvError) as e:
        B.dkv_create(B.config_of(w, 0, 0x100))
    assert e.value.code == B.DKV_ERR_INVALID_ARG
    with pytest.raises(B.DkvError) as e:
        B.dkv_create(B.config_of(w, 2, 0))
    assert e.value.code == B.DKV_ERR_UNSUPPORTED
