"""GPU-vs-oracle parity of the one-sweep scoring entry point (dkv_score_lse) through the C ABI.

The window rows' log-sum-exp values come from the oracle in fp64, are rounded to fp32 once, and those
fp32 values (widened exactly) are the shared input of both sides, like the bf16 queries and keys.
"""
import numpy as np
import pytest
import torch

from oracle import dynamickv as O
from paper_2412_14838_b200 import binding as B
from paper_2412_14838_b200 import build, synth
from tests import _util as U
from tests.test_gpu_stages import SHAPES, Ctx, dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()


def _inputs(w, layer):
    t = synth.layer_inputs(w, layer)
    q, k = synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"])
    lse32 = O.window_lse(q, k, w.ws).astype(np.float32)
    return t, q, k, lse32


def _gpu(c, layer, t, lse32):
    w = c.w
    out = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
    B.dkv_score_lse(c.h, layer, dev(t["q"]), dev(t["k"]), torch.from_numpy(lse32).cuda(), out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


FULL = [synth.WORKLOADS["mistral32k"].with_(L=1), synth.WORKLOADS["qwen16k"].with_(L=1)]


@pytest.mark.parametrize("w", SHAPES + FULL, ids=lambda w: w.name)
def test_score_lse_matches_oracle(w):
    with Ctx(w) as c:
        t, q, k, lse32 = _inputs(w, 0)
        got = _gpu(c, 0, t, lse32)
        ref = O.window_scores_from_lse(q, k, lse32.astype(np.float64), w.ws, w.pool)["score"]
        U.assert_scores_close(got, ref, f"{w.name} from lse")
        # and, the normalisers being the true ones up to fp32 rounding, the two-sweep definition as well
        U.assert_scores_close(got, O.window_scores(q, k, w.ws, w.pool)["score"], f"{w.name} vs Eq. 1-2")
        # the history slot holds what was copied out, and the two-sweep entry point agrees
        addr, _ = B.dkv_layer_views(c.h, 0)
        hist = np.empty_like(got)
        B.dkv_memcpy_to_host(c.h, hist, addr, hist.nbytes)
        assert (hist == got).all()
        two = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
        B.dkv_score(c.h, 0, dev(t["q"]), dev(t["k"]), two)
        torch.cuda.synchronize()
        U.assert_scores_close(two.cpu().numpy(), ref, f"{w.name} two sweeps")


def test_score_lse_feeds_the_selection():
    w = synth.Workload("lse_sel", 21, L=1, Hq=8, Hkv=2, D=128, Bt=2, S=3000, ws=16, pool=5, N=32, Bl=64, m=1,
                       recipe="sink")
    with Ctx(w) as c:
        t, q, k, lse32 = _inputs(w, 0)
        got = _gpu(c, 0, t, lse32)
        idx = torch.empty((w.Bt, w.Hkv, w.Bl), dtype=torch.int32, device="cuda")
        B.dkv_select_topk(c.h, 0, idx, None)
        torch.cuda.synchronize()
        idx = idx.cpu().numpy()
        for b in range(w.Bt):
            for h in range(w.Hkv):
                # bit-exact against the top-k of the very scores the GPU produced
                assert (idx[b, h] == O.select_topk(got[b, h].astype(np.float64), w.Bl)["idx"]).all()


def test_score_lse_variants_and_arguments():
    w = synth.Workload("lse_var", 22, L=1, Hq=6, Hkv=2, D=64, Bt=1, S=700, ws=8, pool=5, N=8, Bl=16, m=1,
                       recipe="iid")
    cfg = B.config_of(w)
    cfg.pool_kind = 1
    cfg.flags = B.DKV_F_WINDOW_MEAN
    h = B.dkv_create(cfg)
    try:
        t, q, k, lse32 = _inputs(w, 0)
        out = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
        dq, dk, dl = dev(t["q"]), dev(t["k"]), torch.from_numpy(lse32).cuda()
        B.dkv_score_lse(h, 0, dq, dk, dl, out)
        torch.cuda.synchronize()
        ref = O.window_scores_from_lse(q, k, lse32.astype(np.float64), w.ws, w.pool, pool_kind=1, window_mean=True)
        U.assert_scores_close(out.cpu().numpy(), ref["score"], "mean + average pool")
        with pytest.raises(B.DkvError):
            B.dkv_score_lse(h, 0, dq, dk, None, out)
        with pytest.raises(B.DkvError):
            B.dkv_score_lse(h, 1, dq, dk, dl, out)
    finally:
        B.dkv_destroy(h)
