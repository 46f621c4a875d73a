"""dkv_score_static: the scoring entry point for callers that cannot allocate device memory.

Some users of the library may not call cudaMalloc where they score a layer (a server whose own
pool already owns all of the GPU's memory, or a path that cannot afford cudaMalloc's device-wide
synchronisation), so they cannot create a context.  This file checks, through the C ABI, that the
context-free call returns what dkv_score returns, on two calls in a row with different inputs (the
second call finds the first call's leftovers in the shared static scratch), and that a problem
larger than the static scratch is refused.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import dynamickv as O
from paper_2412_14838_b200 import binding as B
from paper_2412_14838_b200 import build, synth
from tests import _util as U

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


def test_static_scoring_matches_the_context_path_twice_in_a_row():
    build.build()
    B.load()
    # second shape: several key tiles per CTA, ragged tail, G = 3 (24 window rows)
    shapes = [synth.WORKLOADS["tiny"],
              synth.Workload("na", 61, L=2, Hq=6, Hkv=2, D=128, Bt=2, S=5003, ws=8, pool=7, N=8, Bl=16, m=1,
                             recipe="sink")]
    for w in shapes:
        ctx = B.dkv_create(B.config_of(w))
        try:
            for layer in range(2):                       # two calls in a row, different inputs
                t = synth.layer_inputs(w, layer, want_v=False)
                q, k = _dev(t["q"]), _dev(t["k"])
                want = torch.empty((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
                got = torch.full_like(want, -1.0)
                B.dkv_score(ctx, layer, q, k, want)
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                B.dkv_score_static(B.config_of(w), q, k, got)
                torch.cuda.synchronize()
                if layer == 1:                           # past the first call's one-time set-up
                    assert torch.cuda.mem_get_info()[0] == free_before, "the call took device memory"
                code, status = B.dkv_static_last_status()
                assert code == B.DKV_OK and status[0] == 0
                want, got = want.cpu().numpy(), got.cpu().numpy()
                assert (got >= 0).all(), "some scores were never written"
                rel = np.abs(got - want) / np.maximum(want, U.TINY)
                assert rel.max() <= U.REL_TOL, f"{w.name} call {layer}: off by {rel.max():.2e}"
                ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"]), w.ws, w.pool)
                U.assert_scores_close(got, ref["score"], f"{w.name} call {layer} against the oracle")
        finally:
            B.dkv_destroy(ctx)


def test_static_scoring_refuses_what_does_not_fit():
    build.build()
    B.load()
    # 4096 heads need about 16 MB of partial statistics: more than the static array
    big = B.make_config(L=1, Hq=4096, Hkv=4096, D=64, Bt=1, S=256, ws=16, pool=1, N=4, Bl=8, m=1)
    dummy = torch.zeros(16, dtype=torch.float32, device="cuda")
    with pytest.raises(B.DkvError) as e:
        B.dkv_score_static(big, dummy, dummy, dummy)
    assert e.value.code == B.DKV_ERR_TOO_LARGE
    with pytest.raises(B.DkvError) as e:
        B.dkv_score_static(B.config_of(synth.WORKLOADS["tiny"]), dummy, dummy, None)
    assert e.value.code == B.DKV_ERR_INVALID_ARG
