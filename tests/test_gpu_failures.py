"""Failure reporting of the library on the GPU, exercised without faulting it.

The scoring kernel waits on mbarriers (copies landed, accumulators ready, stages free).  Every such wait is
bounded; when one runs out the thread block stops issuing work, drains what it has in flight, frees its
tensor memory and ends, and the host reads DKV_ERR_TIMEOUT from dkv_last_status.  The test makes a wait run
out the harmless way: the copy of one key tile is simply never issued (dkv_debug_withhold_tile), with the
wait limit set to about a millisecond.  Nothing traps, no address is invalid, the context stays usable.
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


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


@pytest.mark.parametrize("sweep", [1, 2])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(sweep):
    w = synth.WORKLOADS["tiny"]
    t = synth.layer_inputs(w, 0, want_v=False)
    q, k = _dev(t["q"]), _dev(t["k"])
    ref = O.window_scores(synth.bf16_bits_to_f64(t["q"]), synth.bf16_bits_to_f64(t["k"]), w.ws, w.pool)["score"]
    ctx = B.dkv_create(B.config_of(w))
    try:
        out = torch.zeros((w.Bt, w.Hkv, w.P), dtype=torch.float32, device="cuda")
        B.dkv_set_wait_limit(ctx, 2_000_000)              # about a millisecond of SM clock
        B.dkv_debug_withhold_tile(ctx, sweep, 0)           # block 0 never gets its first key tile of that sweep
        B.dkv_score(ctx, 0, q, k, out)                     # enqueues; the kernels end by themselves
        torch.cuda.synchronize()
        code, status = B.dkv_last_status(ctx)
        assert code == B.DKV_ERR_TIMEOUT, f"expected a timeout report, got {code} {status}"
        assert 101 <= status[0] <= 107 and status[2] == 0, status
        assert "timed out" in B.strerror(code)
        code, status = B.dkv_last_status(ctx)              # reported once
        assert code == B.DKV_OK and status[0] == 0
        # the same context, hook off: a normal call gives the right scores
        B.dkv_debug_withhold_tile(ctx, 0, -1)
        B.dkv_set_wait_limit(ctx, 4_000_000_000)
        B.dkv_score(ctx, 0, q, k, out)
        torch.cuda.synchronize()
        code, status = B.dkv_last_status(ctx)
        assert code == B.DKV_OK and status[0] == 0
        U.assert_scores_close(out.cpu().numpy(), ref, "after a reported timeout")
    finally:
        B.dkv_destroy(ctx)


def test_wait_limit_and_hook_arguments_are_checked():
    ctx = B.dkv_create(B.config_of(synth.WORKLOADS["tiny"]))
    try:
        with pytest.raises(B.DkvError) as e:
            B.dkv_set_wait_limit(ctx, 10)
        assert e.value.code == B.DKV_ERR_INVALID_ARG
        with pytest.raises(B.DkvError) as e:
            B.dkv_debug_withhold_tile(ctx, 3, 0)
        assert e.value.code == B.DKV_ERR_INVALID_ARG
    finally:
        B.dkv_destroy(ctx)


def test_two_live_contexts_with_different_layer_budgets():
    """The select kernel's shared-memory attribute belongs to the kernel, not to a context: a second context with
    a small per-layer maximum must not break the first one's launches."""
    big = synth.Workload("bigbl", 71, L=1, Hq=2, Hkv=1, D=64, Bt=1, S=12000, ws=8, pool=3, N=4096, Bl=8192, m=1,
                         recipe="iid")
    small = synth.Workload("smallbl", 72, L=1, Hq=2, Hkv=1, D=64, Bt=1, S=600, ws=8, pool=3, N=16, Bl=32, m=1,
                           recipe="iid")
    a = B.dkv_create(B.config_of(big))
    b = B.dkv_create(B.config_of(small))                   # created second, needs far less shared memory
    try:
        for ctx, w in ((a, big), (b, small), (a, big)):
            sc = synth.pooled_like_scores((w.Bt, w.Hkv, w.P), w.pool, seed=w.cid, tie_fraction=0.2)
            B.dkv_set_scores(ctx, 0, torch.from_numpy(sc).cuda())
            idx = torch.zeros((w.Bt, w.Hkv, w.Blc), dtype=torch.int32, device="cuda")
            B.dkv_select_topk(ctx, 0, idx)
            torch.cuda.synchronize()
            want = O.select_topk(sc[0, 0].astype(np.float64), w.Bl)["idx"]
            assert (idx.cpu().numpy()[0, 0] == want).all()
    finally:
        B.dkv_destroy(a)
        B.dkv_destroy(b)
