"""The seeded generators: determinism, bf16 rounding, and the structure each recipe plants."""
import numpy as np
import torch

from paper_2412_14838_b200 import synth


def test_bf16_rounding_matches_torch_rne():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 37
    x[:4] = [1.0, 1.00390625, 1.01171875, -0.0]          # ties: 1+2^-8 rounds to even
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (bits == ref).all()
    assert (synth.bf16_bits_to_f64(bits) == torch.from_numpy(x).to(torch.bfloat16).double().numpy()).all()


def test_layers_are_deterministic_and_independent():
    w = synth.WORKLOADS["tiny"]
    a, b = synth.layer_inputs(w, 2), synth.layer_inputs(w, 2)
    c = synth.layer_inputs(w, 3)
    for key in ("q", "k", "v"):
        assert a[key].dtype == np.uint16 and (a[key] == b[key]).all() and (a[key] != c[key]).any()
    assert a["q"].shape == (1, 8, 16, 64) and a["k"].shape == (1, 2, 1024, 64)


def test_sink_recipe_structure():
    w = synth.WORKLOADS["mistral8k"].with_(S=512)
    t = synth.layer_inputs(w, 0)
    k = synth.bf16_bits_to_f64(t["k"])
    q = synth.bf16_bits_to_f64(t["q"])
    # keys 0..3 are identical (the mean query) and aligned with the window queries of their group
    assert (k[0, :, 0] == k[0, :, 3]).all()
    for h in range(w.Hkv):
        mu = k[0, h, 0]
        qq = q[0, h * w.G:(h + 1) * w.G].reshape(-1, w.D)
        cos = qq @ mu / (np.linalg.norm(qq, axis=1) * np.linalg.norm(mu))
        assert cos.mean() > 0.5
        ch_std = k[0, h, 4:].std(axis=0)
        assert (ch_std > 4).sum() == 4                     # four outlier channels x8


def test_needle_recipe_structure():
    w = synth.WORKLOADS["needle32k"].with_(S=2048)
    starts = synth.needle_positions(w)
    assert len(starts) == 8 and (np.diff(starts) >= 16).all() and starts.min() >= 4
    assert synth.needle_token_mask(w).sum() == 128
    for layer, planted in ((0, False), (7, True), (23, True), (24, False)):
        t = synth.layer_inputs(w, layer, want_v=False)
        k = synth.bf16_bits_to_f64(t["k"])
        mu = k[0, 0, 0]
        span = k[0, 0, starts[0]:starts[0] + 16]
        cos = span @ mu / (np.linalg.norm(span, axis=1) * np.linalg.norm(mu))
        assert (cos.mean() > 0.85) == planted


def test_pooled_like_scores_have_ties():
    s = synth.pooled_like_scores((2, 3, 1000), pool=7, seed=1, tie_fraction=0.05)
    assert s.dtype == np.float32 and (s > 0).all()
    assert (np.diff(s, axis=-1) == 0).mean() > 0.3
