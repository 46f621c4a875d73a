"""Seeded synthetic inputs for DynamicKV prefill-time KV-cache compression.

This module only *draws data*: window queries, keys and values as bf16 bit patterns
(``uint16``), shaped like the paper's workloads (Table 3: 32 layers, 32 query / 8 KV heads,
head size 128; Section 5.1: 8K-32K contexts; cache sizes 64/128/512).  It holds none of the
method's arithmetic (no softmax, no pooling, no top-k, no budget maths), so both the CPU
oracle's tests and the CUDA path's tests may use it without sharing method code.

Every tensor of every layer comes from its own counter-based Philox stream keyed by
``(seed, config id, tensor id, layer)``, so a layer can be drawn alone, in any order, on any
machine, and always gives the same bits.

Notation (paper -> here): ``L`` layers, ``Hq``/``Hkv`` query/KV heads, ``G = Hq/Hkv``,
``D = d_k``, ``S`` prompt length including the window, ``ws`` window, ``P = S - ws`` prefix,
``N = wt - ws`` average retained prefix tokens per head per layer, ``Bl = B^l`` per-layer
maximum, ``m`` update interval.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

BASE_SEED = 20241214

_T_Q, _T_K, _T_V, _T_MU, _T_AUX, _T_SCORES, _T_QDEC = 1, 2, 3, 4, 5, 6, 7


@dataclass(frozen=True)
class Workload:
    """Shape + budget parameters of one compression problem, plus its input recipe."""

    name: str
    cid: int                 # config id mixed into the Philox key
    L: int
    Hq: int
    Hkv: int
    D: int
    Bt: int
    S: int
    ws: int
    pool: int                # odd max-pool kernel
    N: int                   # average budget, tokens / head / layer (window excluded)
    Bl: int                  # per-layer maximum  B^l = N * r_max
    m: int                   # update interval
    recipe: str              # "iid" | "sink" | "layervar" | "needle"

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def P(self) -> int:
        return self.S - self.ws

    @property
    def M(self) -> int:
        """Window-query rows scored per KV head (``ws * G``)."""
        return self.ws * self.G

    @property
    def Blc(self) -> int:
        """Per-layer maximum clamped to the number of candidates."""
        return min(self.Bl, self.P)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    def algorithmic_bytes(self) -> int:
        """K read once + kept K/V rows read and written (first compaction of each layer)."""
        per_head = self.S * self.D * 2 + 2 * 2 * (self.Blc + self.ws) * self.D * 2
        return self.L * self.Bt * self.Hkv * per_head

    def k_bytes_per_layer(self) -> int:
        return self.Bt * self.Hkv * self.S * self.D * 2


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("tiny", 1, L=4, Hq=8, Hkv=2, D=64, Bt=1, S=1024, ws=16, pool=5, N=64, Bl=128, m=2,
                 recipe="iid"),
        Workload("mistral8k", 2, L=32, Hq=32, Hkv=8, D=128, Bt=1, S=8192, ws=32, pool=7, N=128,
                 Bl=512, m=4, recipe="sink"),
        Workload("mistral32k", 3, L=32, Hq=32, Hkv=8, D=128, Bt=1, S=32768, ws=32, pool=7, N=512,
                 Bl=2048, m=4, recipe="layervar"),
        Workload("llama16k_b4", 4, L=32, Hq=32, Hkv=8, D=128, Bt=4, S=16384, ws=32, pool=7, N=64,
                 Bl=256, m=4, recipe="sink"),
        Workload("needle32k", 5, L=32, Hq=32, Hkv=8, D=128, Bt=1, S=32768, ws=32, pool=7, N=64,
                 Bl=512, m=4, recipe="needle"),
        # a second model shape: 28 layers, 28 query / 4 KV heads (G = 7, 224 window rows: not a power of two)
        Workload("qwen16k", 6, L=28, Hq=28, Hkv=4, D=128, Bt=1, S=16384, ws=32, pool=7, N=128,
                 Bl=512, m=4, recipe="sink"),
    ]
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def _rng(seed: int, cid: int, tensor: int, layer: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64((cid << 40) | (tensor << 32) | (layer & 0xFFFFFFFF))],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _normal(g: np.random.Generator, shape) -> np.ndarray:
    return g.standard_normal(size=shape, dtype=np.float32)


def needle_positions(w: Workload, seed: int = BASE_SEED, spans: int = 8, span_len: int = 16) -> np.ndarray:
    """Start positions of the planted spans (shared by all layers), non-overlapping, in [4, P - span_len)."""
    g = _rng(seed, w.cid, _T_AUX, 0xFFFF)
    starts = []
    while len(starts) < spans:
        s = int(g.integers(4, w.P - span_len))
        if all(abs(s - t) >= span_len for t in starts):
            starts.append(s)
    return np.array(sorted(starts), dtype=np.int64)


def needle_token_mask(w: Workload, seed: int = BASE_SEED, spans: int = 8, span_len: int = 16) -> np.ndarray:
    mask = np.zeros(w.P, dtype=bool)
    for s in needle_positions(w, seed, spans, span_len):
        mask[s:s + span_len] = True
    return mask


def layer_inputs(w: Workload, layer: int, seed: int = BASE_SEED, want_v: bool = True) -> Dict[str, np.ndarray]:
    """Draw one layer's ``q`` [Bt,Hq,ws,D], ``k`` and ``v`` [Bt,Hkv,S,D] as bf16 bit patterns.

    Recipes (``layer`` is 0-based here; the needle recipe's "layers 8-24" are 1-based inclusive):

    * ``iid``      q, k, v ~ N(0,1).
    * ``sink``     k ~ N(0,1) with 4 seeded channels per (layer, KV head) scaled by 8; a mean query
                   direction mu ~ N(0,1) per (sample, KV head); q = mu + eps; keys 0..3 set to mu.
    * ``layervar`` as ``sink`` plus, per layer, n_l in [0,4096] seeded positions per head whose key is
                   sqrt(1-c_l^2) eps + c_l sqrt(D) mu/|mu| with c_l in [0,0.6] drawn per layer.
    * ``needle``   as ``sink``; in 1-based layers 8..24 the planted span keys are
                   0.9 sqrt(D) mu/|mu| + sqrt(0.19) eps and q = mu + 0.3 eps.
    """
    Bt, Hq, Hkv, D, S, ws, G = w.Bt, w.Hq, w.Hkv, w.D, w.S, w.ws, w.G
    gq, gk, gv = (_rng(seed, w.cid, t, layer) for t in (_T_Q, _T_K, _T_V))
    k = _normal(gk, (Bt, Hkv, S, D))
    eps_q = _normal(gq, (Bt, Hq, ws, D))
    out: Dict[str, np.ndarray] = {}
    if w.recipe == "iid":
        q = eps_q
    else:
        gm, ga = _rng(seed, w.cid, _T_MU, layer), _rng(seed, w.cid, _T_AUX, layer)
        mu = _normal(gm, (Bt, Hkv, D))
        mu_hat = mu / np.linalg.norm(mu, axis=-1, keepdims=True)
        for h in range(Hkv):
            ch = ga.choice(D, size=4, replace=False)
            k[:, h, :, ch] *= np.float32(8.0)
        q_noise = np.float32(1.0)
        if w.recipe == "layervar":
            n_l = int(ga.integers(0, 4097))
            c_l = np.float32(ga.uniform(0.0, 0.6))
            n_l = min(n_l, w.P - 4)
            for b in range(Bt):
                for h in range(Hkv):
                    pos = 4 + ga.choice(w.P - 4, size=n_l, replace=False)
                    k[b, h, pos, :] = (np.sqrt(np.float32(1.0) - c_l * c_l) * k[b, h, pos, :]
                                       + c_l * np.float32(np.sqrt(D)) * mu_hat[b, h])
        elif w.recipe == "needle" and 8 <= layer + 1 <= 24:
            q_noise = np.float32(0.3)
            gn = _rng(seed, w.cid, _T_AUX, 0x10000 + layer)
            for s0 in needle_positions(w, seed):
                e = _normal(gn, (Bt, Hkv, 16, D))
                k[:, :, s0:s0 + 16, :] = (np.float32(0.9 * np.sqrt(D)) * mu_hat[:, :, None, :]
                                          + np.float32(np.sqrt(0.19)) * e)
        k[:, :, 0:4, :] = mu[:, :, None, :]
        q = np.repeat(mu, G, axis=1)[:, :, None, :] + q_noise * eps_q
    out["q"] = f32_to_bf16_bits(q)
    out["k"] = f32_to_bf16_bits(k)
    del k
    if want_v:
        out["v"] = f32_to_bf16_bits(_normal(gv, (Bt, Hkv, S, D)))
    return out


def decode_queries(w: Workload, layer: int, nq: int = 1, seed: int = BASE_SEED) -> np.ndarray:
    """Queries of ``nq`` newly generated tokens per sample for one layer, bf16 bit patterns [Bt, Hq, nq, D]:
    N(0,1) plus, for the recipes that have one, the layer's mean query direction of the head group (so that the
    decode step attends to the same sinks and planted keys as the window queries did)."""
    g = _rng(seed, w.cid, _T_QDEC, layer)
    q = _normal(g, (w.Bt, w.Hq, nq, w.D))
    if w.recipe != "iid":
        mu = _normal(_rng(seed, w.cid, _T_MU, layer), (w.Bt, w.Hkv, w.D))
        q = q + np.repeat(mu, w.G, axis=1)[:, :, None, :]
    return f32_to_bf16_bits(q)


def pooled_like_scores(shape, pool: int, seed: int, tie_fraction: float = 0.0) -> np.ndarray:
    """Positive float32 arrays with runs of exactly equal neighbours, as max-pooling produces.

    Pure data for selection tests: log-normal values, each repeated over a run of 1..pool
    positions along the last axis; optionally a fraction of all entries is overwritten with one
    shared value so that ties also occur across heads and layers.
    """
    g = _rng(seed, 0, _T_SCORES, 0)
    n = int(np.prod(shape))
    base = np.exp(_normal(g, (n,)) * np.float32(1.5) - np.float32(8.0)).astype(np.float32)
    runs = g.integers(1, pool + 1, size=n)
    starts = np.cumsum(runs) - runs
    starts = starts[starts < n]
    src = np.zeros(n, dtype=np.int64)
    src[starts] = 1
    src = np.cumsum(src) - 1
    out = base[starts][src]
    if tie_fraction > 0:
        hit = g.random(n) < tie_fraction
        out[hit] = np.float32(np.median(base))
    return out.reshape(shape)
