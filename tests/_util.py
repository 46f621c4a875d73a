"""Shared helpers of the parity tests: oracle runs on seeded inputs, near-tie accounting."""
from __future__ import annotations

import numpy as np

from oracle import dynamickv as O
from paper_2412_14838_b200 import synth

REL_TOL = 1e-3          # scores: max relative error, bf16 inputs / fp32 accumulation
NEAR_TIE = 1e-5         # relative score gap below which two candidates count as tied at a cut
TINY = 1e-30            # scores below this are compared absolutely (fp32 flushes them to zero)


def oracle_inputs(w, layer, seed=synth.BASE_SEED):
    t = synth.layer_inputs(w, layer, seed)
    return {"q": synth.bf16_bits_to_f64(t["q"]), "k": synth.bf16_bits_to_f64(t["k"]),
            "k_rows": t["k"], "v_rows": t["v"], "bits": t}


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    big = ref >= TINY
    rel = np.abs(gpu[big] - ref[big]) / ref[big]
    worst = float(rel.max()) if rel.size else 0.0
    assert worst <= REL_TOL, f"{what}: max relative score error {worst:.3e} > {REL_TOL}"
    assert (np.abs(gpu[~big] - ref[~big]) <= 1e-33).all(), f"{what}: tiny scores differ"
    return worst


def select_matches(ref_score: np.ndarray, gpu_idx: np.ndarray, keep: int):
    """Compare a kept set with the oracle's top-`keep`.  Returns (exact, near_tie_events).

    A difference is tolerated only if every element on either side of it lies within NEAR_TIE
    (relative) of the oracle's cut, i.e. of the scores ranked keep and keep+1.
    """
    ref = O.select_topk(ref_score, keep)["idx"]
    gpu_idx = np.asarray(gpu_idx, dtype=np.int64)
    assert gpu_idx.shape == ref.shape, f"kept {gpu_idx.shape} vs oracle {ref.shape}"
    assert (np.diff(gpu_idx) > 0).all(), "kept positions not ascending/unique"
    if (gpu_idx == ref).all():
        return True, 0
    only_g = np.setdiff1d(gpu_idx, ref)
    only_o = np.setdiff1d(ref, gpu_idx)
    order = np.sort(ref_score)[::-1]
    cut_hi, cut_lo = order[keep - 1], order[min(keep, len(order) - 1)]
    lo = cut_lo * (1 - NEAR_TIE)
    hi = cut_hi * (1 + NEAR_TIE)
    bad = [int(p) for p in np.concatenate([only_g, only_o]) if not (lo <= ref_score[p] <= hi)]
    assert not bad, f"kept sets differ away from the cut at positions {bad[:8]}"
    assert (cut_hi - cut_lo) <= NEAR_TIE * cut_hi, "kept sets differ although the cut is not a near-tie"
    return False, len(only_g)


def global_cut_gap(history, k):
    """Relative gap between the k-th and (k+1)-th largest entries of the flattened history."""
    flat = np.concatenate([np.asarray(a, dtype=np.float64).reshape(-1) for a in history])
    if k >= flat.size:
        return np.inf
    part = np.partition(flat, flat.size - k - 1)
    lo = part[flat.size - k - 1]
    hi = part[flat.size - k:].min()
    return (hi - lo) / hi if hi > 0 else 0.0


def buffer_order(rows: np.ndarray, rank: np.ndarray, n: int) -> np.ndarray:
    """Oracle rows (kept rows in position order, then window rows) rearranged into the library's buffer
    order: kept rows by rank (score descending, ties by position), window rows last."""
    order = np.argsort(np.asarray(rank[:n]), kind="stable")
    return np.concatenate([rows[:n][order], rows[n:]], axis=0)
