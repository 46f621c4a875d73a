"""CPU oracle for DynamicKV's prefill-time KV-cache compression (arXiv 2412.14838).

TEST INFRASTRUCTURE ONLY.  This file defines the right answer for the tests, the smoke
check and the benchmark's CPU-baseline leg.  It is plain NumPy in float64, slow on purpose,
and shares no code with the CUDA path; nothing in the product may import it.

Each function follows one passage of the paper, in the paper's order and notation
(``L`` layers, ``H`` = KV heads, ``G`` query heads per KV head, ``ws`` window, ``P = S - ws``
prefix tokens, ``N = wt - ws``, ``B^l`` = ``Bl`` per-layer maximum, ``m`` update interval):

* ``window_scores``        Eq. 1-2 and the scoring statement of Algorithm 1.
* ``window_lse``, ``window_scores_from_lse``  the same scores from Eq. 1's log-denominators (one sweep).
* ``select_topk``          Eq. 3 and Algorithm 1's per-layer ``topk(B^l)``.
* ``gather_rows``          Algorithm 1's gather of K/V plus the appended window.
* ``global_topk_counts``   Eq. 4: top-K over all accumulated layers and the count function Phi.
* ``budget_from_counts``   Eq. 5-6 with the ``int()`` truncations of Update_Buffer_Length.
* ``rebudget``             Update_Buffer_Length as a whole + the "buffers only shrink" clamp.
* ``shrink_rows``          Algorithm 1's truncation of every preceding layer's buffer.
* ``run_prefill_pass``     Algorithm 1's loop over layers (optionally scored from given log-denominators).
* ``decode_attention``     Eq. 1 applied to one new query over a layer's compressed, ragged cache (Section 4.3:
                           decoding runs unchanged over whatever the prefill phase kept).
* ``policy_counts``, ``positions_sinks_recent``   the fixed-pattern budgets the paper compares with (the
                           "Baselines" paragraph of Section 5.1), as budget / position policies only.

Alternative readings, off by default, selectable per call: the window MEAN instead of the sum, an
average pool (``avg_pool_same``), the pro-rata budget ``B = N * l`` at an intermediate update, and
min-max normalisation of the layer counts.

Readings taken where the paper is silent or inconsistent (each is listed in the design
notes): window reduction is a SUM over the ``ws`` window rows and the ``G`` query heads of a KV
head (the mean differs by a constant factor and selects the same tokens); logits are scaled by
``1/sqrt(d_k)`` (Eq. 1); the softmax of window row ``r`` runs over the keys it can see causally,
``0 .. P + r``, and only the prefix columns are kept afterwards; pooling is a stride-1 max-pool
of odd width over the prefix, borders ignoring the missing neighbours; ties are broken by the
lowest index (flat index, layer-major, for the global top-K); ``Norm`` is a positive scaling,
so Eq. 5 is evaluated in exact integers; counts never grow.

For the decode step: a hand-worked 3-key case (tests/golden/decode_handworked.txt), torch's masked softmax
attention on the padded buffers, invariance under a permutation of the kept rows, the single-row and
equal-keys special cases.  For the policies: hand-worked schedules (tests/golden/policies_handworked.txt),
their sums and monotonicity.
Pins (tests/test_oracle_*.py): closed forms for zero keys, probability-mass conservation,
a hand-worked 3-key softmax, an independent torch softmax / max_pool1d route, torch's logsumexp and the
ln 6 of the hand-worked case for the log-denominators, permutation
equivariance, brute-force subset enumeration for the top-k, hand-worked budget cases
(tests/golden/), full-sort brute force for the global counts, nestedness of shrink, and the
reduction of the whole pass to a plain top-N when ``r_max = 1`` and ``L = 1``.
Parity unpinned: nothing ties these outputs to the paper's LongBench / Needle-in-a-Haystack
accuracy tables (no weights or datasets are available).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------- scoring (Eq. 1-2)
def softmax_rows_causal(q_rows: np.ndarray, keys: np.ndarray, P: int) -> np.ndarray:
    """Eq. 1 restricted to the window rows: ``softmax(Q K^T / sqrt(d_k))`` row by row.

    ``q_rows`` [ws, D] are the queries at absolute positions ``P .. P+ws-1``; ``keys`` [S, D].
    Row ``r`` attends to keys ``0 .. P+r`` (causal); later keys get probability 0.
    Returns the [ws, S] probability matrix.
    """
    ws, D = q_rows.shape
    S = keys.shape[0]
    logits = (q_rows @ keys.T) / np.sqrt(np.float64(D))          # [ws, S]
    col = np.arange(S)[None, :]
    row = np.arange(ws)[:, None]
    visible = col <= (P + row)
    logits = np.where(visible, logits, -np.inf)
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    return e / e.sum(axis=1, keepdims=True)


def max_pool_same(x: np.ndarray, kernel: int) -> np.ndarray:
    """Stride-1 max-pool of odd width along the last axis; missing neighbours are ignored."""
    if kernel % 2 != 1 or kernel < 1:
        raise ValueError("pool kernel must be odd and >= 1")
    half = kernel // 2
    n = x.shape[-1]
    out = x.copy()
    for off in range(1, half + 1):
        if off >= n:
            break
        out[..., :-off] = np.maximum(out[..., :-off], x[..., off:])      # neighbour j + off
        out[..., off:] = np.maximum(out[..., off:], x[..., :-off])       # neighbour j - off
    return out


def avg_pool_same(x: np.ndarray, kernel: int) -> np.ndarray:
    """Stride-1 average pool of odd width along the last axis: the mean over the neighbours that exist
    (an alternative reading of the paper's unspecified "pooling"; the default is the max-pool above)."""
    if kernel % 2 != 1 or kernel < 1:
        raise ValueError("pool kernel must be odd and >= 1")
    half = kernel // 2
    n = x.shape[-1]
    tot = x.copy()
    cnt = np.ones(n, dtype=np.float64)
    for off in range(1, half + 1):
        if off >= n:
            break
        tot[..., :-off] += x[..., off:]
        tot[..., off:] += x[..., :-off]
        cnt[:-off] += 1
        cnt[off:] += 1
    return tot / cnt


def window_scores(q_win: np.ndarray, k: np.ndarray, ws: int, pool: int, *, pool_kind: int = 0,
                  window_mean: bool = False) -> Dict[str, np.ndarray]:
    """Eq. 2 / Algorithm 1's scoring line for one layer.

    ``q_win`` [Bt, Hq, ws, D] and ``k`` [Bt, Hkv, S, D] in float64 (exactly widened bf16).
    For every sample and KV head: sum, over the ``G`` query heads of the group and the ``ws``
    window rows, of the causal softmax probabilities on each prefix key, then max-pool.

    Returns ``score`` [Bt, Hkv, P] (pooled), ``raw`` [Bt, Hkv, P] (un-pooled) and ``window_mass``
    [Bt, Hkv] (probability that fell on the window's own columns), so that
    ``raw.sum(-1) + window_mass == ws * G`` can be checked.

    Variant readings: ``window_mean`` takes Algorithm 1's ``.mean`` over the window rows (and the group)
    instead of the sum, i.e. divides ``raw`` by ``ws * G``; ``pool_kind = 1`` pools with the average.
    """
    Bt, Hq, ws_, D = q_win.shape
    _, Hkv, S, _ = k.shape
    assert ws_ == ws and Hq % Hkv == 0
    G, P = Hq // Hkv, S - ws
    raw = np.zeros((Bt, Hkv, P), dtype=np.float64)
    wmass = np.zeros((Bt, Hkv), dtype=np.float64)
    for b in range(Bt):
        for h in range(Hkv):
            for g in range(G):
                A = softmax_rows_causal(q_win[b, h * G + g], k[b, h], P)   # [ws, S]
                raw[b, h] += A[:, :P].sum(axis=0)
                wmass[b, h] += A[:, P:].sum()
    if window_mean:
        raw = raw / float(ws * G)
    pooled = avg_pool_same(raw, pool) if pool_kind == 1 else max_pool_same(raw, pool)
    return {"score": pooled, "raw": raw, "window_mass": wmass}


def window_lse(q_win: np.ndarray, k: np.ndarray, ws: int) -> np.ndarray:
    """Natural logarithm of Eq. 1's softmax denominator for every window row: ``lse[b, hq, r] =
    ln sum_{i <= P + r} exp(q_r . k_i / sqrt(d_k))``, the value a prefill attention kernel returns
    beside its output.  ``q_win`` [Bt, Hq, ws, D], ``k`` [Bt, Hkv, S, D]; returns [Bt, Hq, ws]."""
    Bt, Hq, ws_, D = q_win.shape
    _, Hkv, S, _ = k.shape
    assert ws_ == ws and Hq % Hkv == 0
    G, P = Hq // Hkv, S - ws
    out = np.zeros((Bt, Hq, ws), dtype=np.float64)
    for b in range(Bt):
        for hq in range(Hq):
            logits = (q_win[b, hq] @ k[b, hq // G].T) / np.sqrt(np.float64(D))      # [ws, S]
            for r in range(ws):
                row = logits[r, :P + r + 1]
                top = row.max()
                out[b, hq, r] = top + np.log(np.exp(row - top).sum())
    return out


def window_scores_from_lse(q_win: np.ndarray, k: np.ndarray, lse: np.ndarray, ws: int, pool: int, *,
                           pool_kind: int = 0, window_mean: bool = False) -> Dict[str, np.ndarray]:
    """Eq. 2 with Eq. 1's denominators supplied: ``raw[j] = sum_{g, r} exp(q_{g,r} . k_j / sqrt(d_k) - lse[g, r])``
    over the prefix keys ``j < P``, then the pooling of ``window_scores``.  With ``lse = window_lse(...)`` this
    is the same quantity as ``window_scores`` computes by normalising each row."""
    Bt, Hq, ws_, D = q_win.shape
    _, Hkv, S, _ = k.shape
    assert ws_ == ws and Hq % Hkv == 0 and lse.shape == (Bt, Hq, ws)
    G, P = Hq // Hkv, S - ws
    raw = np.zeros((Bt, Hkv, P), dtype=np.float64)
    for b in range(Bt):
        for h in range(Hkv):
            for g in range(G):
                hq = h * G + g
                logits = (q_win[b, hq] @ k[b, h, :P].T) / np.sqrt(np.float64(D))     # [ws, P]
                raw[b, h] += np.exp(logits - lse[b, hq][:, None]).sum(axis=0)
    if window_mean:
        raw = raw / float(ws * G)
    pooled = avg_pool_same(raw, pool) if pool_kind == 1 else max_pool_same(raw, pool)
    return {"score": pooled, "raw": raw}


# --------------------------------------------------------------------------- per-head top-k (Eq. 3)
def select_topk(score: np.ndarray, Bl: int) -> Dict[str, np.ndarray]:
    """Eq. 3: the ``min(Bl, P)`` positions of one head with the largest score.

    Total order: score descending, then index ascending.  ``idx`` holds the kept positions in
    ascending order; ``rank[i]`` is the place of ``idx[i]`` in the total order (0 = best), which
    is the order Algorithm 1 stores them in and truncates by.
    """
    P = score.shape[0]
    keep = min(int(Bl), P)
    order = np.argsort(-score, kind="stable")          # stable => equal scores keep index order
    top = order[:keep]
    pos_sorted = np.sort(top)
    rank_of = np.empty(keep, dtype=np.int64)
    rank_of[np.searchsorted(pos_sorted, top)] = np.arange(keep)
    return {"idx": pos_sorted.astype(np.int64), "rank": rank_of}


def gather_rows(full: np.ndarray, idx: np.ndarray, ws: int) -> np.ndarray:
    """Algorithm 1's buffer build: kept prefix rows (ascending position), then the window rows.

    ``full`` [S, D] (any dtype; bytes are only moved).  Returns [len(idx) + ws, D].
    """
    S = full.shape[0]
    return np.concatenate([full[idx], full[S - ws:]], axis=0)


# --------------------------------------------------------------------------- re-budget (Eq. 4-6)
def global_topk_counts(history: Sequence[np.ndarray], k: int) -> np.ndarray:
    """Eq. 4's ``Phi(TopK(A, k))``: how many of the ``k`` largest scores fall in each layer.

    ``history`` is a list of per-layer arrays [H, P] (one sample).  The arrays are concatenated
    layer-major and flattened; ties go to the lowest flat index.
    """
    flat = np.concatenate([np.asarray(a, dtype=np.float64).reshape(-1) for a in history])
    per_layer = int(np.asarray(history[0]).size)
    k = min(int(k), flat.size)
    top = np.argsort(-flat, kind="stable")[:k]
    layer_of = top // per_layer
    return np.bincount(layer_of, minlength=len(history)).astype(np.int64)


def budget_from_counts(cnt: Sequence[int], Bl: int, N: int, L: int, *, prorata: bool = False,
                       minmax: bool = False) -> Dict[str, List[int]]:
    """Eq. 5 and Eq. 6 with Update_Buffer_Length's integer truncations.

    ``Z_i = floor(Bl * cnt_i / max(cnt))`` (any positive normalisation of the counts cancels),
    ``Z'_i = floor(Z_i * (N * L) / sum(Z))`` with ``B = N * L`` the global budget.

    Variant readings: ``prorata`` uses the budget of the layers seen so far, ``B = N * len(cnt)``, at an
    intermediate update; ``minmax`` reads "Norm ... range in (0,1)" as min-max normalisation,
    ``t_i = (cnt_i - min) / (max - min)`` (all ``t_i = 1`` when every layer has the same count), so that
    ``Z_i = floor(Bl * (cnt_i - min) / (max - min))``.
    """
    c = [int(x) for x in cnt]
    cmax = max(c)
    if cmax <= 0:
        raise ValueError("no hits in any layer")
    if minmax:
        cmin = min(c)
        Z = [int(Bl)] * len(c) if cmax == cmin else [(int(Bl) * (t - cmin)) // (cmax - cmin) for t in c]
    else:
        Z = [(int(Bl) * t) // cmax for t in c]
    total = sum(Z)
    B = int(N) * (len(c) if prorata else int(L))
    Zp = [(z * B) // total for z in Z]
    return {"Z": Z, "Zp": Zp}


def rebudget(history: Sequence[np.ndarray], counts: Sequence[int], N: int, Bl: int, L: int, *,
             prorata: bool = False, minmax: bool = False) -> Dict[str, List[int]]:
    """Update_Buffer_Length after ``l = len(history)`` layers for one sample.

    ``k = N * H * l`` entries are selected globally (all of them if fewer exist).  The new count of
    layer ``i < l`` is ``min(counts[i], Z'_i)``: buffers only ever shrink.
    """
    l = len(history)
    H, P = np.asarray(history[0]).shape
    k = min(int(N) * H * l, l * H * P)
    cnt = global_topk_counts(history, k)
    zz = budget_from_counts(cnt, Bl, N, L, prorata=prorata, minmax=minmax)
    new_counts = [int(x) for x in counts]
    for i in range(l):
        new_counts[i] = min(new_counts[i], zz["Zp"][i])
    return {"cnt": [int(x) for x in cnt], "Z": zz["Z"], "Zp": zz["Zp"], "counts": new_counts}


# --------------------------------------------------------------------------- progressive update
def shrink_rows(buf: np.ndarray, idx: np.ndarray, rank: np.ndarray, valid: int, new_count: int, ws: int):
    """Algorithm 1's truncation of one head's buffer to ``new_count`` kept rows + the window.

    ``buf`` [>= valid + ws, D] holds ``valid`` kept rows (ascending position) then ``ws`` window
    rows.  The rows whose rank is below ``new_count`` survive, in position order.
    Returns (rows [new_count' + ws, D], idx', rank') with ``new_count' = min(new_count, valid)``.
    """
    keep = np.nonzero(rank[:valid] < new_count)[0]
    rows = np.concatenate([buf[keep], buf[valid:valid + ws]], axis=0)
    return rows, idx[keep], rank[keep]


def run_prefill_pass(layer_fn, L: int, *, ws: int, pool: int, N: int, Bl: int, m: int, pool_kind: int = 0,
                     window_mean: bool = False, prorata: bool = False, minmax: bool = False,
                     lse_fn=None) -> Dict[str, object]:
    """Algorithm 1's loop over the layers, for all samples.

    ``layer_fn(l)`` returns one layer's inputs as a dict: ``q`` [Bt,Hq,ws,D] and ``k`` [Bt,Hkv,S,D]
    in float64 (used for scoring), and ``k_rows`` / ``v_rows`` [Bt,Hkv,S,D] in any dtype (the
    rows that are moved; typically the raw bf16 bit patterns).  A layer's full K/V is only
    touched while that layer is processed, as in the paper's prefill loop.  If ``L % m != 0``
    one more update runs after the last layer.  With ``lse_fn`` given, ``lse_fn(l)`` supplies layer ``l``'s
    log-denominators [Bt,Hq,ws] and the scores come from ``window_scores_from_lse`` (one sweep).

    Returns per layer: ``score`` [Bt,Hkv,P]; ``idx``/``rank`` lists [L][Bt][Hkv] of the final kept
    positions and their ranks; ``kb``/``vb`` lists [L][Bt][Hkv] of final buffers (kept rows then
    window rows); ``counts`` [Bt, L]; ``first_idx``/``first_rank`` as selected before any update;
    and ``updates`` = the trail of (layers done, per-sample rebudget results).
    """
    scores: List[np.ndarray] = []
    idx, rank, kb, vb, first_idx, first_rank = ([] for _ in range(6))
    counts = None
    updates = []

    def update(l_done: int):
        trail = []
        Bt, Hkv = counts.shape[0], len(idx[0][0])
        for b in range(Bt):
            res = rebudget([scores[i][b] for i in range(l_done)], counts[b], N, Bl, L, prorata=prorata, minmax=minmax)
            for i in range(l_done):
                new = res["counts"][i]
                valid = int(counts[b, i])
                for h in range(Hkv):
                    kb[i][b][h], idx_new, rank_new = shrink_rows(kb[i][b][h], idx[i][b][h], rank[i][b][h],
                                                                 valid, new, ws)
                    vb[i][b][h], _, _ = shrink_rows(vb[i][b][h], idx[i][b][h], rank[i][b][h], valid, new, ws)
                    idx[i][b][h], rank[i][b][h] = idx_new, rank_new
                counts[b, i] = new
            trail.append(res)
        updates.append((l_done, trail))

    for l in range(L):
        inp = layer_fn(l)
        Bt, Hkv, S, D = inp["k"].shape
        P = S - ws
        if counts is None:
            counts = np.zeros((Bt, L), dtype=np.int64)
        if lse_fn is None:
            sc = window_scores(inp["q"], inp["k"], ws, pool, pool_kind=pool_kind, window_mean=window_mean)["score"]
        else:
            sc = window_scores_from_lse(inp["q"], inp["k"], lse_fn(l), ws, pool, pool_kind=pool_kind,
                                        window_mean=window_mean)["score"]
        scores.append(sc)
        for lst in (idx, rank, kb, vb, first_idx, first_rank):
            lst.append([[None] * Hkv for _ in range(Bt)])
        for b in range(Bt):
            for h in range(Hkv):
                sel = select_topk(sc[b, h], Bl)
                idx[l][b][h], rank[l][b][h] = sel["idx"], sel["rank"]
                first_idx[l][b][h], first_rank[l][b][h] = sel["idx"], sel["rank"]
                kb[l][b][h] = gather_rows(inp["k_rows"][b, h], sel["idx"], ws)
                vb[l][b][h] = gather_rows(inp["v_rows"][b, h], sel["idx"], ws)
            counts[b, l] = min(Bl, P)
        del inp
        if (l + 1) % m == 0:
            update(l + 1)
    if L % m != 0:
        update(L)
    return {"score": scores, "idx": idx, "rank": rank, "kb": kb, "vb": vb, "counts": counts,
            "first_idx": first_idx, "first_rank": first_rank, "updates": updates}


# --------------------------------------------------------------------------- decoding over the compressed cache
def decode_attention(q_dec: np.ndarray, kb, vb, lengths: Sequence[int]) -> np.ndarray:
    """Eq. 1 for newly generated tokens over one layer's compressed cache (Section 4.3: the decoding phase
    is the model's own attention, run over what the prefill phase kept).

    ``q_dec`` [Bt, Hq, nq, D] float64: ``nq`` independent queries per sample and query head.  ``kb`` and
    ``vb`` are indexable as ``[b][h]`` and give that KV head's buffer [rows, D] (kept prefix rows followed by
    the ``ws`` window rows; rows past ``lengths[b]`` are padding and never read).  Query head ``hq`` reads KV
    head ``hq // G``.  Every query sees all ``lengths[b]`` rows: the cache holds only earlier positions.
    Returns [Bt, Hq, nq, D]: ``softmax(q K^T / sqrt(d_k)) V`` row by row.
    """
    Bt, Hq, nq, D = q_dec.shape
    Hkv = len(kb[0])
    assert Hq % Hkv == 0
    G = Hq // Hkv
    out = np.zeros((Bt, Hq, nq, D), dtype=np.float64)
    for b in range(Bt):
        n = int(lengths[b])
        for hq in range(Hq):
            K = np.asarray(kb[b][hq // G], dtype=np.float64)[:n]
            V = np.asarray(vb[b][hq // G], dtype=np.float64)[:n]
            for i in range(nq):
                logits = (K @ q_dec[b, hq, i]) / np.sqrt(np.float64(D))
                e = np.exp(logits - logits.max())
                out[b, hq, i] = (e / e.sum()) @ V
    return out


# --------------------------------------------------------------------------- fixed-pattern policies
def policy_counts(policy: str, L: int, N: int) -> List[int]:
    """Per-layer budgets of the fixed-pattern methods the paper compares with, as plain schedules (no
    scores involved): ``"uniform"`` keeps the same ``N`` tokens per head in every layer (the fixed
    per-layer cache of SnapKV-like methods); ``"pyramid"`` decreases monotonically with depth (the pyramid
    pattern): ``N + floor(N * (L - 1 - 2 i) / (2 (L - 1)))`` for layer ``i``, i.e. linearly from about
    ``3N/2`` at the first layer to ``N/2`` at the last, summing to ``N * L`` up to the floors (``N``
    when ``L = 1``).  The kept tokens are then the best ``count_i`` of each head under Eq. 3's order."""
    if policy == "uniform":
        return [int(N)] * L
    if policy == "pyramid":
        if L == 1:
            return [int(N)]
        return [int(N) + (int(N) * (L - 1 - 2 * i)) // (2 * (L - 1)) for i in range(L)]
    raise ValueError(f"unknown policy {policy!r}")


def positions_sinks_recent(P: int, n_sink: int, n_recent: int) -> np.ndarray:
    """Kept prefix positions of a sinks-plus-recent cache (attention sinks and a rolling window of the most
    recent tokens, StreamingLLM-like): the first ``n_sink`` and the last ``n_recent`` of the ``P`` prefix
    positions, ascending, each once (the two ranges merge when they meet)."""
    n_sink, n_recent = max(0, min(int(n_sink), P)), max(0, min(int(n_recent), P))
    first_recent = max(P - n_recent, n_sink)
    return np.concatenate([np.arange(n_sink), np.arange(first_recent, P)]).astype(np.int64)
