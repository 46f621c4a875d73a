"""ctypes view of libdkv.so: the same entry points as include/dkv.h, argument marshalling only.

Every step of the path runs inside the CUDA library; this module converts torch tensors (or raw
integer addresses) to pointers, passes the current CUDA stream, and raises ``DkvError`` on a
non-zero return code.  There is no CPU fallback: ``load()`` raises when the library is missing.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdkv.so")

EXPORTS = [
    "dkv_create", "dkv_destroy", "dkv_reset", "dkv_score", "dkv_score_static", "dkv_score_lse", "dkv_set_scores", "dkv_select_topk", "dkv_rebudget",
    "dkv_compact", "dkv_compact_all", "dkv_run_prefill_pass", "dkv_run_prefill_pass_lse", "dkv_run_prefill_pass_host", "dkv_host_pass_bytes",
    "dkv_apply_policy", "dkv_select_positions", "dkv_decode_attend", "dkv_get_counts",
    "dkv_layer_views", "dkv_kept_sorted", "dkv_budget_views", "dkv_memcpy_to_host", "dkv_last_status",
    "dkv_static_last_status", "dkv_set_wait_limit", "dkv_debug_withhold_tile", "dkv_profile", "dkv_profile_read", "dkv_launch_count", "dkv_last_cuda_error",
    "dkv_strerror", "dkv_version",
]

DKV_OK, DKV_ERR_INVALID_ARG, DKV_ERR_STATE, DKV_ERR_CUDA = 0, -1, -2, -3
DKV_ERR_TIMEOUT, DKV_ERR_UNSUPPORTED, DKV_ERR_NOMEM, DKV_ERR_TOO_LARGE = -4, -5, -6, -7


class DkvConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "batch", "seq_len", "window", "pool_kernel",
        "pool_kind", "avg_budget", "layer_max", "update_interval")] + [("flags", ctypes.c_uint32)]


class DkvError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {code} ({strerror(code)})")


_lib = None


def load() -> ctypes.CDLL:
    """Load libdkv.so (built by ``paper_2412_14838_b200.build``); fail loudly if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2412_14838_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, pp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_void_p)
    sig = {
        "dkv_create": [ctypes.POINTER(DkvConfig), pp],
        "dkv_destroy": [vp],
        "dkv_reset": [vp, vp],
        "dkv_score": [vp, i32, vp, vp, vp, vp],
        "dkv_score_static": [ctypes.POINTER(DkvConfig), vp, vp, vp, vp],
        "dkv_score_lse": [vp, i32, vp, vp, vp, vp, vp],
        "dkv_set_scores": [vp, i32, vp, vp],
        "dkv_select_topk": [vp, i32, vp, vp, vp],
        "dkv_rebudget": [vp, i32, vp, vp],
        "dkv_compact": [vp, i32, vp, vp, vp, vp, vp, vp],
        "dkv_compact_all": [vp, i32, pp, pp, vp],
        "dkv_run_prefill_pass": [vp, pp, pp, pp, pp, pp, vp],
        "dkv_run_prefill_pass_host": [vp, pp, pp, pp, pp, pp, vp],
        "dkv_run_prefill_pass_lse": [vp, pp, pp, pp, pp, pp, pp, vp],
        "dkv_host_pass_bytes": [vp, vp, vp],
        "dkv_apply_policy": [vp, i32, vp, vp],
        "dkv_select_positions": [vp, i32, i32, i32, vp],
        "dkv_decode_attend": [vp, i32, i32, i32, pp, pp, pp, pp, vp],
        "dkv_get_counts": [vp, vp, vp],
        "dkv_layer_views": [vp, i32, pp, pp],
        "dkv_kept_sorted": [vp, i32, vp, vp],
        "dkv_budget_views": [vp, pp, pp, pp, pp],
        "dkv_memcpy_to_host": [vp, vp, vp, ctypes.c_uint64, vp],
        "dkv_last_status": [vp, vp],
        "dkv_static_last_status": [vp],
        "dkv_set_wait_limit": [vp, ctypes.c_int64],
        "dkv_debug_withhold_tile": [vp, i32, i32],
        "dkv_profile": [vp, ctypes.c_int],
        "dkv_profile_read": [vp, vp, vp],
        "dkv_last_cuda_error": [vp],
        "dkv_strerror": [ctypes.c_int],
        "dkv_version": [],
        "dkv_launch_count": [vp],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = ctypes.c_int
    lib.dkv_strerror.restype = ctypes.c_char_p
    lib.dkv_launch_count.restype = ctypes.c_int64
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().dkv_strerror(code).decode()


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / int; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)}")


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _ptr_array(items: Sequence) -> ctypes.Array:
    arr = (ctypes.c_void_p * len(items))()
    for i, it in enumerate(items):
        arr[i] = _ptr(it)
    return arr


def _check(code: int, what: str) -> None:
    if code != 0:
        raise DkvError(code, what)


# dkv_config.flags: alternative readings of the paper (see include/dkv.h)
DKV_F_WINDOW_MEAN = 0x1
DKV_F_PRORATA = 0x2
DKV_F_NORM_MINMAX = 0x4


def make_config(L, Hq, Hkv, D, Bt, S, ws, pool, N, Bl, m, pool_kind=0, flags=0) -> DkvConfig:
    return DkvConfig(L, Hq, Hkv, D, Bt, S, ws, pool, pool_kind, N, Bl, m, flags)


def config_of(w, pool_kind: int = 0, flags: int = 0) -> DkvConfig:
    """DkvConfig of a ``synth.Workload``-like object (fields L,Hq,Hkv,D,Bt,S,ws,pool,N,Bl,m)."""
    return make_config(w.L, w.Hq, w.Hkv, w.D, w.Bt, w.S, w.ws, w.pool, w.N, w.Bl, w.m, pool_kind, flags)


# ---- the entry points, same names as the C ABI ----------------------------------------------------
def dkv_version() -> int:
    return load().dkv_version()


def dkv_create(cfg: DkvConfig) -> int:
    h = ctypes.c_void_p()
    _check(load().dkv_create(ctypes.byref(cfg), ctypes.byref(h)), "dkv_create")
    return h.value


def dkv_destroy(ctx: int) -> None:
    _check(load().dkv_destroy(ctx), "dkv_destroy")


def dkv_reset(ctx: int, stream=None) -> None:
    _check(load().dkv_reset(ctx, _stream(stream)), "dkv_reset")


def dkv_score(ctx: int, layer: int, q_win, k, scores_out=None, stream=None) -> None:
    _check(load().dkv_score(ctx, layer, _ptr(q_win), _ptr(k), _ptr(scores_out), _stream(stream)), "dkv_score")


def dkv_score_static(cfg: DkvConfig, q_win, k, scores_out, stream=None) -> None:
    """Score one layer without a context and without any device allocation (see include/dkv.h)."""
    _check(load().dkv_score_static(ctypes.byref(cfg), _ptr(q_win), _ptr(k), _ptr(scores_out), _stream(stream)),
           "dkv_score_static")


def dkv_score_lse(ctx: int, layer: int, q_win, k, lse, scores_out=None, stream=None) -> None:
    """Score one layer in a single sweep, given the window rows' log-sum-exp fp32 [Bt, Hq, ws] (see include/dkv.h)."""
    _check(load().dkv_score_lse(ctx, layer, _ptr(q_win), _ptr(k), _ptr(lse), _ptr(scores_out), _stream(stream)),
           "dkv_score_lse")


def dkv_set_scores(ctx: int, layer: int, scores, stream=None) -> None:
    _check(load().dkv_set_scores(ctx, layer, _ptr(scores), _stream(stream)), "dkv_set_scores")


def dkv_select_topk(ctx: int, layer: int, idx_out=None, rank_out=None, stream=None) -> None:
    _check(load().dkv_select_topk(ctx, layer, _ptr(idx_out), _ptr(rank_out), _stream(stream)), "dkv_select_topk")


def dkv_rebudget(ctx: int, upto_layer: int, counts_out=None, stream=None) -> None:
    _check(load().dkv_rebudget(ctx, upto_layer, _ptr(counts_out), _stream(stream)), "dkv_rebudget")


def dkv_compact(ctx: int, layer: int, k_src, v_src, kb, vb, len_out=None, stream=None) -> None:
    _check(load().dkv_compact(ctx, layer, _ptr(k_src), _ptr(v_src), _ptr(kb), _ptr(vb), _ptr(len_out),
                              _stream(stream)), "dkv_compact")


def dkv_compact_all(ctx: int, upto_layer: int, kb: Sequence, vb: Sequence, stream=None) -> None:
    _check(load().dkv_compact_all(ctx, upto_layer, _ptr_array(kb), _ptr_array(vb), _stream(stream)),
           "dkv_compact_all")


def dkv_run_prefill_pass(ctx: int, q_win: Sequence, k: Sequence, v: Sequence, kb: Sequence, vb: Sequence,
                         stream=None) -> None:
    _check(load().dkv_run_prefill_pass(ctx, _ptr_array(q_win), _ptr_array(k), _ptr_array(v), _ptr_array(kb),
                                       _ptr_array(vb), _stream(stream)), "dkv_run_prefill_pass")


def dkv_run_prefill_pass_host(ctx: int, q_win: Sequence, k: Sequence, v: Sequence, kb: Sequence, vb: Sequence,
                              counts_out=None) -> None:
    _check(load().dkv_run_prefill_pass_host(ctx, _ptr_array(q_win), _ptr_array(k), _ptr_array(v), _ptr_array(kb),
                                            _ptr_array(vb), _ptr(counts_out)), "dkv_run_prefill_pass_host")


def dkv_host_pass_bytes(ctx: int):
    """(host-to-device, device-to-host) bytes moved by the context's last dkv_run_prefill_pass_host."""
    h2d, d2h = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(load().dkv_host_pass_bytes(ctx, ctypes.byref(h2d), ctypes.byref(d2h)), "dkv_host_pass_bytes")
    return int(h2d.value), int(d2h.value)


def dkv_run_prefill_pass_lse(ctx: int, q_win: Sequence, k: Sequence, v: Sequence, lse: Sequence, kb: Sequence,
                             vb: Sequence, stream=None) -> None:
    """The pass with every layer scored in one sweep from the window rows' log-denominators (see include/dkv.h)."""
    _check(load().dkv_run_prefill_pass_lse(ctx, _ptr_array(q_win), _ptr_array(k), _ptr_array(v), _ptr_array(lse),
                                           _ptr_array(kb), _ptr_array(vb), _stream(stream)), "dkv_run_prefill_pass_lse")


DKV_POLICY_UNIFORM, DKV_POLICY_PYRAMID = 0, 1


def dkv_apply_policy(ctx: int, policy: int, counts_out=None, stream=None) -> None:
    _check(load().dkv_apply_policy(ctx, policy, _ptr(counts_out), _stream(stream)), "dkv_apply_policy")


def dkv_select_positions(ctx: int, layer: int, n_sink: int, n_recent: int, stream=None) -> None:
    _check(load().dkv_select_positions(ctx, layer, n_sink, n_recent, _stream(stream)), "dkv_select_positions")


def dkv_decode_attend(ctx: int, layer0: int, n_layers: int, nq: int, q_dec: Sequence, kb: Sequence, vb: Sequence,
                      out: Sequence, stream=None) -> None:
    """Attention of nq new queries per sample over the compressed buffers of layers [layer0, layer0 + n_layers)."""
    _check(load().dkv_decode_attend(ctx, layer0, n_layers, nq, _ptr_array(q_dec), _ptr_array(kb), _ptr_array(vb),
                                    _ptr_array(out), _stream(stream)), "dkv_decode_attend")


def dkv_get_counts(ctx: int, host_counts, stream=None) -> None:
    _check(load().dkv_get_counts(ctx, _ptr(host_counts), _stream(stream)), "dkv_get_counts")


def dkv_layer_views(ctx: int, layer: int):
    """Device addresses (scores, kept positions in buffer order) of one layer's state inside the context."""
    a, b = ctypes.c_void_p(), ctypes.c_void_p()
    _check(load().dkv_layer_views(ctx, layer, ctypes.byref(a), ctypes.byref(b)), "dkv_layer_views")
    return a.value, b.value


def dkv_kept_sorted(ctx: int, layer: int, sorted_out, stream=None) -> None:
    _check(load().dkv_kept_sorted(ctx, layer, _ptr(sorted_out), _stream(stream)), "dkv_kept_sorted")


def dkv_budget_views(ctx: int):
    """Device addresses (cnt, Z, Z', held), int32 [Bt, L] each."""
    v = [ctypes.c_void_p() for _ in range(4)]
    _check(load().dkv_budget_views(ctx, *[ctypes.byref(x) for x in v]), "dkv_budget_views")
    return tuple(x.value for x in v)


def dkv_memcpy_to_host(ctx: int, host_dst, dev_src: int, nbytes: int, stream=None) -> None:
    _check(load().dkv_memcpy_to_host(ctx, _ptr(host_dst), dev_src, nbytes, _stream(stream)), "dkv_memcpy_to_host")


def read_device_i32(ctx: int, dev_src: int, shape):
    """numpy int32 copy of a device view returned by dkv_layer_views / dkv_budget_views."""
    import numpy as np
    out = np.empty(shape, dtype=np.int32)
    dkv_memcpy_to_host(ctx, out, dev_src, out.nbytes)
    return out


def dkv_last_status(ctx: int):
    buf = (ctypes.c_int32 * 8)()
    code = load().dkv_last_status(ctx, buf)
    return code, list(buf)


def dkv_static_last_status():
    buf = (ctypes.c_int32 * 8)()
    code = load().dkv_static_last_status(buf)
    return code, list(buf)


def dkv_set_wait_limit(ctx: int, clock_ticks: int) -> None:
    _check(load().dkv_set_wait_limit(ctx, clock_ticks), "dkv_set_wait_limit")


def dkv_debug_withhold_tile(ctx: int, sweep: int, tile: int) -> None:
    _check(load().dkv_debug_withhold_tile(ctx, sweep, tile), "dkv_debug_withhold_tile")


STEP_NAMES = ["score_stats", "score_emit", "select", "gather", "rebudget", "shrink", "decode", "other7"]


def dkv_profile(ctx: int, enable: bool) -> None:
    _check(load().dkv_profile(ctx, int(enable)), "dkv_profile")


def dkv_profile_read(ctx: int):
    """{step name: (milliseconds, kernels)} accumulated since the last read."""
    ms = (ctypes.c_double * 8)()
    n = (ctypes.c_int64 * 8)()
    _check(load().dkv_profile_read(ctx, ms, n), "dkv_profile_read")
    return {STEP_NAMES[i]: (ms[i], int(n[i])) for i in range(8)}


def dkv_launch_count(ctx: int) -> int:
    return int(load().dkv_launch_count(ctx))


def dkv_last_cuda_error(ctx: int) -> int:
    return load().dkv_last_cuda_error(ctx)
