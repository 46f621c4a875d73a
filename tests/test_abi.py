"""The C-ABI library: it builds for sm_100a, loads, exports every symbol include/dkv.h declares,
and rejects bad configurations before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2412_14838_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "dkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dkv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 19 and "dkv_score" in names and "dkv_select_topk" in names
    assert "dkv_rebudget" in names and "dkv_compact" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dkv.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_version_and_strerror(lib):
    assert binding.dkv_version() >= 1000
    assert binding.strerror(0) == "ok"
    assert "argument" in binding.strerror(binding.DKV_ERR_INVALID_ARG)


@pytest.mark.parametrize("kw,code", [
    (dict(Hq=7), binding.DKV_ERR_INVALID_ARG),            # Hq not a multiple of Hkv
    (dict(pool=4), binding.DKV_ERR_INVALID_ARG),          # even pooling width
    (dict(S=16), binding.DKV_ERR_INVALID_ARG),            # S must exceed the window
    (dict(Bl=32), binding.DKV_ERR_INVALID_ARG),           # Bl < N
    (dict(m=0), binding.DKV_ERR_INVALID_ARG),
    (dict(D=96), binding.DKV_ERR_UNSUPPORTED),
    (dict(L=500), binding.DKV_ERR_UNSUPPORTED),
    (dict(Bl=100000), binding.DKV_ERR_UNSUPPORTED),
    (dict(ws=128, S=4096), binding.DKV_ERR_UNSUPPORTED),  # ws*G = 512 window rows
    (dict(pool_kind=2), binding.DKV_ERR_UNSUPPORTED),     # 0 = max, 1 = average
    (dict(flags=0x100), binding.DKV_ERR_INVALID_ARG),     # not one of the DKV_F_* bits
])
def test_bad_configs_are_rejected_on_the_host(lib, kw, code):
    base = dict(L=4, Hq=8, Hkv=2, D=64, Bt=1, S=1024, ws=16, pool=5, N=64, Bl=128, m=2)
    base.update(kw)
    cfg = binding.make_config(**base)
    h = ctypes.c_void_p()
    assert lib.dkv_create(ctypes.byref(cfg), ctypes.byref(h)) == code
    assert h.value is None


def test_null_arguments(lib):
    assert lib.dkv_create(None, None) == binding.DKV_ERR_INVALID_ARG
    assert lib.dkv_destroy(None) == binding.DKV_ERR_INVALID_ARG
    assert lib.dkv_score(None, 0, None, None, None, None) == binding.DKV_ERR_INVALID_ARG
    assert lib.dkv_launch_count(None) == -1
