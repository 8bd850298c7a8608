"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol,
and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2403_10444_b200 as bv
from paper_2403_10444_b200 import build as bv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    bv_build.build()
    return bv.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:bv|tv|gbv)_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(bv.EXPORTS) == names


def test_version_and_status_strings(lib):
    assert bv.bv_version() >= 100
    assert bv.bv_status_string(0) == "ok"
    assert "invalid" in bv.bv_status_string(-1)
    assert "unknown" in bv.bv_status_string(-99)


def test_bad_arguments_are_rejected_without_a_device(lib):
    buf = (ctypes.c_float * 64)()
    p = ctypes.addressof(buf)
    ok = dict(B=1, gamma=2, V=4, dtype=0, T=1.0)

    def call(fn="bv_verify", tgt=p, drf=p, tok=p, uni=p, ot=p, ol=p, **kw):
        a = dict(ok, **kw)
        return getattr(lib, fn)(tgt, drf, tok, uni, a["B"], a["gamma"], a["V"], a["dtype"],
                                ctypes.c_float(a["T"]), ot, ol, None)

    for fn in ("bv_verify", "tv_verify", "gbv_verify"):
        assert call(fn, tgt=None) == -1
        assert call(fn, ol=None) == -1
        assert call(fn, B=-1) == -1
        assert call(fn, gamma=0) == -1
        assert call(fn, V=0) == -1
        assert call(fn, dtype=7) == -1
        assert call(fn, T=0.0) == -1
        assert call(fn, T=float("nan")) == -1
        assert call(fn, T=float("inf")) == -1
        assert call(fn, tgt=p + 2) == -1          # fp32 logits must be 4-byte aligned
        assert call(fn, gamma=65) == -2           # longer than BV_MAX_GAMMA
        assert call(fn, B=0) == 0                 # empty batch: nothing to do
    assert lib.bv_verify_host(None, p, p, p, 1, 2, 4, 0, ctypes.c_float(1.0), p, p) == -1


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError):
        bv.load_library(str(tmp_path / "nope.so"))


def test_options_are_checked_by_name(lib):
    assert lib.bv_set_option(b"flow_chunks", 0) == 0
    assert lib.bv_set_option(b"no_such_option", 1) == -1
    assert lib.bv_set_option(None, 1) == -1
