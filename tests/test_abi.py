"""The C-ABI library loads, exports every symbol include/choco.h declares, and rejects bad
arguments on the host before touching a device (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_1907_09356_b200 as choco
from paper_1907_09356_b200 import build as choco_build
import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    choco_build.build()
    return choco.load()


def test_exports_match_header(lib):
    with open(os.path.join(ROOT, "include", "choco.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(choco_[a-z_]+)\s*\(", text)))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in choco.h but not exported"
    assert sorted(choco.EXPORTS) == declared


def _init(lib, w, n, d, ld, kind, k=0, s=16, bucket=0):
    p = choco.choco_params(kind, s, bucket, 1, k)
    ctx = ctypes.c_void_p()
    rc = lib.choco_init(ctypes.byref(ctx), n, d, ld, w.row_ptr.ctypes.data, w.col.ctypes.data,
                        w.val.ctypes.data, ctypes.byref(p), 0)
    assert ctx.value is None or rc == 0
    return rc


def test_argument_checks(lib):
    w = workloads.ring(4)
    assert _init(lib, w, 4, 100, 99, choco.Q_SIGN) == -1            # ld < d
    assert _init(lib, w, 0, 100, 100, choco.Q_SIGN) == -1
    assert _init(lib, w, 4, 100, 100, choco.Q_TOPK, k=0) == -1
    assert _init(lib, w, 4, 100, 100, choco.Q_TOPK, k=101) == -1
    assert _init(lib, w, 4, 100, 100, choco.Q_QSGD, s=12) == -1     # not a power of two
    assert _init(lib, w, 4, 100, 100, choco.Q_QSGD, s=16, bucket=96) == -6
    assert _init(lib, w, 4, 100, 100, 9) == -1
    assert _init(lib, w, 4, 1 << 31, 1 << 31, choco.Q_SIGN) == -7
    assert lib.choco_init(None, 4, 100, 100, None, None, None, None, 0) == -1


def test_mixing_matrix_checks(lib):
    good = workloads.ring(5)

    def variant(**kw):
        return workloads.MixingCSR(5, kw.get("rp", good.row_ptr.copy()), kw.get("col", good.col.copy()),
                                   kw.get("val", good.val.copy()))

    v = good.val.copy(); v[0] = 0.5                                  # row sum != 1
    assert _init(lib, variant(val=v), 5, 10, 10, choco.Q_SIGN) == -2
    v = good.val.copy(); v[1] = -v[1]                                # negative weight
    assert _init(lib, variant(val=v), 5, 10, 10, choco.Q_SIGN) == -2
    c = good.col.copy(); c[0], c[1] = c[1], c[0]                     # columns not ascending
    assert _init(lib, variant(col=c), 5, 10, 10, choco.Q_SIGN) == -2
    c = good.col.copy(); c[2] = 7                                    # column out of range
    assert _init(lib, variant(col=c), 5, 10, 10, choco.Q_SIGN) == -2
    # asymmetric: row 0 reaches node 2 instead of node 1, node 2 does not reach back
    c = good.col.copy()
    assert list(c[:3]) == [0, 1, 4]
    c[1] = 2
    assert _init(lib, variant(col=c), 5, 10, 10, choco.Q_SIGN) == -2
    # diagonal missing
    w3 = workloads.MixingCSR(2, np.array([0, 1, 2], np.int32), np.array([1, 0], np.int32),
                             np.array([1.0, 1.0], np.float32))
    assert _init(lib, w3, 2, 10, 10, choco.Q_SIGN) == -2


def test_strerror(lib):
    assert lib.choco_strerror(0) == b"ok"
    for code in range(-8, 0):
        assert lib.choco_strerror(code) not in (b"ok", b"unknown error")
    assert lib.choco_strerror(-99) == b"unknown error"


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(choco, "_lib", None)
    monkeypatch.setattr(choco, "LIB_PATH", "/nonexistent/libchoco.so")
    with pytest.raises(choco.ChocoError):
        choco.load()
