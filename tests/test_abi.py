"""The C-ABI library loads, exports every symbol include/wcc.h declares, and rejects bad arguments on the host
(before any launch, so these run without a GPU)."""
import ctypes as C
import os
import re

import pytest

from paper_2205_12268_b200 import build as wbuild
from paper_2205_12268_b200 import wcc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    wbuild.build()
    return wcc.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "wcc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wcc_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert set(wcc.EXPORTS) <= set(names)
    raw = C.CDLL(wcc.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_status_strings(L):
    assert L.wcc_status_str(0) == b"ok"
    assert b"workspace" in L.wcc_status_str(7)


def test_kpad(L):
    assert L.wcc_kpad(24, 8) == 32 and L.wcc_kpad(144, 8) == 160 and L.wcc_kpad(192, 8) == 192
    assert L.wcc_kpad(24, 0) == 32 and L.wcc_kpad(144, 0) == 144 and L.wcc_kpad(20, 0) == 32


def test_workspace_query(L):
    n = L.wcc_workspace_bytes(1, 32, 32, 64, 64, 2, 1024, 8, 0)
    assert n >= 3 * 4096 * 4                # norms, per-position max, rank map
    assert n % 256 == 0
    m = L.wcc_staged_workspace_bytes(1, 32, 32, 64, 64, 2, 1024, 8, 0)
    assert m > 1 * 32 * 4096 * 4 and m > n  # also holds the coefficient map
    assert L.wcc_staged_workspace_bytes(1, 32, 32, 60, 64, 3, 10, 8, 0) == 0
    assert L.wcc_workspace_bytes(1, 32, 32, 64, 64, 2, 1024, 8, 0) == n
    # invalid arguments give 0
    assert L.wcc_workspace_bytes(1, 32, 32, 60, 64, 3, 10, 8, 0) == 0     # 60 % 8 != 0
    assert L.wcc_workspace_bytes(1, 32, 32, 64, 64, 2, 0, 8, 0) == 0
    assert L.wcc_workspace_bytes(1, 32, 32, 64, 64, 2, 10, 1, 0) == 0
    assert L.wcc_workspace_bytes(1, 8193, 32, 64, 64, 2, 10, 8, 0) == 0
    # channel counts beyond one operand tile run stage by stage: the size query accounts for the larger scratch
    big = L.wcc_workspace_bytes(1, 256, 256, 16, 32, 3, 10, 0, 0)
    assert big == L.wcc_staged_workspace_bytes(1, 256, 256, 16, 32, 3, 10, 0, 0) and big > 0
    assert L.wcc_workspace_bytes(1, 1024, 512, 16, 32, 3, 10, 8, 0) == L.wcc_staged_workspace_bytes(1, 1024, 512, 16, 32, 3, 10, 8, 0)
    assert 0 < L.wcc_workspace_bytes(1, 256, 256, 16, 32, 3, 10, 8, 0) < L.wcc_staged_workspace_bytes(1, 256, 256, 16, 32, 3, 10, 8, 0)
    assert L.wcc_select_workspace_bytes(2, 1000) > 0 and L.wcc_select_workspace_bytes(0, 10) == 0


def test_host_side_argument_errors(L):
    a = 4096                                   # fake, aligned, never dereferenced: errors come first
    assert L.wcc_haar_fwd(None, 1, 1, 8, 8, 1, 0, a, a, None) == 1
    assert L.wcc_haar_fwd(a, 1, 1, 12, 8, 3, 0, a, a, None) == 2
    assert L.wcc_haar_fwd(a, 1, 1, 8, 8, 4, 0, a, a, None) == 2
    assert L.wcc_haar_fwd(a, 1, 1, 8, 8, 1, 7, a, a, None) == 5
    assert L.wcc_haar_fwd(a + 4, 1, 1, 8, 8, 1, 0, a, a, None) == 6
    assert L.wcc_haar_inv(a, 1, 0, 8, 8, 1, 0, a, None) == 2
    assert L.wcc_select_topk(a, 1, 64, 0, a, a, a, 1 << 20, None) == 3
    assert L.wcc_select_topk(a, 1, 64, 65, a, a, a, 1 << 20, None) == 3
    assert L.wcc_select_topk(a, 1, 64, 8, a, a, a, 16, None) == 7
    fwd = lambda **kw: L.wcc_forward(*[kw.get(k, d) for k, d in (
        ("x", a), ("Wt", a), ("N", 1), ("Cin", 8), ("Cout", 8), ("H", 16), ("W", 16), ("levels", 2), ("k", 64),
        ("bits", 8), ("y", a), ("dt", 0), ("ws", a), ("ws_bytes", 1 << 30), ("stream", None))])
    assert fwd(x=None) == 1
    assert fwd(H=18) == 2
    assert fwd(k=257) == 3
    assert fwd(bits=9) == 4 and fwd(bits=1) == 4
    assert fwd(dt=3) == 5
    assert fwd(y=a + 8) == 6
    assert fwd(ws_bytes=1024) == 7
    assert fwd(Cout=8193) == 2
    assert fwd(Cin=1024, Cout=512, ws_bytes=1 << 16) == 7  # large channel counts need the stage-by-stage scratch
