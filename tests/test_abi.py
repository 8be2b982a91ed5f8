"""The C-ABI library loads on a machine without a GPU, exports every declared symbol and rejects
bad arguments on the host before touching the device."""
import ctypes as C
import os
import re

from paper_2406_18139_b200 import binding as B, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _layout(hq=32, hkv=32, d=128):
    return B.Layout(hq, hkv, d, hq * d, d, hkv * d, d, 0.0)


def test_library_builds_loads_and_exports_every_declared_symbol():
    build.build()
    lib = B.lib()
    header = open(os.path.join(ROOT, "include", "lookm.h")).read()
    declared = set(re.findall(r"\b(lookm_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror_and_workspace_size():
    assert B.lookm_strerror(B.OK) == "ok"
    assert "workspace" in B.lookm_strerror(B.ERR_WORKSPACE_TOO_SMALL)
    n1 = B.lookm_workspace_size(_layout(), [8192])
    n2 = B.lookm_workspace_size(_layout(), [8192, 8192])
    assert 0 < n1 < n2 < 4 * n1
    assert n1 % 256 == 0
    assert B.lookm_workspace_size(_layout(), [8192], [1638]) == n1      # budgets do not change it
    assert B.lookm_workspace_size(_layout(d=64), [8192]) == 0           # unsupported head_dim
    assert B.lookm_workspace_size(_layout(hq=30, hkv=4), [8192]) == 0   # heads not divisible
    assert B.lookm_workspace_size(_layout(), [0]) == 0
    assert B.lookm_workspace_size(_layout(), [100], [0]) == 0


def test_host_side_argument_errors_need_no_device():
    lib = B.lib()
    lay = _layout()
    out_len = C.c_int(-1)
    fake = C.c_void_p(256)          # never dereferenced: the call must fail before any launch
    args = lambda **kw: [kw.get("q", fake), fake, fake, fake, kw.get("L", 100), kw.get("B", 20),
                         kw.get("M", 4), kw.get("mode", 0), C.byref(kw.get("lay", lay)), fake, fake,
                         C.byref(out_len), kw.get("ws", fake), kw.get("wsb", 1 << 40), None]
    assert lib.lookm_compress_layer(*args(q=None)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(L=0)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(B=0)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(M=-1)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(mode=3)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(lay=_layout(d=64))) == B.ERR_UNSUPPORTED
    assert lib.lookm_compress_layer(*args(q=C.c_void_p(264))) == B.ERR_INVALID_ARG   # 8-byte aligned only
    bad = _layout()
    bad.q_stride_tok = 4100                                                            # not a multiple of 8
    assert lib.lookm_compress_layer(*args(lay=bad)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(wsb=1024)) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.lookm_compress_layer(*args(ws=C.c_void_p(128))) == B.ERR_INVALID_ARG   # workspace alignment
    assert out_len.value == -1
    assert lib.lookm_device_status(None, None) == B.ERR_INVALID_ARG
