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
    assert lib.lookm_compress_layer(*args(mode=4)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(mode=-1)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(lay=_layout(d=64))) == B.ERR_UNSUPPORTED
    assert lib.lookm_compress_layer(*args(q=C.c_void_p(264))) == B.ERR_INVALID_ARG   # 8-byte aligned only
    bad = _layout()
    bad.q_stride_tok = 4100                                                            # not a multiple of 8
    assert lib.lookm_compress_layer(*args(lay=bad)) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*args(wsb=1024)) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.lookm_compress_layer(*args(ws=C.c_void_p(128))) == B.ERR_INVALID_ARG   # workspace alignment
    assert out_len.value == -1
    assert lib.lookm_device_status(None, None) == B.ERR_INVALID_ARG


def test_misaligned_outputs_lists_and_bad_options_are_rejected_on_the_host():
    lib = B.lib()
    lay = _layout()
    out_len = C.c_int(-1)
    fake, odd16, odd4 = C.c_void_p(256), C.c_void_p(264), C.c_void_p(258)
    # outputs are written with 16-byte stores
    base = [fake, fake, fake, fake, 100, 20, 4, 0, C.byref(lay)]
    tail = [C.byref(out_len), fake, 1 << 40, None]
    assert lib.lookm_compress_layer(*base, odd16, fake, *tail) == B.ERR_INVALID_ARG
    assert lib.lookm_compress_layer(*base, fake, odd16, *tail) == B.ERR_INVALID_ARG
    # options: unknown flag bits, a misaligned log-sum-exp, a head stride below the dense one,
    # a missing mask while the text prior is on
    def opt_call(opt, mask=fake):
        return lib.lookm_compress_layer_opt(fake, fake, fake, mask, 100, 20, 4, 0, C.byref(lay),
                                            C.byref(opt), fake, fake, *tail)
    assert opt_call(B.Options(2, None, 0)) == B.ERR_INVALID_ARG
    assert opt_call(B.Options(0, 258, 0)) == B.ERR_INVALID_ARG
    assert opt_call(B.Options(0, None, 20 * 128 - 8)) == B.ERR_INVALID_ARG
    assert opt_call(B.Options(0, None, 20 * 128 + 4)) == B.ERR_INVALID_ARG
    assert opt_call(B.Options(0, None, 0), mask=None) == B.ERR_INVALID_ARG
    cu = (C.c_int * 2)(0, 100)
    one = lambda v: (C.c_int * 1)(v)
    # a varlen call takes no head stride
    assert lib.lookm_compress_varlen_opt(fake, fake, fake, fake, cu, 1, one(20), one(4), one(0), C.byref(lay),
                                         C.byref(B.Options(0, None, 4096)), fake, fake, None, fake, 1 << 40,
                                         None) == B.ERR_INVALID_ARG
    # index and weight lists are read as 32-bit words
    merge = lambda kept=fake, sim=fake, outk=fake, mode=0: lib.lookm_merge(
        fake, fake, kept, fake, fake, sim, cu, 1, one(20), one(mode), C.byref(lay), 0, outk, fake, fake, 1 << 40, None)
    assert merge(kept=odd4) == B.ERR_INVALID_ARG
    assert merge(sim=odd4) == B.ERR_INVALID_ARG
    assert merge(outk=odd16) == B.ERR_INVALID_ARG
    assert merge(sim=None) == B.ERR_INVALID_ARG                       # weights are needed to merge ...
    noalloc = lambda kept=fake, outk=fake: lib.lookm_merge_noalloc(
        fake, fake, kept, fake, fake, fake, cu, 1, one(20), one(0), C.byref(lay), 0, outk, fake, None)
    assert noalloc(kept=odd4) == B.ERR_INVALID_ARG
    assert noalloc(outk=odd16) == B.ERR_INVALID_ARG
    sel = lambda scores=fake, kept=fake: lib.lookm_select(scores, fake, cu, 1, one(20), one(4), 32, kept, fake,
                                                          None, fake, 1 << 40, None)
    assert sel(scores=odd4) == B.ERR_INVALID_ARG
    assert sel(kept=odd4) == B.ERR_INVALID_ARG
    assert out_len.value == -1


def test_decode_step_host_side_argument_errors():
    lib = B.lib()
    lay = B.CacheLayout(32, 8, 128, 128, 4096, 0.0)
    fake = C.c_void_p(256)
    call = lambda **kw: lib.lookm_decode_step(kw.get("q", fake), fake, fake, kw.get("ck", fake), fake,
                                              kw.get("n", 10), C.byref(kw.get("lay", lay)), fake,
                                              kw.get("ws", fake), kw.get("wsb", 1 << 30), None)
    assert call(q=None) == B.ERR_INVALID_ARG
    assert call(n=-1) == B.ERR_INVALID_ARG
    assert call(ck=C.c_void_p(264)) == B.ERR_INVALID_ARG
    assert call(lay=B.CacheLayout(32, 8, 64, 64, 4096, 0.0)) == B.ERR_UNSUPPORTED
    assert call(lay=B.CacheLayout(32, 5, 128, 128, 4096, 0.0)) == B.ERR_INVALID_ARG
    assert call(lay=B.CacheLayout(32, 8, 128, 130, 4096, 0.0)) == B.ERR_INVALID_ARG
    assert call(wsb=16) == B.ERR_WORKSPACE_TOO_SMALL
    assert call(ws=C.c_void_p(8)) == B.ERR_INVALID_ARG
    assert B.lookm_decode_workspace_size(B.CacheLayout(32, 8, 64, 64, 4096, 0.0), [10]) == 0
    n1 = B.lookm_decode_workspace_size(lay, [10])
    assert n1 > 0 and n1 % 256 == 0 and B.lookm_decode_workspace_size(lay, [1 << 20]) == n1


def test_wait_expiry_selftest_argument_errors():
    lib = B.lib()
    fake = C.c_void_p(0x1000)
    assert lib.lookm_selftest_wait_expiry(0, fake, 256, None) == B.ERR_INVALID_ARG
    assert lib.lookm_selftest_wait_expiry(100001, fake, 256, None) == B.ERR_INVALID_ARG
    assert lib.lookm_selftest_wait_expiry(1000, None, 256, None) == B.ERR_INVALID_ARG
    assert lib.lookm_selftest_wait_expiry(1000, C.c_void_p(0x1010), 256, None) == B.ERR_INVALID_ARG
    assert lib.lookm_selftest_wait_expiry(1000, fake, 128, None) == B.ERR_WORKSPACE_TOO_SMALL


def test_the_binding_loads_the_in_tree_library_only():
    here = os.path.join(ROOT, "paper_2406_18139_b200", "liblookm.so")
    assert os.path.samefile(B.LIB_PATH, here)
    B.lib()
    mapped = [l.split()[-1] for l in open("/proc/self/maps") if "liblookm" in l]
    assert mapped and all(os.path.samefile(m, here) for m in mapped)
