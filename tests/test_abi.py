"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on
the host before any launch (no GPU needed: none of these calls reaches a kernel)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2507_14811_b200 import binding as B
from paper_2507_14811_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "segquant.h")


@pytest.fixture(scope="module")
def L():
    build_mod.build()
    return B.lib()


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(segquant_\w+)\s*\(", src)))


def test_header_symbols_are_exported(L):
    names = declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in segquant.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_constants(L):
    assert B.workspace_bytes() >= 256 and B.workspace_bytes() % 256 == 0
    assert L.segquant_status_string(0) == b"ok"
    assert B.layer_scratch_bytes(100, 200, True) == 2 * ((100 * 256 + 255) // 256 * 256)
    assert B.layer_scratch_bytes(0, 200, True) == 0


FAKE = 0x10000   # a non-null, 256-byte aligned address that is never dereferenced on these paths


def _seg(kb, nb):
    return B.SegTable(kb, nb)


def gemm(L, M=128, N=64, K=128, kb=(0, 128), nb=(0, 64), ldx=128, ldw=128, ldy=64, code=0, xq=FAKE, wq=FAKE,
         y=FAKE, ws=FAKE, ws_bytes=None, dual=False, s=FAKE):
    seg = _seg(list(kb), list(nb))
    ws_bytes = B.workspace_bytes() if ws_bytes is None else ws_bytes
    if dual:
        return L.segquant_dualscale_gemm(C.c_void_p(xq), C.c_void_p(xq), C.c_int64(ldx), C.c_void_p(wq), C.c_int64(ldw),
                                         C.c_int64(M), C.c_int64(N), C.c_int64(K), seg.ref(), C.c_int(code),
                                         C.c_void_p(s), C.c_void_p(s), C.c_void_p(s), None, C.c_void_p(y), C.c_int(1),
                                         C.c_int64(ldy), None, C.c_void_p(ws), C.c_size_t(ws_bytes), None)
    return L.segquant_seglinear_gemm(C.c_void_p(xq), C.c_int64(ldx), C.c_void_p(wq), C.c_int64(ldw), C.c_int64(M),
                                     C.c_int64(N), C.c_int64(K), seg.ref(), C.c_int(code), C.c_void_p(s),
                                     C.c_void_p(s), None, C.c_void_p(y), C.c_int(1), C.c_int64(ldy), None,
                                     C.c_void_p(ws), C.c_size_t(ws_bytes), None)


def test_gemm_argument_validation(L):
    assert gemm(L, xq=0) == 1                                   # null
    assert gemm(L, s=0) == 1
    assert gemm(L, M=0) == 2                                    # shape
    assert gemm(L, ldx=64) == 2                                 # ld < K
    assert gemm(L, K=262144, kb=(0, 262144), ldx=262144, ldw=262144) == 2   # int32 accumulation bound
    assert gemm(L, kb=(0, 64, 64, 128)) == 3                    # not strictly ascending
    assert gemm(L, kb=(0, 64)) == 3                             # does not end at K
    assert gemm(L, nb=(8, 64)) == 3                             # does not start at 0
    assert gemm(L, xq=FAKE + 4) == 4                            # pointer alignment
    assert gemm(L, ldx=136) == 4                                # pitch not a multiple of 16 bytes
    assert gemm(L, kb=(0, 48, 128)) == 4                        # interior K bound not a multiple of 32
    assert gemm(L, K=136, kb=(0, 136), ldx=144, ldw=144) == 4   # K not a multiple of 16
    assert gemm(L, N=68, nb=(0, 68), ldy=72) == 4               # N not a multiple of 8
    assert gemm(L, code=7) == 5                                 # unknown code
    kb65 = tuple(range(0, 65 * 32 + 1, 32))
    assert gemm(L, K=65 * 32, kb=kb65, ldx=65 * 32, ldw=65 * 32) == 5      # more K-segments than SQ_MAX_P
    kb40 = tuple(range(0, 40 * 32 + 1, 32))
    nb64 = tuple(range(0, 64 * 8 + 1, 8))
    assert gemm(L, N=512, K=40 * 32, kb=kb40, nb=nb64, ldx=40 * 32, ldw=40 * 32, ldy=512) == 5   # 2560 factors > 2048
    assert gemm(L, ws=0) == 8                                   # workspace
    assert gemm(L, ws_bytes=8) == 8
    assert gemm(L, ws=FAKE + 16) == 4


def test_quantize_and_calib_argument_validation(L):
    seg = _seg([0, 128], [0, 64])
    q = lambda **kw: L.segquant_quantize_act(
        C.c_void_p(kw.get("x", FAKE)), C.c_int(kw.get("dt", 1)), C.c_int64(kw.get("M", 4)), C.c_int64(128),
        C.c_int64(kw.get("ld", 128)), kw.get("seg", seg).ref(), C.c_void_p(kw.get("s", FAKE)), None,
        C.c_int(kw.get("code", 0)), C.c_uint32(0), C.c_void_p(kw.get("c", FAKE)), None, C.c_int64(kw.get("ldc", 128)), None)
    assert q(x=0) == 1 and q(s=0) == 1 and q(c=0) == 1
    assert q(M=-1) == 2 and q(ld=100) == 2
    assert q(dt=9) == 5 and q(code=3) == 5
    assert q(ld=132) == 4                                      # 132 bf16 = 264 bytes: not a 16-byte multiple
    assert q(ldc=136) == 4
    assert q(seg=_seg([0, 100], [0, 64])) == 3
    cal = lambda **kw: L.segquant_calib_scales(
        C.c_void_p(kw.get("x", FAKE)), C.c_int(1), C.c_int64(8), C.c_int64(128), C.c_int64(128), seg.ref(), C.c_int(0),
        C.c_int(0), C.c_int(1), C.c_uint32(0), C.c_void_p(kw.get("sp", FAKE)), C.c_void_p(kw.get("sn", FAKE)),
        C.c_void_p(kw.get("ws", FAKE)), C.c_size_t(kw.get("wsb", B.workspace_bytes())), None)
    assert cal(x=0) == 1 and cal(sp=0) == 1 and cal(sn=0) == 1
    assert cal(ws=0) == 8 and cal(wsb=1) == 8


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        B.lib()


def test_plan_calls_reject_on_the_host(L):
    plan = (C.c_uint64 * (B.SQ_PLAN_BYTES // 8))()
    # a plan that was never built (all zero) does not run
    assert L.segquant_plan_run(C.byref(plan), None) == 5
    assert L.segquant_plan_run(None, None) == 1
    seg = _seg([0, 128], [0, 64])

    def plan_layer(x=FAKE, y=FAKE, scratch=FAKE, scratch_bytes=1 << 20, K=128, ld=128, kb=(0, 128), s=FAKE, dt=1, code=0):
        sg = _seg(list(kb), [0, 64])
        return L.segquant_plan_layer(C.byref(plan), C.c_void_p(x), C.c_int(dt), C.c_int64(128), C.c_int64(K), C.c_int64(ld),
                                     C.c_void_p(FAKE), C.c_int64(128), C.c_int64(64), sg.ref(), C.c_int(code), C.c_void_p(s),
                                     None, C.c_void_p(FAKE), None, C.c_uint32(0), C.c_void_p(y), C.c_int(1), C.c_int64(64),
                                     C.c_void_p(scratch), C.c_size_t(scratch_bytes), C.c_void_p(FAKE),
                                     C.c_size_t(B.workspace_bytes()))
    assert plan_layer(x=0) == 1 and plan_layer(y=0) == 1 and plan_layer(scratch=0) == 1 and plan_layer(s=0) == 1
    assert plan_layer(dt=7) == 5 and plan_layer(code=9) == 5
    assert plan_layer(ld=64) == 2                                 # pitch below K
    assert plan_layer(scratch_bytes=100) == 8                     # code matrices do not fit
    assert plan_layer(scratch=FAKE + 16) == 4
    assert plan_layer(kb=(0, 40, 128)) == 4                       # interior K-bound not a multiple of 32
    assert plan_layer(kb=(0, 64, 32, 128)) == 3
    # a failed build leaves a plan that does not run
    assert L.segquant_plan_run(C.byref(plan), None) == 5
    assert seg.P == 1 and B.SQ_PLAN_BYTES == 4096
