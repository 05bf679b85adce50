"""Thin ctypes binding over libsegquant.so: argument marshalling only.

Function names mirror the C ABI (include/segquant.h).  Tensors are torch CUDA tensors used as
device memory; every step of the path runs inside the library's kernels.  There is no fallback:
if the library is missing or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsegquant.so")

SQ_OK = 0
SQ_CODE = {"int8": 0, "e4m3": 1}
SQ_F32, SQ_BF16 = 0, 1
SQ_FLAG_QMIN_SYM = 1
STATUS_NAMES = {0: "SQ_OK", 1: "SQ_ERR_NULL", 2: "SQ_ERR_SHAPE", 3: "SQ_ERR_SEGTABLE", 4: "SQ_ERR_ALIGN",
                5: "SQ_ERR_UNSUPPORTED", 6: "SQ_ERR_CUDA", 7: "SQ_ERR_TIMEOUT", 8: "SQ_ERR_WORKSPACE"}

EXPORTS = [
    "segquant_workspace_bytes", "segquant_calib_scales", "segquant_calib_scales_static", "segquant_quantize_act", "segquant_quantize_weight",
    "segquant_seglinear_gemm", "segquant_dualscale_gemm", "segquant_layer_scratch_bytes",
    "segquant_layer_forward", "segquant_layer_forward_pipelined", "segquant_last_device_status", "segquant_set_tuning", "segquant_launch_count", "segquant_last_cuda_error",
    "segquant_status_string", "segquant_quantize_act_fused", "segquant_calib_zero_point",
    "segquant_quantize_act_zero_point", "segquant_fold_zero_point", "segquant_plan_layer", "segquant_plan_run",
    "segquant_quantize_per_row", "segquant_pack_w4", "segquant_unpack_w4", "segquant_w4a8_gemm",
    "segquant_split_workspace_bytes", "segquant_set_quantize_tuning",
]


class SegquantError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class _SegTable(C.Structure):
    _fields_ = [("P", C.c_int32), ("kb", C.POINTER(C.c_int32)), ("Q", C.c_int32), ("nb", C.POINTER(C.c_int32))]


_lib = None


def lib():
    """Loads the shared library; raises if it has not been built (no silent fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2507_14811_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.segquant_workspace_bytes.restype = C.c_size_t
        L.segquant_split_workspace_bytes.restype = C.c_size_t
        L.segquant_split_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int]
        L.segquant_layer_scratch_bytes.restype = C.c_size_t
        L.segquant_layer_scratch_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int]
        L.segquant_launch_count.restype = C.c_uint64
        L.segquant_last_cuda_error.restype = C.c_char_p
        L.segquant_status_string.restype = C.c_char_p
        L.segquant_status_string.argtypes = [C.c_int]
        _lib = L
    return _lib


class SegTable:
    """Host-side segment table: kb[0..P], nb[0..Q]."""

    def __init__(self, kb, nb):
        self.kb = np.ascontiguousarray(kb, np.int32)
        self.nb = np.ascontiguousarray(nb, np.int32)
        self._c = _SegTable(len(self.kb) - 1, self.kb.ctypes.data_as(C.POINTER(C.c_int32)),
                            len(self.nb) - 1, self.nb.ctypes.data_as(C.POINTER(C.c_int32)))

    @property
    def P(self):
        return len(self.kb) - 1

    @property
    def Q(self):
        return len(self.nb) - 1

    def ref(self):
        return C.byref(self._c)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SQ_F32
    if t.dtype == torch.bfloat16:
        return SQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status, where):
    if status != SQ_OK:
        if status == 6:
            where = f"{where} ({lib().segquant_last_cuda_error().decode()})"
        raise SegquantError(status, where)


def workspace_bytes() -> int:
    return int(lib().segquant_workspace_bytes())


def segquant_set_quantize_tuning(fused_table_mode: int = 0):
    _check(lib().segquant_set_quantize_tuning(C.c_int(fused_table_mode)), "segquant_set_quantize_tuning")


def split_workspace_bytes(M: int, N: int, dual: bool) -> int:
    """Size of the larger workspace that lets the GEMM calls split tiles for an [M, N] output (current device)."""
    return int(lib().segquant_split_workspace_bytes(C.c_int64(M), C.c_int64(N), C.c_int(int(dual))))


def new_workspace(device="cuda", split_for=None) -> torch.Tensor:
    """Zero-filled, 256-byte aligned device scratch for the calls below.  split_for=(M, N, dual) makes it large
    enough for the GEMM calls to split tiles of such a layer."""
    n = workspace_bytes()
    if split_for is not None:
        with torch.cuda.device(device):
            n = max(n, split_workspace_bytes(*split_for))
    return torch.zeros(n, dtype=torch.uint8, device=device)


def segquant_calib_scales(X: torch.Tensor, seg: SegTable, code: str, is_weight: bool, dual: bool,
                          workspace: torch.Tensor, flags: int = 0):
    """Returns (s_pos, s_neg|None) for activations, (s_w [P*Q], None) for weights."""
    rows, K = X.shape
    n = seg.P * (seg.Q if is_weight else 1)
    s_pos = torch.empty(n, dtype=torch.float32, device=X.device)
    s_neg = torch.empty(n, dtype=torch.float32, device=X.device) if (dual and not is_weight) else None
    st = lib().segquant_calib_scales(_ptr(X), C.c_int(_dt(X)), C.c_int64(rows), C.c_int64(K), C.c_int64(X.stride(0)),
                                     seg.ref(), C.c_int(SQ_CODE[code]), C.c_int(int(is_weight)), C.c_int(int(dual)),
                                     C.c_uint32(flags), _ptr(s_pos), _ptr(s_neg), _ptr(workspace),
                                     C.c_size_t(workspace.numel()), _stream())
    _check(st, "segquant_calib_scales")
    return s_pos, s_neg


def segquant_calib_scales_static(X: torch.Tensor, seg: SegTable, code: str, is_weight: bool, dual: bool,
                                 flags: int = 0, s_pos=None, s_neg=None):
    """segquant_calib_scales without a workspace: for callers that may not allocate device memory, the
    library keeps the reduction partials in a fixed array of its own.  Pass preallocated s_pos / s_neg
    to keep this wrapper allocation-free as well; calls on one GPU must not overlap."""
    rows, K = X.shape
    n = seg.P * (seg.Q if is_weight else 1)
    if s_pos is None:
        s_pos = torch.empty(n, dtype=torch.float32, device=X.device)
    if s_neg is None and dual and not is_weight:
        s_neg = torch.empty(n, dtype=torch.float32, device=X.device)
    st = lib().segquant_calib_scales_static(_ptr(X), C.c_int(_dt(X)), C.c_int64(rows), C.c_int64(K),
                                            C.c_int64(X.stride(0)), seg.ref(), C.c_int(SQ_CODE[code]),
                                            C.c_int(int(is_weight)), C.c_int(int(dual)), C.c_uint32(flags),
                                            _ptr(s_pos), _ptr(s_neg if (dual and not is_weight) else None), _stream())
    _check(st, "segquant_calib_scales_static")
    return s_pos, (s_neg if (dual and not is_weight) else None)


def _ldc(K: int) -> int:
    return (K + 127) // 128 * 128


def new_codes(M: int, K: int, device) -> torch.Tensor:
    """Code matrix [M,K] with a 128-byte padded row pitch (view of a [M, ldc] buffer)."""
    return torch.empty((M, _ldc(K)), dtype=torch.uint8, device=device)[:, :K]


def segquant_quantize_act(X: torch.Tensor, seg: SegTable, s_pos, s_neg, code: str, flags: int = 0,
                          c_pos=None, c_neg=None):
    M, K = X.shape
    if c_pos is None:
        c_pos = new_codes(M, K, X.device)
    if s_neg is not None and c_neg is None:
        c_neg = new_codes(M, K, X.device)
    st = lib().segquant_quantize_act(_ptr(X), C.c_int(_dt(X)), C.c_int64(M), C.c_int64(K), C.c_int64(X.stride(0)),
                                     seg.ref(), _ptr(s_pos), _ptr(s_neg), C.c_int(SQ_CODE[code]), C.c_uint32(flags),
                                     _ptr(c_pos), _ptr(c_neg), C.c_int64(c_pos.stride(0)), _stream())
    _check(st, "segquant_quantize_act")
    return c_pos, (c_neg if s_neg is not None else None)


SQ_ACT = {None: 0, "none": 0, "silu": 1, "gelu": 2, "geglu": 3}


def segquant_quantize_act_fused(H: torch.Tensor, seg: SegTable, s_pos, s_neg, code: str, act=None, mult=None,
                                flags: int = 0, c_pos=None, c_neg=None):
    """Activation function and / or per-channel multiplier in front of the quantizer, in one pass over H.
    act="geglu": H is [M, 2K] (value half, gate half) and the codes are [M, K]."""
    M, K = H.shape
    if act == "geglu":
        K //= 2
    if c_pos is None:
        c_pos = new_codes(M, K, H.device)
    if s_neg is not None and c_neg is None:
        c_neg = new_codes(M, K, H.device)
    st = lib().segquant_quantize_act_fused(_ptr(H), C.c_int(_dt(H)), C.c_int64(M), C.c_int64(K), C.c_int64(H.stride(0)),
                                           seg.ref(), _ptr(s_pos), _ptr(s_neg), C.c_int(SQ_CODE[code]), C.c_uint32(flags),
                                           C.c_int(SQ_ACT[act]), _ptr(mult), _ptr(c_pos), _ptr(c_neg),
                                           C.c_int64(c_pos.stride(0)), _stream())
    _check(st, "segquant_quantize_act_fused")
    return c_pos, (c_neg if s_neg is not None else None)


def segquant_calib_zero_point(X: torch.Tensor, seg: SegTable, workspace: torch.Tensor):
    """(s_x [P] fp32, z_x [P] int32) of the zero-point comparison scheme."""
    rows, K = X.shape
    s_x = torch.empty(seg.P, dtype=torch.float32, device=X.device)
    z_x = torch.empty(seg.P, dtype=torch.int32, device=X.device)
    st = lib().segquant_calib_zero_point(_ptr(X), C.c_int(_dt(X)), C.c_int64(rows), C.c_int64(K), C.c_int64(X.stride(0)),
                                         seg.ref(), _ptr(s_x), _ptr(z_x), _ptr(workspace), C.c_size_t(workspace.numel()),
                                         _stream())
    _check(st, "segquant_calib_zero_point")
    return s_x, z_x


def segquant_quantize_act_zero_point(X: torch.Tensor, seg: SegTable, s_x, z_x, codes=None):
    M, K = X.shape
    if codes is None:
        codes = new_codes(M, K, X.device)
    st = lib().segquant_quantize_act_zero_point(_ptr(X), C.c_int(_dt(X)), C.c_int64(M), C.c_int64(K),
                                                C.c_int64(X.stride(0)), seg.ref(), _ptr(s_x), _ptr(z_x), _ptr(codes),
                                                C.c_int64(codes.stride(0)), _stream())
    _check(st, "segquant_quantize_act_zero_point")
    return codes


def segquant_fold_zero_point(Wq: torch.Tensor, seg: SegTable, s_x, z_x, s_w, bias=None):
    N, K = Wq.shape
    out = torch.empty(N, dtype=torch.float32, device=Wq.device)
    st = lib().segquant_fold_zero_point(_ptr(Wq), C.c_int64(Wq.stride(0)), C.c_int64(N), C.c_int64(K), seg.ref(),
                                        _ptr(s_x), _ptr(z_x), _ptr(s_w), _ptr(bias), _ptr(out), _stream())
    _check(st, "segquant_fold_zero_point")
    return out


def segquant_quantize_weight(W: torch.Tensor, seg: SegTable, s_w, code: str, flags: int = 0, Wq=None):
    N, K = W.shape
    if Wq is None:
        Wq = new_codes(N, K, W.device)
    st = lib().segquant_quantize_weight(_ptr(W), C.c_int(_dt(W)), C.c_int64(N), C.c_int64(K), C.c_int64(W.stride(0)),
                                        seg.ref(), _ptr(s_w), C.c_int(SQ_CODE[code]), C.c_uint32(flags),
                                        _ptr(Wq), C.c_int64(Wq.stride(0)), _stream())
    _check(st, "segquant_quantize_weight")
    return Wq


def _new_y(M, N, y_dtype, device):
    return torch.empty((M, N), dtype=y_dtype, device=device)


def _new_dump(nacc, M, N, code, device):
    return torch.zeros((nacc, M, N), dtype=torch.int32 if code == "int8" else torch.float32, device=device)


def segquant_seglinear_gemm(Xq, Wq, seg: SegTable, code: str, s_x, s_w, bias, workspace,
                            y_dtype=torch.bfloat16, Y=None, dump_acc=False):
    M, K = Xq.shape
    N = Wq.shape[0]
    if Y is None:
        Y = _new_y(M, N, y_dtype, Xq.device)
    dump = _new_dump(seg.P, M, N, code, Xq.device) if dump_acc else None
    st = lib().segquant_seglinear_gemm(_ptr(Xq), C.c_int64(Xq.stride(0)), _ptr(Wq), C.c_int64(Wq.stride(0)),
                                       C.c_int64(M), C.c_int64(N), C.c_int64(K), seg.ref(), C.c_int(SQ_CODE[code]),
                                       _ptr(s_x), _ptr(s_w), _ptr(bias), _ptr(Y), C.c_int(_dt(Y)),
                                       C.c_int64(Y.stride(0)), _ptr(dump), _ptr(workspace),
                                       C.c_size_t(workspace.numel()), _stream())
    _check(st, "segquant_seglinear_gemm")
    return (Y, dump) if dump_acc else Y


def segquant_dualscale_gemm(Xq_pos, Xq_neg, Wq, seg: SegTable, code: str, s_pos, s_neg, s_w, bias, workspace,
                            y_dtype=torch.bfloat16, Y=None, dump_acc=False):
    M, K = Xq_pos.shape
    N = Wq.shape[0]
    assert Xq_neg.stride(0) == Xq_pos.stride(0)
    if Y is None:
        Y = _new_y(M, N, y_dtype, Xq_pos.device)
    dump = _new_dump(seg.P * 2, M, N, code, Xq_pos.device) if dump_acc else None
    st = lib().segquant_dualscale_gemm(_ptr(Xq_pos), _ptr(Xq_neg), C.c_int64(Xq_pos.stride(0)), _ptr(Wq),
                                       C.c_int64(Wq.stride(0)), C.c_int64(M), C.c_int64(N), C.c_int64(K), seg.ref(),
                                       C.c_int(SQ_CODE[code]), _ptr(s_pos), _ptr(s_neg), _ptr(s_w), _ptr(bias),
                                       _ptr(Y), C.c_int(_dt(Y)), C.c_int64(Y.stride(0)), _ptr(dump), _ptr(workspace),
                                       C.c_size_t(workspace.numel()), _stream())
    _check(st, "segquant_dualscale_gemm")
    return (Y, dump) if dump_acc else Y


def layer_scratch_bytes(M: int, K: int, dual: bool) -> int:
    return int(lib().segquant_layer_scratch_bytes(M, K, int(dual)))


def segquant_layer_forward(X, Wq, seg: SegTable, code: str, s_pos, s_neg, s_w, bias, Y, scratch, workspace,
                           x_stage=None, y_stage=None, flags: int = 0):
    """Quantize -> GEMM -> epilogue in one call.  X / Y may be (pinned) host tensors, in which case
    x_stage / y_stage are device buffers of the same shape and the copies are part of the call."""
    M, K = X.shape
    N = Wq.shape[0]
    x_host, y_host = not X.is_cuda, not Y.is_cuda
    st = lib().segquant_layer_forward(
        _ptr(X), C.c_int(int(x_host)), _ptr(x_stage), C.c_int(_dt(X)), C.c_int64(M), C.c_int64(K),
        C.c_int64(X.stride(0)), _ptr(Wq), C.c_int64(Wq.stride(0)), C.c_int64(N), seg.ref(), C.c_int(SQ_CODE[code]),
        _ptr(s_pos), _ptr(s_neg), _ptr(s_w), _ptr(bias), C.c_uint32(flags), _ptr(Y), C.c_int(int(y_host)),
        _ptr(y_stage), C.c_int(_dt(Y)), C.c_int64(Y.stride(0)), _ptr(scratch), C.c_size_t(scratch.numel()),
        _ptr(workspace), C.c_size_t(workspace.numel()), _stream())
    _check(st, "segquant_layer_forward")
    return Y


def segquant_layer_forward_pipelined(X, Wq, seg: SegTable, code: str, s_pos, s_neg, s_w, bias, Y, scratch, workspace,
                                     x_stage, y_stage, chunks: int, stream_in, stream_out, flags: int = 0):
    """segquant_layer_forward for pinned host X / Y with the copies overlapped with the kernels: chunks of rows
    go in on stream_in, through the kernels on the current stream, and out on stream_out (torch streams)."""
    M, K = X.shape
    N = Wq.shape[0]
    st = lib().segquant_layer_forward_pipelined(
        _ptr(X), _ptr(x_stage), C.c_int(_dt(X)), C.c_int64(M), C.c_int64(K), C.c_int64(X.stride(0)), _ptr(Wq),
        C.c_int64(Wq.stride(0)), C.c_int64(N), seg.ref(), C.c_int(SQ_CODE[code]), _ptr(s_pos), _ptr(s_neg), _ptr(s_w),
        _ptr(bias), C.c_uint32(flags), _ptr(Y), _ptr(y_stage), C.c_int(_dt(Y)), C.c_int64(Y.stride(0)), _ptr(scratch),
        C.c_size_t(scratch.numel()), _ptr(workspace), C.c_size_t(workspace.numel()), C.c_int(chunks), _stream(),
        C.c_void_p(stream_in.cuda_stream), C.c_void_p(stream_out.cuda_stream))
    _check(st, "segquant_layer_forward_pipelined")
    return Y


def segquant_quantize_per_row(X: torch.Tensor, seg: SegTable, dual: bool, bits: int = 8, flags: int = 0):
    """Per-row scales [rows, P] (per token, or per output channel for bits = 4) and the int8 codes made with them."""
    rows, K = X.shape
    s_pos = torch.empty((rows, seg.P), dtype=torch.float32, device=X.device)
    s_neg = torch.empty((rows, seg.P), dtype=torch.float32, device=X.device) if dual else None
    c_pos = new_codes(rows, K, X.device)
    c_neg = new_codes(rows, K, X.device) if dual else None
    st = lib().segquant_quantize_per_row(_ptr(X), C.c_int(_dt(X)), C.c_int64(rows), C.c_int64(K), C.c_int64(X.stride(0)),
                                         seg.ref(), C.c_int(bits), C.c_uint32(flags), _ptr(s_pos), _ptr(s_neg), _ptr(c_pos),
                                         _ptr(c_neg), C.c_int64(c_pos.stride(0)), _stream())
    _check(st, "segquant_quantize_per_row")
    return s_pos, s_neg, c_pos, c_neg


def segquant_pack_w4(Wq8: torch.Tensor):
    N, K = Wq8.shape
    out = torch.empty((N, K // 2), dtype=torch.uint8, device=Wq8.device)
    st = lib().segquant_pack_w4(_ptr(Wq8), C.c_int64(Wq8.stride(0)), C.c_int64(N), C.c_int64(K), _ptr(out),
                                C.c_int64(out.stride(0)), _stream())
    _check(st, "segquant_pack_w4")
    return out


def segquant_unpack_w4(Wq4: torch.Tensor, out=None):
    N, K2 = Wq4.shape
    if out is None:
        out = new_codes(N, 2 * K2, Wq4.device)
    st = lib().segquant_unpack_w4(_ptr(Wq4), C.c_int64(Wq4.stride(0)), C.c_int64(N), C.c_int64(2 * K2), _ptr(out),
                                  C.c_int64(out.stride(0)), _stream())
    _check(st, "segquant_unpack_w4")
    return out


def segquant_w4a8_gemm(Xq_pos, Xq_neg, Wq8, seg: SegTable, s_pos, s_neg, s_w, bias, workspace,
                       y_dtype=torch.bfloat16, Y=None, dump_acc=False):
    M, K = Xq_pos.shape
    N = Wq8.shape[0]
    dual = Xq_neg is not None
    if Y is None:
        Y = _new_y(M, N, y_dtype, Xq_pos.device)
    dump = _new_dump(seg.P * (2 if dual else 1), M, N, "int8", Xq_pos.device) if dump_acc else None
    st = lib().segquant_w4a8_gemm(_ptr(Xq_pos), _ptr(Xq_neg), C.c_int64(Xq_pos.stride(0)), _ptr(Wq8),
                                  C.c_int64(Wq8.stride(0)), C.c_int64(M), C.c_int64(N), C.c_int64(K), seg.ref(),
                                  _ptr(s_pos), _ptr(s_neg), _ptr(s_w), _ptr(bias), _ptr(Y), C.c_int(_dt(Y)),
                                  C.c_int64(Y.stride(0)), _ptr(dump), _ptr(workspace), C.c_size_t(workspace.numel()),
                                  _stream())
    _check(st, "segquant_w4a8_gemm")
    return (Y, dump) if dump_acc else Y


SQ_PLAN_BYTES = 4096


class LayerPlan:
    """A prepared layer call (segquant_plan_layer): holds the plan's storage and the tensors it refers to."""

    def __init__(self, X, Wq, seg: SegTable, code, s_pos, s_neg, s_w, bias, Y, scratch, workspace, flags: int = 0):
        M, K = X.shape
        N = Wq.shape[0]
        self._keep = (X, Wq, seg, s_pos, s_neg, s_w, bias, Y, scratch, workspace)
        self._buf = (C.c_uint64 * (SQ_PLAN_BYTES // 8))()
        st = lib().segquant_plan_layer(
            C.byref(self._buf), _ptr(X), C.c_int(_dt(X)), C.c_int64(M), C.c_int64(K), C.c_int64(X.stride(0)), _ptr(Wq),
            C.c_int64(Wq.stride(0)), C.c_int64(N), seg.ref(), C.c_int(SQ_CODE[code]), _ptr(s_pos), _ptr(s_neg), _ptr(s_w),
            _ptr(bias), C.c_uint32(flags), _ptr(Y), C.c_int(_dt(Y)), C.c_int64(Y.stride(0)), _ptr(scratch),
            C.c_size_t(scratch.numel()), _ptr(workspace), C.c_size_t(workspace.numel()))
        _check(st, "segquant_plan_layer")
        self._run = lib().segquant_plan_run
        self._ref = C.byref(self._buf)

    def run(self):
        st = self._run(self._ref, _stream())
        if st != SQ_OK:
            _check(st, "segquant_plan_run")


def segquant_last_device_status(workspace) -> tuple[int, int]:
    detail = C.c_uint32(0)
    st = lib().segquant_last_device_status(_ptr(workspace), _stream(), C.byref(detail))
    return int(st), int(detail.value)


def check_device_status(workspace):
    st, detail = segquant_last_device_status(workspace)
    if st != SQ_OK:
        raise SegquantError(st, f"device status (detail 0x{detail:x})")


def segquant_set_tuning(tile_n: int = 0, stages: int = 0, cta_group: int = 0, segment_mode: int = 0):
    _check(lib().segquant_set_tuning(C.c_int(tile_n), C.c_int(stages), C.c_int(cta_group), C.c_int(segment_mode)),
           "segquant_set_tuning")


def segquant_launch_count() -> int:
    return int(lib().segquant_launch_count())
