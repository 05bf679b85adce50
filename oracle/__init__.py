"""CPU oracle for the SegLinear + DualScale quantized linear layer.

TEST INFRASTRUCTURE ONLY.  This package wraps ``segquant_oracle.c`` (plain C
loops, gcc) with numpy marshalling.  It shares no code with the CUDA library and
must never be imported by it; only the test-suite, the smoke check and the
``cpu_baseline`` / ``--impl reference`` legs of the benchmark may call it.

Every function follows one step of the method, in the paper's order:
calibration (Sec. 4.3.2 scale formula), weight and activation codes (Sec. 3
quantizer, Sec. 4.3.2 Q_dual and the polarity split), per-K-segment
accumulation (Sec. 4.2.2, Sec. 4.3.2), and the dequantizing recombination
(Sec. 4.3.2 last display, App. A symmetric recovery).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "segquant_oracle.c")
_LIB = os.path.join(_HERE, "libsegquant_oracle.so")

INT8_QMAX = 127.0      # positive bound of the int8 range
INT8_QMIN_ABS = 128.0  # magnitude of the negative bound used by the dual quantizer
E4M3_MAX = 448.0


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (building the checker is not using it)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        # SEGQUANT_ORACLE_LIB lets the mutation test load a deliberately broken build of the oracle
        _lib = C.CDLL(os.environ.get("SEGQUANT_ORACLE_LIB") or build())
        _lib.sqo_e4m3_decode.restype = C.c_double
        _lib.sqo_e4m3_decode.argtypes = [C.c_uint8]
        _lib.sqo_e4m3_encode.restype = C.c_uint8
        _lib.sqo_e4m3_encode.argtypes = [C.c_float]
        _lib.sqo_bf16_from_f64.restype = C.c_uint16
        _lib.sqo_bf16_from_f64.argtypes = [C.c_double]
        _lib.sqo_accumulate_i8.restype = C.c_int64
        _lib.sqo_num_threads.restype = C.c_int
        _lib.sqo_silu.restype = C.c_double
        _lib.sqo_silu.argtypes = [C.c_double]
        _lib.sqo_gelu.restype = C.c_double
        _lib.sqo_gelu.argtypes = [C.c_double]
        _lib.sqo_geglu.restype = C.c_double
        _lib.sqo_geglu.argtypes = [C.c_double, C.c_double]
    return _lib


def num_threads() -> int:
    return int(lib().sqo_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


@dataclass
class SegTable:
    """K-partition kb[0..P] and N-partition nb[0..Q] (Sec. 4.2.2)."""
    kb: np.ndarray
    nb: np.ndarray

    def __post_init__(self):
        self.kb = _i32(self.kb)
        self.nb = _i32(self.nb)

    @property
    def P(self):
        return len(self.kb) - 1

    @property
    def Q(self):
        return len(self.nb) - 1


# ------------------------------------------------------------------ step 1

def calib_act(X, kb, dual, q_max=INT8_QMAX, q_min_abs=INT8_QMIN_ABS):
    """Min/max activation scales per K-segment.  Returns (s_pos, s_neg|None)."""
    X = _f32(X)
    kb = _i32(kb)
    P = len(kb) - 1
    s_pos = np.zeros(P, np.float32)
    s_neg = np.zeros(P, np.float32)
    lib().sqo_calib_act(_p(X), C.c_int64(X.shape[0]), C.c_int64(X.shape[1]), C.c_int64(X.shape[1]),
                        C.c_int(P), _p(kb), C.c_int(int(dual)),
                        C.c_float(q_max), C.c_float(q_min_abs), _p(s_pos), _p(s_neg))
    return s_pos, (s_neg if dual else None)


def calib_weight(W, kb, nb, w_max=INT8_QMAX):
    """Abs-max weight scales per (K-segment, N-segment) block, shape [P,Q]."""
    W = _f32(W)
    kb, nb = _i32(kb), _i32(nb)
    P, Q = len(kb) - 1, len(nb) - 1
    s_w = np.zeros((P, Q), np.float32)
    lib().sqo_calib_weight(_p(W), C.c_int64(W.shape[0]), C.c_int64(W.shape[1]), C.c_int64(W.shape[1]),
                           C.c_int(P), _p(kb), C.c_int(Q), _p(nb), C.c_float(w_max), _p(s_w))
    return s_w


# ------------------------------------------------------------- steps 2, 3

def quantize_act(X, kb, s_pos, s_neg=None, code="int8",
                 q_max=INT8_QMAX, q_min_abs=INT8_QMIN_ABS):
    """Activation codes.  Dual (s_neg given): returns (c_pos, c_neg); else (c, None)."""
    X = _f32(X)
    kb = _i32(kb)
    M, K = X.shape
    P = len(kb) - 1
    s_pos = _f32(s_pos)
    s_neg = None if s_neg is None else _f32(s_neg)
    dt = np.int8 if code == "int8" else np.uint8
    c_pos = np.zeros((M, K), dt)
    c_neg = np.zeros((M, K), dt) if s_neg is not None else None
    if code == "int8":
        lib().sqo_quantize_act_i8(_p(X), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_int(P), _p(kb),
                                  _p(s_pos), _p(s_neg), C.c_float(q_max), C.c_float(q_min_abs),
                                  _p(c_pos), _p(c_neg), C.c_int64(K))
    elif code == "e4m3":
        lib().sqo_quantize_act_e4m3(_p(X), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_int(P), _p(kb),
                                    _p(s_pos), _p(s_neg), _p(c_pos), _p(c_neg), C.c_int64(K))
    else:
        raise ValueError(code)
    return c_pos, c_neg


def quantize_weight(W, kb, nb, s_w, code="int8", w_max=INT8_QMAX):
    W = _f32(W)
    kb, nb = _i32(kb), _i32(nb)
    N, K = W.shape
    P, Q = len(kb) - 1, len(nb) - 1
    s_w = _f32(s_w).reshape(P, Q)
    if code == "int8":
        Wq = np.zeros((N, K), np.int8)
        lib().sqo_quantize_weight_i8(_p(W), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(P), _p(kb),
                                     C.c_int(Q), _p(nb), _p(s_w), C.c_float(w_max), _p(Wq), C.c_int64(K))
    elif code == "e4m3":
        Wq = np.zeros((N, K), np.uint8)
        lib().sqo_quantize_weight_e4m3(_p(W), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(P), _p(kb),
                                       C.c_int(Q), _p(nb), _p(s_w), _p(Wq), C.c_int64(K))
    else:
        raise ValueError(code)
    return Wq


# ------------------------------------------------------------------ step 4

def accumulate(Xq, Wq, kb, code="int8"):
    """acc[p,m,n] = sum over K-segment p of Xq[m,k]*Wq[n,k].  int32 (int8 codes) or fp64 (e4m3)."""
    kb = _i32(kb)
    P = len(kb) - 1
    M, K = Xq.shape
    N = Wq.shape[0]
    assert Wq.shape[1] == K
    if code == "int8":
        Xq = np.ascontiguousarray(Xq, np.int8)
        Wq = np.ascontiguousarray(Wq, np.int8)
        acc = np.zeros((P, M, N), np.int32)
        ovf = lib().sqo_accumulate_i8(_p(Xq), C.c_int64(K), _p(Wq), C.c_int64(K), C.c_int64(M),
                                      C.c_int64(N), C.c_int64(K), C.c_int(P), _p(kb), _p(acc))
        if ovf:
            raise OverflowError(f"{ovf} accumulators exceed int32")
    else:
        Xq = np.ascontiguousarray(Xq, np.uint8)
        Wq = np.ascontiguousarray(Wq, np.uint8)
        acc = np.zeros((P, M, N), np.float64)
        lib().sqo_accumulate_e4m3(_p(Xq), C.c_int64(K), _p(Wq), C.c_int64(K), C.c_int64(M),
                                  C.c_int64(N), C.c_int64(K), C.c_int(P), _p(kb), _p(acc))
    return acc


# ------------------------------------------------------------------ step 5

def dequant(acc_pos, acc_neg, nb, s_pos, s_neg, s_w, bias=None, with_abs=False):
    """fp64 recombination  sum_p (s_pos s_w acc_pos + s_neg s_w acc_neg) + bias."""
    nb = _i32(nb)
    P, M, N = acc_pos.shape
    Q = len(nb) - 1
    a_pos = np.ascontiguousarray(acc_pos, np.float64)
    a_neg = None if acc_neg is None else np.ascontiguousarray(acc_neg, np.float64)
    s_pos = _f32(s_pos)
    s_neg = None if s_neg is None else _f32(s_neg)
    s_w = _f32(s_w).reshape(P, Q)
    bias = None if bias is None else _f32(bias)
    y = np.zeros((M, N), np.float64)
    ya = np.zeros((M, N), np.float64) if with_abs else None
    lib().sqo_dequant(_p(a_pos), _p(a_neg), C.c_int64(M), C.c_int64(N), C.c_int(P), C.c_int(Q), _p(nb),
                      _p(s_pos), _p(s_neg), _p(s_w), _p(bias), _p(y), _p(ya))
    return (y, ya) if with_abs else y


def bf16_bits(y64):
    """Round fp64 values to bf16 (nearest-even, directly from fp64); returns uint16 bit patterns."""
    y64 = np.ascontiguousarray(y64, np.float64)
    out = np.zeros(y64.shape, np.uint16)
    lib().sqo_bf16_from_f64_array(_p(y64), C.c_int64(y64.size), _p(out))
    return out


def e4m3_decode(codes):
    lut = np.array([lib().sqo_e4m3_decode(c) for c in range(256)], np.float64)
    return lut[np.asarray(codes, np.uint8)]


def e4m3_encode(values):
    v = _f32(values)
    f = lib().sqo_e4m3_encode
    return np.array([f(float(x)) for x in v.ravel()], np.uint8).reshape(v.shape)


# ------------------------------------------- comparison scheme: zero-point quantization (App. A)

def calib_act_asym(X, kb, q_min=-128.0, q_max=127.0):
    """(s [P] fp32, z [P] int32) per K-segment from strict min/max with the range widened to contain 0."""
    X = _f32(X)
    kb = _i32(kb)
    P = len(kb) - 1
    s = np.zeros(P, np.float32)
    z = np.zeros(P, np.int32)
    lib().sqo_calib_act_asym(_p(X), C.c_int64(X.shape[0]), C.c_int64(X.shape[1]), C.c_int64(X.shape[1]),
                             C.c_int(P), _p(kb), C.c_float(q_min), C.c_float(q_max), _p(s), _p(z))
    return s, z


def quantize_act_asym(X, kb, s, z, q_min=-128.0, q_max=127.0):
    """int8 codes clip(round(x / s[p]) + z[p], q_min, q_max)."""
    X = _f32(X)
    kb = _i32(kb)
    M, K = X.shape
    c = np.zeros((M, K), np.int8)
    lib().sqo_quantize_act_asym_i8(_p(X), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_int(len(kb) - 1), _p(kb),
                                   _p(_f32(s)), _p(_i32(z)), C.c_float(q_min), C.c_float(q_max), _p(c), C.c_int64(K))
    return c


def segment_sums(A, kb):
    """out[p, r] = sum over K-segment p of the int8 codes A[r, k] (exact)."""
    A = np.ascontiguousarray(A, np.int8)
    kb = _i32(kb)
    out = np.zeros((len(kb) - 1, A.shape[0]), np.int64)
    lib().sqo_segment_sums_i8(_p(A), C.c_int64(A.shape[1]), C.c_int64(A.shape[0]), C.c_int(len(kb) - 1), _p(kb), _p(out))
    return out


def dequant_asym(acc, xsum, wsum, kb, nb, s_x, z_x, s_w, z_w=None, bias=None):
    """App. A asymmetric recovery in fp64; returns (y, sum of |terms|)."""
    kb, nb = _i32(kb), _i32(nb)
    P, M, N = acc.shape
    Q = len(nb) - 1
    acc = np.ascontiguousarray(acc, np.float64)
    xsum = np.ascontiguousarray(xsum, np.int64)
    wsum = np.ascontiguousarray(wsum, np.int64)
    y = np.zeros((M, N), np.float64)
    ya = np.zeros((M, N), np.float64)
    zw = None if z_w is None else _i32(np.asarray(z_w).reshape(P, Q))
    b = None if bias is None else _f32(bias)
    lib().sqo_dequant_asym(_p(acc), _p(xsum), _p(wsum), C.c_int64(M), C.c_int64(N), C.c_int(P), _p(kb), C.c_int(Q),
                           _p(nb), _p(_f32(s_x)), _p(_i32(z_x)), _p(_f32(s_w).reshape(P, Q)), _p(zw), _p(b), _p(y), _p(ya))
    return y, ya


def fold_zero_point(wsum, nb, s_x, z_x, s_w, bias=None):
    """bias'[n] = bias[n] - sum_p s_x[p] s_w[p][q(n)] z_x[p] wsum[p][n] in fp64 (symmetric weights)."""
    nb = _i32(nb)
    wsum = np.ascontiguousarray(wsum, np.int64)
    P, N = wsum.shape
    Q = len(nb) - 1
    out = np.zeros(N, np.float64)
    b = None if bias is None else _f32(bias)
    lib().sqo_fold_zero_point(_p(wsum), C.c_int64(N), C.c_int(P), C.c_int(Q), _p(nb), _p(_f32(s_x)), _p(_i32(z_x)),
                              _p(_f32(s_w).reshape(P, Q)), _p(b), _p(out))
    return out


@dataclass
class AsymResult:
    codes: np.ndarray
    acc: np.ndarray
    wsum: np.ndarray
    bias_folded: np.ndarray
    y64: np.ndarray
    y_abs: np.ndarray


def layer_forward_asym(X, Wq, seg: SegTable, s_x, z_x, s_w, bias=None) -> AsymResult:
    """The zero-point scheme for one layer with symmetric weight codes: codes, accumulators, the unfolded
    App. A recovery in fp64 and the folded bias."""
    codes = quantize_act_asym(X, seg.kb, s_x, z_x)
    acc = accumulate(codes, Wq, seg.kb, "int8")
    xsum = segment_sums(codes, seg.kb)
    wsum = segment_sums(Wq, seg.kb)
    y64, y_abs = dequant_asym(acc, xsum, wsum, seg.kb, seg.nb, s_x, z_x, s_w, None, bias)
    return AsymResult(codes, acc, wsum, fold_zero_point(wsum, seg.nb, s_x, z_x, s_w, bias), y64, y_abs)


# ------------------------------------------- act-to-linear segment in front of the quantizer

ACT = {"silu": 1, "gelu": 2}


def activation(H, act: str, stored="bf16"):
    """act(H) evaluated in fp64 and rounded once to the stored dtype; returns (fp32 array, fp64 exact values)."""
    H = _f32(H)
    out = np.zeros(H.shape, np.float32)
    exact = np.zeros(H.shape, np.float64)
    lib().sqo_activation(_p(H), C.c_int64(H.size), C.c_int(ACT[act]), C.c_int(int(stored == "bf16")), _p(out), _p(exact))
    return out, exact


def activation_gated(H, stored="bf16"):
    """GEGLU: H [M, 2K] -> H[:, :K] * GELU(H[:, K:]) in fp64, rounded once to the stored dtype.
    Returns (fp32 array [M, K], fp64 exact values)."""
    H = _f32(H)
    M, K2 = H.shape
    assert K2 % 2 == 0
    K = K2 // 2
    out = np.zeros((M, K), np.float32)
    exact = np.zeros((M, K), np.float64)
    lib().sqo_activation_gated(_p(H), C.c_int64(M), C.c_int64(K), C.c_int64(K2), C.c_int(int(stored == "bf16")), _p(out),
                               C.c_int64(K), _p(exact))
    return out, exact


def smooth(X, mult):
    """fl32(x * mult[k]) per element."""
    X = _f32(X)
    mult = _f32(mult)
    out = np.zeros(X.shape, np.float32)
    lib().sqo_smooth(_p(X), C.c_int64(X.shape[0]), C.c_int64(X.shape[1]), C.c_int64(X.shape[1]), _p(mult), _p(out),
                     C.c_int64(X.shape[1]))
    return out


# ------------------------------------------- W4A8: per-channel 4-bit weights, per-token activation scales

def quantize_per_row(X, kb, dual, q_max=INT8_QMAX, q_min_abs=INT8_QMIN_ABS):
    """One scale per (row, K-segment) from the row's own extrema, and the codes quantized with it.
    Returns (s_pos [M,P], s_neg [M,P] | None, c_pos, c_neg | None)."""
    X = _f32(X)
    kb = _i32(kb)
    M, K = X.shape
    P = len(kb) - 1
    s_pos = np.zeros((M, P), np.float32)
    s_neg = np.zeros((M, P), np.float32) if dual else None
    c_pos = np.zeros((M, K), np.int8)
    c_neg = np.zeros((M, K), np.int8) if dual else None
    lib().sqo_quantize_per_row_i8(_p(X), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_int(P), _p(kb), C.c_int(int(dual)),
                                  C.c_float(q_max), C.c_float(q_min_abs), _p(s_pos), _p(s_neg), _p(c_pos), _p(c_neg),
                                  C.c_int64(K))
    return s_pos, s_neg, c_pos, c_neg


def pack_w4(Wq):
    Wq = np.ascontiguousarray(Wq, np.int8)
    N, K = Wq.shape
    out = np.zeros((N, K // 2), np.uint8)
    lib().sqo_pack_w4(_p(Wq), C.c_int64(N), C.c_int64(K), C.c_int64(K), _p(out), C.c_int64(K // 2))
    return out


def unpack_w4(packed):
    packed = np.ascontiguousarray(packed, np.uint8)
    N, K2 = packed.shape
    out = np.zeros((N, 2 * K2), np.int8)
    lib().sqo_unpack_w4(_p(packed), C.c_int64(N), C.c_int64(2 * K2), C.c_int64(K2), _p(out), C.c_int64(2 * K2))
    return out


def dequant_per_token(acc_pos, acc_neg, s_pos, s_neg, s_w, bias=None):
    """fp64 recombination with per-token activation scales [M,P] and per-channel weight scales [N,P]."""
    P, M, N = acc_pos.shape
    a_pos = np.ascontiguousarray(acc_pos, np.float64)
    a_neg = None if acc_neg is None else np.ascontiguousarray(acc_neg, np.float64)
    y = np.zeros((M, N), np.float64)
    ya = np.zeros((M, N), np.float64)
    b = None if bias is None else _f32(bias)
    lib().sqo_dequant_per_token(_p(a_pos), _p(a_neg), C.c_int64(M), C.c_int64(N), C.c_int(P), _p(_f32(s_pos)),
                                _p(None if s_neg is None else _f32(s_neg)), _p(_f32(s_w)), _p(b), _p(y), _p(ya))
    return y, ya


@dataclass
class W4A8Result:
    s_pos: np.ndarray
    s_neg: np.ndarray | None
    c_pos: np.ndarray
    c_neg: np.ndarray | None
    acc_pos: np.ndarray
    acc_neg: np.ndarray | None
    y64: np.ndarray
    y_abs: np.ndarray


def layer_forward_w4a8(X, Wq, s_w, kb, dual, bias=None) -> W4A8Result:
    """Per-token quantization of X, accumulation against the (unpacked) 4-bit weight codes, recombination."""
    s_pos, s_neg, c_pos, c_neg = quantize_per_row(X, kb, dual)
    acc_pos = accumulate(c_pos, Wq, kb, "int8")
    acc_neg = accumulate(c_neg, Wq, kb, "int8") if dual else None
    y64, y_abs = dequant_per_token(acc_pos, acc_neg, s_pos, s_neg, s_w, bias)
    return W4A8Result(s_pos, s_neg, c_pos, c_neg, acc_pos, acc_neg, y64, y_abs)


# ----------------------------------------------------------- whole layer

@dataclass
class LayerResult:
    c_pos: np.ndarray
    c_neg: np.ndarray | None
    acc_pos: np.ndarray
    acc_neg: np.ndarray | None
    y64: np.ndarray
    y_abs: np.ndarray


def layer_forward(X, Wq, seg: SegTable, s_pos, s_neg, s_w, bias=None, code="int8",
                  q_max=INT8_QMAX, q_min_abs=INT8_QMIN_ABS) -> LayerResult:
    """Steps 3-5 for one layer (weights already quantized)."""
    c_pos, c_neg = quantize_act(X, seg.kb, s_pos, s_neg, code, q_max, q_min_abs)
    acc_pos = accumulate(c_pos, Wq, seg.kb, code)
    acc_neg = accumulate(c_neg, Wq, seg.kb, code) if c_neg is not None else None
    y64, y_abs = dequant(acc_pos, acc_neg, seg.nb, s_pos, s_neg, s_w, bias, with_abs=True)
    return LayerResult(c_pos, c_neg, acc_pos, acc_neg, y64, y_abs)
