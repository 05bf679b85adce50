"""Comparison helpers for the GPU-vs-oracle parity tests (test code; uses the oracle)."""
from __future__ import annotations

import numpy as np
import torch

import oracle as O

QRANGE = {"int8": (127.0, 128.0), "e4m3": (448.0, 448.0)}


def to_f32_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def oracle_scales(data, flags_qmin_sym=False):
    """Calibration + weight quantization by the oracle for a workloads.LayerData."""
    sp = data.spec
    qmax, qmin_abs = QRANGE[sp.code]
    if flags_qmin_sym and sp.code == "int8":
        qmin_abs = 127.0
    s_pos, s_neg = O.calib_act(to_f32_np(data.X_cal), sp.kb, sp.dual, q_max=qmax, q_min_abs=qmin_abs)
    s_w = O.calib_weight(to_f32_np(data.W), sp.kb, sp.nb, w_max=qmax)
    Wq = O.quantize_weight(to_f32_np(data.W), sp.kb, sp.nb, s_w, code=sp.code, w_max=qmax)
    return s_pos, s_neg, s_w, Wq, (qmax, qmin_abs)


def fp32_epilogue_tolerance(y64, y_abs, nacc):
    """The 1e-5 relative bound required of the fp32 epilogue, plus the rounding the fp32 evaluation
    itself can commit on cancelling terms: each of the nacc products carries the rounding of the
    scale product, of the int->float conversion and of one FMA, and the bias add rounds once more,
    all relative to the sum of |terms| (2^-24 each)."""
    return 1e-5 * np.abs(y64) + (3 * nacc + 1) * 2.0 ** -24 * y_abs


def bf16_ordered(bits_u16: np.ndarray) -> np.ndarray:
    b = bits_u16.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def bf16_value(bits_u16: np.ndarray) -> np.ndarray:
    return (bits_u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def check_bf16_output(y_gpu_bf16: torch.Tensor, y64, y_abs, nacc, extra=0.0):
    """bf16 outputs within 1 bf16 ulp of the oracle's bf16 rounding of its fp64 result.  Where the
    terms cancel so far that the fp32 evaluation error is not small against a bf16 ulp of the result,
    the value is checked against the fp64 result with that error allowance instead.
    extra: a further allowance per output (fp32 accumulators summed in another order than the reference's)."""
    got_bits = y_gpu_bf16.detach().cpu().view(torch.int16).numpy().astype(np.uint16)
    ref_bits = O.bf16_bits(y64)
    tol32 = fp32_epilogue_tolerance(y64, y_abs, nacc) + extra
    ulp = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(y64), 1e-300))) - 7), 2.0 ** -133)
    stable = tol32 < 0.25 * ulp
    dist = np.abs(bf16_ordered(got_bits) - bf16_ordered(ref_bits))
    assert np.all(dist[stable] <= 1), f"bf16 differs by {dist[stable].max()} ulp"
    got = bf16_value(got_bits)
    err = np.abs(got - y64)
    assert np.all(err[~stable] <= ulp[~stable] + tol32[~stable])
    return float((dist[stable] == 0).mean()) if stable.any() else 1.0


def check_fp32_output(y_gpu_f32: torch.Tensor, y64, y_abs, nacc):
    got = y_gpu_f32.detach().cpu().numpy().astype(np.float64)
    err = np.abs(got - y64)
    tol = fp32_epilogue_tolerance(y64, y_abs, nacc)
    bad = err > tol
    assert not bad.any(), f"{bad.sum()} outputs outside the fp32 tolerance; worst ratio {(err / tol).max():.3g}"
    nz = np.abs(y64) > 0
    return float((err[nz] / np.abs(y64[nz])).max()) if nz.any() else 0.0
