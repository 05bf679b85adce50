"""Derives the polynomial the fused GELU prologue evaluates (csrc/quantize.cu, gelu_f32) and prints its
coefficients.  Not used at run time.

erfc(t) = exp(-t^2) g(t) with g the scaled complementary error function.  g is smooth and positive on [0, inf);
with z = (t - c) / (t + c), c = 2.5, the range t in [0, 9.6] (beyond it exp(-t^2) underflows in fp32) maps to
z in [-1, 0.59), and a degree-9 polynomial in z, fitted by least squares on the RELATIVE error at Chebyshev nodes,
reproduces g to 2^-29.  The script also replays the kernel's fp32 operation sequence in numpy over every bf16
input in [-13, 13] and prints the largest relative error against h Phi(h) and against the bound the C header states.
"""
import numpy as np
import scipy.special as sp

C, DEG, T_MAX = 2.5, 9, 9.6
f32 = np.float32


def fit():
    z_max = (T_MAX - C) / (T_MAX + C)
    k = np.arange(6000)
    z = (np.cos(np.pi * (k + 0.5) / 6000) + 1) / 2 * (z_max + 1) - 1
    t = C * (1 + z) / (1 - z)
    g = sp.erfcx(t)
    V = np.polynomial.polynomial.polyvander(z, DEG)
    coef, *_ = np.linalg.lstsq(V / g[:, None], np.ones_like(g), rcond=None)
    return coef


def gelu_f32(h, coef):
    h = h.astype(f32)
    t = np.abs(h) * f32(0.70710678118654752440)
    z = ((t - f32(C)) / (t + f32(C))).astype(f32)
    g = np.full(h.shape, f32(coef[-1]), f32)
    for a in coef[-2::-1]:
        g = (g * z + f32(a)).astype(f32)                  # the kernel uses one FMA per step: this is pessimistic
    s = (t * t).astype(f32)
    e = (t.astype(np.float64) ** 2 - s.astype(np.float64)).astype(f32)
    E = (np.exp(-s.astype(np.float64)).astype(f32) * g).astype(f32)
    E = (E - E * e).astype(f32)
    half = (f32(0.5) * h).astype(f32)
    v = np.where(h >= 0, (h - half * E).astype(f32), (half * E).astype(f32))
    return np.where(t >= f32(13.5), np.where(h >= 0, h, f32(-0.0)), v)      # the kernel's cut-off beyond the underflow


if __name__ == "__main__":
    coef = fit()
    print("coefficients, constant term first:")
    print(", ".join("%.9ef" % f32(c) for c in coef))
    h = (np.arange(65536, dtype=np.uint32) << 16).view(np.float32)
    h = h[np.isfinite(h) & (np.abs(h) <= 13.0) & (np.abs(h) >= 2.0 ** -100)]
    exact = h.astype(np.float64) * sp.ndtr(h.astype(np.float64))
    rel = np.abs(gelu_f32(h, coef).astype(np.float64) / exact - 1)
    bound = (3 * h.astype(np.float64) ** 2 + 48) * 2.0 ** -24
    print("every bf16 input in [-13, 13]: max relative error 2^%.1f, at most %.2f of the stated bound; "
          "|h| <= 4: 2^%.1f" % (np.log2(rel.max()), (rel / bound).max(), np.log2(rel[np.abs(h) <= 4].max())))
