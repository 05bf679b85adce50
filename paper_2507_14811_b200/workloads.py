"""Seeded synthetic layer inputs.

This module only draws random tensors with the shapes and value structure of
the layers the method is applied to (polarity-asymmetric GELU / SiLU outputs,
concatenated streams with different ranges, chunked projections whose segments
have different weight ranges, heavy-tailed pre-activations).  It contains none
of the method's arithmetic: no scale, code, accumulator or dequantization is
computed here.  Both the CPU oracle's tests and the CUDA path's tests and
benchmark take their inputs from here, so that both see identical host buffers.

All tensors are generated on the host with a seeded ``torch.Generator`` in fp32
and then cast to the layer's input dtype.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch


@dataclass
class LayerSpec:
    name: str
    M: int
    K: int
    N: int
    kb: list          # K-partition, P+1 ascending bounds
    nb: list          # N-partition, Q+1 ascending bounds
    dual: bool        # polarity-split activation quantization
    code: str         # "int8" | "e4m3"
    x_dtype: str      # "f32" | "bf16"
    x_kind: str       # input distribution recipe
    w_kind: str       # weight distribution recipe
    seed: int
    cal_rows: int = 256
    x_seg_std: list = field(default_factory=list)  # per-K-segment std of the pre-activation

    @property
    def P(self):
        return len(self.kb) - 1

    @property
    def Q(self):
        return len(self.nb) - 1


def _even_bounds(total, parts):
    assert total % parts == 0
    return [i * (total // parts) for i in range(parts + 1)]


def _gelu(x):
    return 0.5 * x * (1.0 + torch.erf(x / math.sqrt(2.0)))


def _silu(x):
    return x * torch.sigmoid(x)


def _student_t4(shape, g):
    z = torch.randn(shape, generator=g)
    chi2 = torch.zeros(shape)
    for _ in range(4):
        chi2 += torch.randn(shape, generator=g) ** 2
    return z / torch.sqrt(chi2 / 4.0)


def _draw_x(spec: LayerSpec, rows: int, g: torch.Generator) -> torch.Tensor:
    kind = spec.x_kind
    base_kind, _, act = kind.partition("+")
    if base_kind == "normal":
        pre = torch.randn((rows, spec.K), generator=g)
    elif base_kind == "student_t4":
        pre = _student_t4((rows, spec.K), g)
    else:
        raise ValueError(kind)
    if spec.x_seg_std:
        for p, std in enumerate(spec.x_seg_std):
            pre[:, spec.kb[p]:spec.kb[p + 1]] *= std
    if act == "gelu":
        x = _gelu(pre)
    elif act == "silu":
        x = _silu(pre)
    elif act == "geglu":                     # gated GELU: the segment-scaled draw is the value half
        x = pre * _gelu(torch.randn((rows, spec.K), generator=g) * 1.5)
    elif act == "":
        x = pre
    else:
        raise ValueError(kind)
    return x


def _draw_w(spec: LayerSpec, g: torch.Generator) -> torch.Tensor:
    W = torch.randn((spec.N, spec.K), generator=g) * 0.02
    if spec.w_kind == "plain":
        pass
    elif spec.w_kind == "outlier_channels":
        idx = torch.randperm(spec.K, generator=g)[:4]
        W[:, idx] *= 20.0
    elif spec.w_kind == "segment_ladder":
        # N-segment j has standard deviation 0.02 * 10^(j/5): ranges differ by up to 10x
        for j in range(spec.Q):
            W[spec.nb[j]:spec.nb[j + 1], :] *= 10.0 ** (j / 5.0)
    else:
        raise ValueError(spec.w_kind)
    return W


@dataclass
class LayerData:
    spec: LayerSpec
    X: torch.Tensor       # [M,K] in spec.x_dtype
    X_cal: torch.Tensor   # [cal_rows,K] in spec.x_dtype, held-out rows of the same distribution
    W: torch.Tensor       # [N,K] fp32
    bias: torch.Tensor    # [N] fp32


def make_layer(spec: LayerSpec, M: int | None = None) -> LayerData:
    """Draw one layer's tensors.  ``M`` overrides the row count (used by size sweeps and
    by bounded samples of a workload); weights, bias and calibration rows do not depend on it."""
    g = torch.Generator(device="cpu")
    g.manual_seed(spec.seed)
    W = _draw_w(spec, g)
    bias = torch.randn((spec.N,), generator=g) * 0.1
    X_cal = _draw_x(spec, spec.cal_rows, g)
    rows = spec.M if M is None else M
    X = _draw_x(spec, rows, g)
    dt = torch.float32 if spec.x_dtype == "f32" else torch.bfloat16
    return LayerData(spec, X.to(dt).contiguous(), X_cal.to(dt).contiguous(), W.contiguous(), bias)


# --------------------------------------------------------------------------
# The workloads.  Shapes follow the benchmark configurations: a tiny QKV-like
# layer, DiT-XL/2, an SD3-medium MMDiT joint block, FLUX.1 double-stream layers
# (FP8 codes) and an SDXL-like skip-concat 1x1 convolution as a GEMM.
# --------------------------------------------------------------------------

def _spec(name, M, K, N, P=1, Q=1, **kw):
    return LayerSpec(name=name, M=M, K=K, N=N, kb=_even_bounds(K, P), nb=_even_bounds(N, Q), **kw)


WORKLOADS: dict[str, list[LayerSpec]] = {
    "tiny_qkv": [
        _spec("qkv", 256, 256, 768, Q=3, dual=True, code="int8", x_dtype="f32",
              x_kind="normal+gelu", w_kind="outlier_channels", seed=0, cal_rows=64),
    ],
    "dit_xl2": [
        _spec("adaln_mod", 2048, 1152, 6912, Q=6, dual=True, code="int8", x_dtype="bf16",
              x_kind="normal+silu", w_kind="segment_ladder", seed=1000),
        _spec("mlp_fc2", 2048, 4608, 1152, dual=True, code="int8", x_dtype="bf16",
              x_kind="normal+gelu", w_kind="plain", seed=1001, x_seg_std=[1.5]),
    ],
    "sd3_mmdit": [
        _spec("joint_qkv", 8858, 3072, 4608, P=2, Q=3, dual=False, code="int8", x_dtype="bf16",
              x_kind="normal", w_kind="plain", seed=2000, x_seg_std=[1.0, 5.0]),
        _spec("mlp_fc1", 8858, 1536, 6144, dual=False, code="int8", x_dtype="bf16",
              x_kind="normal", w_kind="plain", seed=2001),
        _spec("mlp_fc2", 8858, 6144, 1536, dual=True, code="int8", x_dtype="bf16",
              x_kind="normal+gelu", w_kind="plain", seed=2002, x_seg_std=[1.5]),
    ],
    "flux": [
        _spec("mlp_fc1", 4608, 3072, 12288, dual=False, code="e4m3", x_dtype="bf16",
              x_kind="student_t4", w_kind="plain", seed=3000),
        _spec("mlp_fc2", 4608, 12288, 3072, dual=True, code="e4m3", x_dtype="bf16",
              x_kind="student_t4+gelu", w_kind="plain", seed=3001),
        _spec("modulation", 4608, 3072, 18432, Q=6, dual=True, code="e4m3", x_dtype="bf16",
              x_kind="student_t4+silu", w_kind="segment_ladder", seed=3002),
    ],
    "sdxl_skip": [
        _spec("skip_conv1x1", 32768, 1280, 640, P=2, dual=True, code="int8", x_dtype="bf16",
              x_kind="normal+silu", w_kind="plain", seed=4000, x_seg_std=[1.0, 8.0]),
    ],
}

# the output projection of a gated-GELU feed-forward (SDXL-like transformer blocks at 640 and 1280 channels,
# 64 x 64 and 32 x 32 tokens, batch 2): its input is value * GELU(gate)
WORKLOADS["sdxl_geglu"] = [
    _spec("ff_out_640", 8192, 2560, 640, dual=True, code="int8", x_dtype="bf16",
          x_kind="normal+geglu", w_kind="plain", seed=6000, x_seg_std=[1.5]),
    _spec("ff_out_1280", 2048, 5120, 1280, dual=True, code="int8", x_dtype="bf16",
          x_kind="normal+geglu", w_kind="plain", seed=6001, x_seg_std=[1.5]),
]

# the modulation layers at the row count they have in the real models (one conditioning vector per sample, batch 8
# and batch 1) instead of the token count of the benchmark configurations: bound by streaming the weights
WORKLOADS["modulation_small_m"] = [
    _spec("flux_modulation_M8", 8, 3072, 18432, Q=6, dual=True, code="e4m3", x_dtype="bf16",
          x_kind="student_t4+silu", w_kind="segment_ladder", seed=3002),
    _spec("flux_modulation_M1", 1, 3072, 18432, Q=6, dual=True, code="e4m3", x_dtype="bf16",
          x_kind="student_t4+silu", w_kind="segment_ladder", seed=3002),
    _spec("dit_adaln_M8", 8, 1152, 6912, Q=6, dual=True, code="int8", x_dtype="bf16",
          x_kind="normal+silu", w_kind="segment_ladder", seed=1000),
]

# the other reading of the joint-QKV configuration: 1536 input channels as two concatenated streams of 768
WORKLOADS["sd3_qkv_768x2"] = [
    _spec("joint_qkv_768x2", 8858, 1536, 4608, P=2, Q=3, dual=False, code="int8", x_dtype="bf16",
          x_kind="normal", w_kind="plain", seed=2000, x_seg_std=[1.0, 5.0]),
]

SDXL_SWEEP_M = [512, 1024, 2048, 4096, 8192, 16384, 32768, 65536]

# input segmentation by attention heads: the head-merge reshape in front of an attention output projection
# gives 24 K-segments of 64 channels (SD3.5-medium-like shape), each with its own activation range
WORKLOADS["sd3_heads"] = [
    _spec("attn_out_24x64", 8858, 1536, 1536, P=24, dual=False, code="int8", x_dtype="bf16",
          x_kind="normal", w_kind="plain", seed=5000, x_seg_std=[0.5 + 0.25 * i for i in range(24)]),
    _spec("attn_out_6x256", 8858, 1536, 1536, P=6, dual=False, code="int8", x_dtype="bf16",
          x_kind="normal", w_kind="plain", seed=5001, x_seg_std=[0.5 + i for i in range(6)]),
]

# the skip-concat layer at every row count of the sweep (the points of its roofline curve)
WORKLOADS["sdxl_sweep"] = [
    _spec(f"skip_conv1x1_M{m}", m, 1280, 640, P=2, dual=True, code="int8", x_dtype="bf16",
          x_kind="normal+silu", w_kind="plain", seed=4000, x_seg_std=[1.0, 8.0])
    for m in SDXL_SWEEP_M
]


def small_variant(spec: LayerSpec, M: int, K: int | None = None, N: int | None = None) -> LayerSpec:
    """A reduced copy of a layer (same recipe, segment counts and seed) that the CPU oracle
    finishes in seconds; segment bounds are re-spread evenly over the reduced K and N."""
    K = spec.K if K is None else K
    N = spec.N if N is None else N
    return LayerSpec(name=spec.name + "_small", M=M, K=K, N=N,
                     kb=_even_bounds(K, spec.P), nb=_even_bounds(N, spec.Q),
                     dual=spec.dual, code=spec.code, x_dtype=spec.x_dtype, x_kind=spec.x_kind,
                     w_kind=spec.w_kind, seed=spec.seed, cal_rows=spec.cal_rows,
                     x_seg_std=list(spec.x_seg_std))
