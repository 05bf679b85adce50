"""GPU parity of the rows next to the main path: the zero-point (asymmetric) comparison scheme of App. A and
the act-to-linear prologue (activation function and per-channel multiplier in front of the quantizer), each
against the CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2507_14811_b200 import binding as B
from paper_2507_14811_b200 import workloads as WL
from paper_2507_14811_b200.layer import SegQuantLinear

from parity_util import QRANGE, check_bf16_output, to_f32_np
from test_gpu_parity import custom_spec

pytestmark = pytest.mark.gpu
DEV = "cuda"


# ------------------------------------------------------------------ zero-point scheme (App. A)

def run_zero_point_parity(spec):
    data = WL.make_layer(spec)
    kb, nb, P = spec.kb, spec.nb, spec.P
    Xn, Wn, bn = to_f32_np(data.X), to_f32_np(data.W), to_f32_np(data.bias)
    s_x, z_x = O.calib_act_asym(to_f32_np(data.X_cal), kb)
    s_w = O.calib_weight(Wn, kb, nb)
    Wq = O.quantize_weight(Wn, kb, nb, s_w)
    res = O.layer_forward_asym(Xn, Wq, O.SegTable(kb, nb), s_x, z_x, s_w, bn)

    layer = SegQuantLinear(data.W, data.bias, kb, nb, False, "int8", DEV)
    seg, ws = layer.seg, layer.workspace
    g_s, g_z = B.segquant_calib_zero_point(data.X_cal.to(DEV), seg, ws)
    assert np.array_equal(g_s.cpu().numpy(), s_x) and np.array_equal(g_z.cpu().numpy(), z_x)       # bit-exact
    assert np.array_equal(layer.Wq.cpu().numpy().view(np.int8), Wq)
    codes = B.segquant_quantize_act_zero_point(data.X.to(DEV), seg, g_s, g_z)
    assert np.array_equal(codes.cpu().numpy().view(np.int8), res.codes)                           # bit-exact
    bias_f = B.segquant_fold_zero_point(layer.Wq, seg, g_s, g_z, layer.s_w, layer.bias)
    # the fold in fp32: per K-segment one scale product, one int -> float conversion and one FMA, plus the bias
    fold_abs = np.abs(bn.astype(np.float64))
    for p in range(P):
        q_of_n = np.searchsorted(np.asarray(nb), np.arange(spec.N), side="right") - 1
        fold_abs = fold_abs + np.abs(float(s_x[p]) * s_w[p, q_of_n].astype(np.float64) * int(z_x[p]) * res.wsum[p])
    err = np.abs(bias_f.cpu().numpy().astype(np.float64) - res.bias_folded)
    assert np.all(err <= (3 * P + 1) * 2.0 ** -24 * fold_abs)
    Y32, dump = B.segquant_seglinear_gemm(codes, layer.Wq, seg, "int8", g_s, layer.s_w, bias_f, ws,
                                          y_dtype=torch.float32, dump_acc=True)
    Ybf = B.segquant_seglinear_gemm(codes, layer.Wq, seg, "int8", g_s, layer.s_w, bias_f, ws)
    layer.check_status()
    torch.cuda.synchronize()
    assert np.array_equal(dump.cpu().numpy(), res.acc)                                            # bit-exact
    # the output against the UNFOLDED recovery in fp64: accumulator terms and fold terms each round three times
    tol = 1e-5 * np.abs(res.y64) + (6 * P + 2) * 2.0 ** -24 * res.y_abs
    assert np.all(np.abs(Y32.cpu().numpy().astype(np.float64) - res.y64) <= tol)
    check_bf16_output(Ybf, res.y64, res.y_abs, 2 * P + 1)
    return res


@pytest.mark.parametrize("case", [
    ("zp_small", 200, 256, 136, [0, 256], [0, 136]),
    ("zp_k_segments", 300, 512, 264, [0, 128, 224, 512], [0, 64, 264]),
    ("zp_ragged_tail", 129, 208, 200, [0, 96, 208], [0, 8, 200]),
    ("zp_many_n_segments", 260, 384, 768, [0, 384], [0, 128, 256, 384, 512, 640, 768]),
])
@pytest.mark.parametrize("x_kind", ["normal+gelu", "normal"])
def test_zero_point_scheme_small_shapes(case, x_kind):
    name, M, K, N, kb, nb = case
    run_zero_point_parity(custom_spec(name, M, K, N, kb, nb, False, "int8", x_kind=x_kind,
                                      x_seg_std=[1.0 + 2 * i for i in range(len(kb) - 1)], seed=61))


def test_zero_point_scheme_nonnegative_and_zero_segments():
    """A segment without negative values gets z = -128; an all-zero calibration segment gets s = 1, z = 0."""
    spec = custom_spec("zp_degenerate", 140, 256, 64, [0, 128, 256], [0, 64], False, "int8", x_kind="normal")
    data = WL.make_layer(spec)
    data.X[:, :128] = data.X[:, :128].abs(); data.X_cal[:, :128] = data.X_cal[:, :128].abs()
    data.X_cal[:, 128:] = 0
    s_x, z_x = O.calib_act_asym(to_f32_np(data.X_cal), spec.kb)
    assert z_x[0] == -128 and s_x[1] == 1.0 and z_x[1] == 0
    ws = B.new_workspace(DEV)
    seg = B.SegTable(spec.kb, spec.nb)
    g_s, g_z = B.segquant_calib_zero_point(data.X_cal.to(DEV), seg, ws)
    assert np.array_equal(g_s.cpu().numpy(), s_x) and np.array_equal(g_z.cpu().numpy(), z_x)
    codes = B.segquant_quantize_act_zero_point(data.X.to(DEV), seg, g_s, g_z)
    assert np.array_equal(codes.cpu().numpy().view(np.int8), O.quantize_act_asym(to_f32_np(data.X), spec.kb, s_x, z_x))


def test_zero_point_codes_on_adversarial_values():
    """Exact ties, far-out-of-range inputs, tiny quotients and extreme scales (which take the division path),
    odd and even zero-points."""
    rs = np.random.default_rng(6)
    M, P, seg_len = 512, 8, 256
    K = P * seg_len
    kb = [i * seg_len for i in range(P + 1)]
    exps = [0, -7, 13, -30, 40, -90, 105, 3]
    s = (rs.uniform(1.0, 2.0, P) * np.exp2(exps)).astype(np.float32)
    z = np.array([-128, -77, -1, 0, 1, 64, 127, 13], np.int32)
    X = np.empty((M, K), np.float32)
    for p in range(P):
        blk = rs.uniform(-300, 300, (M, seg_len))
        blk[:, :64] = np.round(blk[:, :64]) + 0.5
        blk[:, 64:96] *= 1e-3
        blk[:, 96:100] *= 1e6
        with np.errstate(over="ignore"):
            X[:, kb[p]:kb[p + 1]] = (blk * float(s[p])).astype(np.float32)
    X[~np.isfinite(X)] = 0.0
    seg = B.SegTable(kb, [0, 8])
    codes = B.segquant_quantize_act_zero_point(torch.from_numpy(X).to(DEV), seg, torch.from_numpy(s).to(DEV),
                                               torch.from_numpy(z).to(DEV))
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy().view(np.int8), O.quantize_act_asym(X, kb, s, z))


@pytest.mark.parametrize("wl,idx", [("dit_xl2", 0), ("dit_xl2", 1), ("sd3_mmdit", 2), ("sdxl_skip", 0)])
def test_zero_point_scheme_full_size_dual_layers(wl, idx):
    """The int8 DualScale layers of the benchmark run as zero-point layers instead (what the benchmark times
    next to them), every row."""
    sp = WL.WORKLOADS[wl][idx]
    run_zero_point_parity(WL.LayerSpec(name=sp.name + "_zp", M=sp.M, K=sp.K, N=sp.N, kb=sp.kb, nb=sp.nb, dual=False,
                                       code="int8", x_dtype=sp.x_dtype, x_kind=sp.x_kind, w_kind=sp.w_kind, seed=sp.seed,
                                       cal_rows=sp.cal_rows, x_seg_std=list(sp.x_seg_std)))


def test_zero_point_calls_reject_bad_arguments_before_launch():
    seg = B.SegTable([0, 128], [0, 64])
    X = torch.zeros((16, 128), dtype=torch.bfloat16, device=DEV)
    ws = B.new_workspace(DEV)
    n0 = B.segquant_launch_count()
    with pytest.raises(B.SegquantError) as e:
        B.segquant_calib_zero_point(X, B.SegTable([0, 64, 32, 128], [0, 64]), ws)
    assert e.value.status == 3
    with pytest.raises(B.SegquantError) as e:
        B.segquant_calib_zero_point(X, seg, torch.zeros(8, dtype=torch.uint8, device=DEV))
    assert e.value.status == 8
    with pytest.raises(B.SegquantError) as e:
        B.segquant_quantize_act_zero_point(X[:, 1:], B.SegTable([0, 127], [0, 64]), torch.ones(1, device=DEV),
                                           torch.zeros(1, dtype=torch.int32, device=DEV))
    assert e.value.status == 4
    assert B.segquant_launch_count() == n0


# ------------------------------------------------------------------ act-to-linear prologue, step 1: the multiplier

@pytest.mark.parametrize("code", ["int8", "e4m3"])
@pytest.mark.parametrize("dual", [True, False])
@pytest.mark.parametrize("x_dtype", ["bf16", "f32"])
def test_per_channel_multiplier_codes_are_exact(code, dual, x_dtype):
    """code = Q(fl32(x * mult[k]) / s): the multiplier is one fp32 multiply on both sides, so the codes are compared
    bit for bit; K-segments, a ragged row end and a chunk that straddles a segment bound included."""
    rs = np.random.default_rng(8)
    spec = custom_spec("mult", 300, 456, 64, [0, 104, 456], [0, 64], dual, code, x_dtype=x_dtype, seed=62,
                       x_seg_std=[1.0, 3.0])
    data = WL.make_layer(spec)
    mult = rs.uniform(0.05, 8.0, spec.K).astype(np.float32)
    Xs = O.smooth(to_f32_np(data.X), mult)
    qmax, qmin_abs = QRANGE[code]
    s_pos, s_neg = O.calib_act(O.smooth(to_f32_np(data.X_cal), mult), spec.kb, dual, q_max=qmax, q_min_abs=qmin_abs)
    r_pos, r_neg = O.quantize_act(Xs, spec.kb, s_pos, s_neg, code=code, q_max=qmax, q_min_abs=qmin_abs)
    seg = B.SegTable(spec.kb, spec.nb)
    c_pos, c_neg = B.segquant_quantize_act_fused(data.X.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                                 torch.from_numpy(s_neg).to(DEV) if dual else None, code,
                                                 act=None, mult=torch.from_numpy(mult).to(DEV))
    torch.cuda.synchronize()
    dt = np.int8 if code == "int8" else np.uint8
    assert np.array_equal(c_pos.cpu().numpy().view(dt), r_pos)
    if dual:
        assert np.array_equal(c_neg.cpu().numpy().view(dt), r_neg)
    # without activation and multiplier the fused entry point is the plain quantizer
    p_pos, p_neg = B.segquant_quantize_act_fused(data.X.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                                 torch.from_numpy(s_neg).to(DEV) if dual else None, code)
    q_pos, q_neg = B.segquant_quantize_act(data.X.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                           torch.from_numpy(s_neg).to(DEV) if dual else None, code)
    assert torch.equal(p_pos, q_pos) and (not dual or torch.equal(p_neg, q_neg))


# ------------------------------------------------------------------ step 2: the activation function

def act_rel_eps(h, act):
    """Relative error bound of the kernel's fp32 evaluation of the activation (stated in the C header)."""
    h = h.astype(np.float64)
    return (np.abs(h) + 8.0) * 2.0 ** -23 if act == "silu" else (3.0 * h ** 2 + 48.0) * 2.0 ** -24


def stored_candidates(h, act, stored):
    """The values the stored activation may take: the oracle's (fp64 evaluation rounded once to the stored dtype)
    and, where the exact value lies within the kernel's error bound of a rounding boundary, its neighbour."""
    a_ref, exact = O.activation(h, act, stored)
    eps = act_rel_eps(h, act)
    lo, hi = exact * (1 - np.sign(exact) * eps), exact * (1 + np.sign(exact) * eps)
    if stored == "bf16":
        rnd = lambda v: (O.bf16_bits(v).astype(np.uint32) << 16).view(np.float32)
    else:
        rnd = lambda v: v.astype(np.float32)
    tiny = np.abs(exact) < 2.0 ** -100                   # below any code's first step: the kernel may flush to zero
    cands = [a_ref, rnd(lo), rnd(hi)]
    return cands, tiny


@pytest.mark.parametrize("table", [2, 1])
@pytest.mark.parametrize("act", ["silu", "gelu"])
@pytest.mark.parametrize("code,dual", [("int8", True), ("int8", False), ("e4m3", True)])
def test_fused_activation_codes_are_valid(act, code, dual, table):
    """H (bf16 pre-activation) -> act -> bf16 -> (multiplier) -> codes in one kernel.  The oracle evaluates the
    activation in fp64 and rounds once; a GPU code must be the oracle's code, or the code of the neighbouring
    bf16 value where the exact activation lies within the kernel's stated error bound of a bf16 rounding
    boundary.  Almost every element must take the first branch.  table: 2 = the activation evaluated per element,
    1 = looked up in the table of all bf16 values that the kernel builds in shared memory."""
    rs = np.random.default_rng(9)
    spec = custom_spec("fact", 700, 512, 64, [0, 192, 512], [0, 64], dual, code, x_kind="normal", seed=63,
                       x_seg_std=[1.5, 3.0])
    data = WL.make_layer(spec)
    H = to_f32_np(data.X)
    H[0, :12] = [0.0, -0.0, 11.5, -11.5, 30.0, -30.0, -60.0, -100.0, 1e-20, -1e-20, 88.0, -88.0]
    H[1, :4] = [1e30, -1e30, 1e19, -1e19]                    # far beyond any activation: the codes saturate, no NaN
    Hb = torch.from_numpy(H).to(torch.bfloat16)
    H = Hb.float().numpy()
    mult = rs.uniform(0.5, 2.0, spec.K).astype(np.float32)
    qmax, qmin_abs = QRANGE[code]
    cal, _ = O.activation(to_f32_np(data.X_cal), act, "bf16")
    s_pos, s_neg = O.calib_act(O.smooth(cal, mult), spec.kb, dual, q_max=qmax, q_min_abs=qmin_abs)
    seg = B.SegTable(spec.kb, spec.nb)
    B.segquant_set_quantize_tuning(table)
    try:
        c_pos, c_neg = B.segquant_quantize_act_fused(Hb.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                                     torch.from_numpy(s_neg).to(DEV) if dual else None, code, act=act,
                                                     mult=torch.from_numpy(mult).to(DEV))
        torch.cuda.synchronize()
    finally:
        B.segquant_set_quantize_tuning(0)
    dt = np.int8 if code == "int8" else np.uint8
    g_pos = c_pos.cpu().numpy().view(dt)
    g_neg = c_neg.cpu().numpy().view(dt) if dual else None
    cands, tiny = stored_candidates(H, act, "bf16")
    ok = np.zeros(H.shape, bool)
    first = None
    for a in cands + [np.zeros_like(cands[0])]:
        r_pos, r_neg = O.quantize_act(O.smooth(a, mult), spec.kb, s_pos, s_neg, code=code, q_max=qmax, q_min_abs=qmin_abs)
        same = (g_pos == r_pos) & ((g_neg == r_neg) if dual else True)
        if first is None:
            first = same
        if a is cands[0] or a is cands[1] or a is cands[2]:
            ok |= same
        else:
            ok |= same & tiny
    assert ok.all(), f"{(~ok).sum()} codes are neither the oracle's nor a neighbour's"
    assert first.mean() > 0.999, f"only {first.mean():.5f} of the codes equal the oracle's"


@pytest.mark.parametrize("act", ["silu", "gelu"])
@pytest.mark.parametrize("case", [
    # M, K, kb, dual, code, scale: several rows per thread, a thread count that is no multiple of the block, two
    # K-segments, both code types, every bf16 bit pattern as input, and scales outside the fast quantizer's range
    (5000, 1024, [0, 1024], True, "int8", None),
    (333, 208, [0, 96, 208], False, "int8", None),
    (700, 512, [0, 192, 512], True, "e4m3", None),
    (4096, 16, [0, 16], True, "int8", None),
    (300, 256, [0, 256], True, "int8", 1e-30),
    (300, 256, [0, 256], False, "e4m3", 1e32),
])
def test_fused_activation_table_equals_the_per_element_evaluation(act, case):
    """The two implementations of the fused activation give the same bytes on every input, all 65536 bf16 bit
    patterns (NaNs and infinities included) among them."""
    M, K, kb, dual, code, scale = case
    g = torch.Generator().manual_seed(91)
    H = (torch.randn((M, K), generator=g) * 2.5).to(torch.bfloat16)
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.bfloat16)
    H.view(-1)[:65536] = bits[: H.numel()] if H.numel() < 65536 else bits
    P = len(kb) - 1
    s_val = [0.02 * (p + 1) for p in range(P)] if scale is None else [scale] * P
    sp = torch.tensor(s_val, dtype=torch.float32, device=DEV)
    sn = (sp * 0.5) if dual else None
    mult = (torch.rand(K, generator=g) + 0.5).to(DEV)
    seg = B.SegTable(kb, [0, 64])
    outs = []
    try:
        for mode in (2, 1):
            B.segquant_set_quantize_tuning(mode)
            outs.append(B.segquant_quantize_act_fused(H.to(DEV), seg, sp, sn, code, act=act, mult=mult))
        torch.cuda.synchronize()
    finally:
        B.segquant_set_quantize_tuning(0)
    assert torch.equal(outs[0][0], outs[1][0])
    if dual:
        assert torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("act", ["silu", "gelu"])
def test_fused_activation_equals_the_unfused_pair_when_the_stored_values_agree(act):
    """Feeding the oracle's stored activation through the plain quantizer gives the codes of the fused call
    wherever the two stored values agree: the quantizer behind the prologue is the same arithmetic."""
    spec = custom_spec("fact2", 400, 384, 64, [0, 384], [0, 64], True, "int8", x_kind="normal", seed=64, x_seg_std=[2.0])
    data = WL.make_layer(spec)
    Hb = data.X
    a_ref, _ = O.activation(to_f32_np(Hb), act, "bf16")
    s_pos, s_neg = O.calib_act(a_ref[:64], spec.kb, True)
    seg = B.SegTable(spec.kb, spec.nb)
    sp, sn = torch.from_numpy(s_pos).to(DEV), torch.from_numpy(s_neg).to(DEV)
    f_pos, f_neg = B.segquant_quantize_act_fused(Hb.to(DEV), seg, sp, sn, "int8", act=act)
    A = torch.from_numpy(a_ref).to(torch.bfloat16)
    assert torch.equal(A.float(), torch.from_numpy(a_ref))             # the oracle's values are bf16 values
    u_pos, u_neg = B.segquant_quantize_act(A.to(DEV), seg, sp, sn, "int8")
    agree = ((f_pos == u_pos) & (f_neg == u_neg)).float().mean().item()
    assert agree > 0.999


@pytest.mark.parametrize("code,dual,dtype", [("int8", True, "bf16"), ("int8", False, "bf16"), ("e4m3", True, "bf16"),
                                             ("int8", True, "f32")])
def test_fused_gated_gelu_codes_are_valid(code, dual, dtype):
    """H [M, 2K] (value half, gate half) -> value * GELU(gate) -> stored dtype -> multiplier -> codes in one kernel
    (App. B: GEGLU is one of the activations in front of DualScale layers).  Same validity rule as for the unary
    activations, with the kernel's bound (3 g^2 + 49) 2^-24 on the relative error of the product."""
    rs = np.random.default_rng(11)
    M, K = 600, 448                                                   # 28 chunks per row; segments of 192 and 256
    kb = [0, 192, K]
    H = np.concatenate([rs.normal(0, 1.5, (M, 192)), rs.normal(0, 3.0, (M, K - 192)), rs.normal(0, 2.0, (M, K))],
                       axis=1).astype(np.float32)
    H[0, :8] = [0.0, -0.0, 5.0, -5.0, 1e-20, 100.0, -100.0, 3.0]
    H[0, K:K + 8] = [1.0, 1.0, -9.0, 9.0, 1.0, -40.0, 40.0, 0.0]
    if dtype == "bf16":
        Hd = torch.from_numpy(H).to(torch.bfloat16)
        H = Hd.float().numpy()
    else:
        Hd = torch.from_numpy(H)
    mult = rs.uniform(0.5, 2.0, K).astype(np.float32)
    qmax, qmin_abs = QRANGE[code]
    a_ref, exact = O.activation_gated(H, dtype)
    s_pos, s_neg = O.calib_act(O.smooth(a_ref[:256], mult), kb, dual, q_max=qmax, q_min_abs=qmin_abs)
    seg = B.SegTable(kb, [0, 64])
    c_pos, c_neg = B.segquant_quantize_act_fused(Hd.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                                 torch.from_numpy(s_neg).to(DEV) if dual else None, code, act="geglu",
                                                 mult=torch.from_numpy(mult).to(DEV))
    torch.cuda.synchronize()
    assert tuple(c_pos.shape) == (M, K)
    dt = np.int8 if code == "int8" else np.uint8
    g_pos = c_pos.cpu().numpy().view(dt)
    g_neg = c_neg.cpu().numpy().view(dt) if dual else None
    gate = H[:, K:].astype(np.float64)
    eps = (3.0 * gate ** 2 + 49.0) * 2.0 ** -24
    lo, hi = exact * (1 - np.sign(exact) * eps), exact * (1 + np.sign(exact) * eps)
    if dtype == "bf16":
        rnd = lambda v: (O.bf16_bits(v).astype(np.uint32) << 16).view(np.float32)
    else:
        rnd = lambda v: v.astype(np.float32)
    tiny = np.abs(exact) < 2.0 ** -100
    ok = np.zeros((M, K), bool)
    first = None
    for j, a in enumerate([a_ref, rnd(lo), rnd(hi), np.zeros_like(a_ref)]):
        r_pos, r_neg = O.quantize_act(O.smooth(a, mult), kb, s_pos, s_neg, code=code, q_max=qmax, q_min_abs=qmin_abs)
        same = (g_pos == r_pos) & ((g_neg == r_neg) if dual else True)
        if first is None:
            first = same
        ok |= same if j < 3 else (same & tiny)
    assert ok.all(), f"{(~ok).sum()} codes are neither the oracle's nor a neighbour's"
    assert first.mean() > 0.999, f"only {first.mean():.5f} of the codes equal the oracle's"


def test_fused_gated_gelu_ragged_row_and_segment_bound_inside_a_chunk():
    """K = 40 (a row tail of 8 elements) with a K-segment bound at 24: every chunk takes the per-element path, and
    the gate half starts at byte 80 of the row."""
    rs = np.random.default_rng(12)
    M, K, kb = 33, 40, [0, 24, 40]
    H = torch.from_numpy(rs.normal(0, 2.0, (M, 2 * K)).astype(np.float32)).to(torch.bfloat16)
    Hn = H.float().numpy()
    a_ref, exact = O.activation_gated(Hn, "bf16")
    s_pos, s_neg = O.calib_act(a_ref, kb, True)
    seg = B.SegTable(kb, [0, 8])
    c_pos, c_neg = B.segquant_quantize_act_fused(H.to(DEV), seg, torch.from_numpy(s_pos).to(DEV),
                                                 torch.from_numpy(s_neg).to(DEV), "int8", act="geglu")
    torch.cuda.synchronize()
    r_pos, r_neg = O.quantize_act(a_ref, kb, s_pos, s_neg, code="int8")
    same = (c_pos.cpu().numpy().view(np.int8) == r_pos) & (c_neg.cpu().numpy().view(np.int8) == r_neg)
    assert same.mean() > 0.995                       # the rest: stored values one bf16 step apart (checked above at size)
    assert np.all(np.abs(c_pos.cpu().numpy().view(np.int8).astype(int) - r_pos) <= 1)
    assert np.all(np.abs(c_neg.cpu().numpy().view(np.int8).astype(int) - r_neg) <= 1)


def test_fused_gated_gelu_rejects_a_gate_half_off_the_16_byte_grid():
    H = torch.zeros(8, 2 * 36, dtype=torch.bfloat16, device=DEV)       # K = 36: the gate half starts at byte 72
    seg = B.SegTable([0, 36], [0, 8])
    s = torch.ones(1, device=DEV)
    with pytest.raises(RuntimeError, match="ALIGN"):
        B.segquant_quantize_act_fused(H, seg, s, s, "int8", act="geglu")


# ------------------------------------------------------------------ W4A8: per-channel 4-bit weights, per-token scales

def run_w4a8_parity(spec):
    data = WL.make_layer(spec)
    kb, P = spec.kb, spec.P
    Xn, Wn, bn = to_f32_np(data.X), to_f32_np(data.W), to_f32_np(data.bias)
    s_w, _, Wq, _ = O.quantize_per_row(Wn, kb, False, q_max=7.0, q_min_abs=7.0)
    res = O.layer_forward_w4a8(Xn, Wq, s_w, kb, spec.dual, bn)

    seg = B.SegTable(kb, [0, spec.N])
    ws = B.new_workspace(DEV)
    # offline: per-channel scales, 4-bit codes, packed
    g_sw, _, g_w8, _ = B.segquant_quantize_per_row(data.W.to(DEV), seg, False, bits=4)
    assert np.array_equal(g_sw.cpu().numpy(), s_w) and np.array_equal(g_w8.cpu().numpy().view(np.int8), Wq)
    packed = B.segquant_pack_w4(g_w8)
    assert np.array_equal(packed.cpu().numpy(), O.pack_w4(Wq))
    # per call: unpack, per-token quantize, GEMM with per-token x per-channel factors
    w8 = B.segquant_unpack_w4(packed)
    assert np.array_equal(w8.cpu().numpy().view(np.int8), Wq)
    g_sp, g_sn, c_pos, c_neg = B.segquant_quantize_per_row(data.X.to(DEV), seg, spec.dual, bits=8)
    assert np.array_equal(g_sp.cpu().numpy(), res.s_pos)
    assert np.array_equal(c_pos.cpu().numpy().view(np.int8), res.c_pos)
    if spec.dual:
        assert np.array_equal(g_sn.cpu().numpy(), res.s_neg)
        assert np.array_equal(c_neg.cpu().numpy().view(np.int8), res.c_neg)
    bias = data.bias.to(DEV)
    Y32, dump = B.segquant_w4a8_gemm(c_pos, c_neg, w8, seg, g_sp, g_sn, g_sw, bias, ws, y_dtype=torch.float32, dump_acc=True)
    Ybf = B.segquant_w4a8_gemm(c_pos, c_neg, w8, seg, g_sp, g_sn, g_sw, bias, ws)
    B.check_device_status(ws)
    torch.cuda.synchronize()
    npol = 2 if spec.dual else 1
    acc = dump.cpu().numpy().reshape(P, npol, spec.M, spec.N)
    assert np.array_equal(acc[:, 0], res.acc_pos)
    if spec.dual:
        assert np.array_equal(acc[:, 1], res.acc_neg)
    from parity_util import check_fp32_output
    check_fp32_output(Y32, res.y64, res.y_abs, P * npol)
    check_bf16_output(Ybf, res.y64, res.y_abs, P * npol)


@pytest.mark.parametrize("dual", [True, False])
@pytest.mark.parametrize("case", [
    ("w4_small", 200, 256, 136, [0, 256]),
    ("w4_k_segments", 300, 512, 264, [0, 128, 224, 512]),
    ("w4_ragged", 129, 208, 200, [0, 96, 208]),
    ("w4_long_row", 70, 16384, 64, [0, 4096, 16384]),
    ("w4_heads", 260, 1536, 320, list(range(0, 1537, 64))),
    ("w4_seg40", 140, 1280, 136, list(range(0, 1281, 32))),      # more K-segments than are staged: checking variant only
])
def test_w4a8_layer_parity(case, dual):
    name, M, K, N, kb = case
    run_w4a8_parity(custom_spec(name, M, K, N, kb, [0, N], dual, "int8", seed=81,
                                x_seg_std=[1.0 + (i % 7) for i in range(len(kb) - 1)]))


@pytest.mark.parametrize("N", [776, 1000, 2048])
def test_w4a8_single_scale_layer_on_wide_tiles(N):
    """The 256 x 512 tiles of single-scale layers with per-(token, channel) factors (forced here; the automatic
    choice takes them on large layers): a ragged last tile, a second half of 8 columns, exact multiples."""
    B.segquant_set_tuning(256, 0, 2, 5)
    try:
        run_w4a8_parity(custom_spec("w4_wide", 700, 384, N, [0, 384], [0, N], False, "int8", seed=83))
    finally:
        B.segquant_set_tuning(0, 0, 0, 0)


def test_w4a8_tokens_of_very_different_magnitude_and_degenerate_rows():
    """Per-token scales: tokens spread over five orders of magnitude, an all-zero token, a token without
    negative values; fp32 input."""
    spec = custom_spec("w4_tokens", 160, 384, 72, [0, 128, 384], [0, 72], True, "int8", x_dtype="f32", seed=82)
    data = WL.make_layer(spec)
    mult = (10.0 ** torch.linspace(-3, 2, spec.M))[:, None]
    data.X = (data.X * mult).contiguous()
    data.X[5] = 0.0
    data.X[6] = data.X[6].abs()
    WL_make = WL.make_layer
    try:
        WL.make_layer = lambda s, M=None: data
        run_w4a8_parity(spec)
    finally:
        WL.make_layer = WL_make


def test_w4a8_full_size_layer_every_row():
    sp = WL.WORKLOADS["dit_xl2"][1]
    run_w4a8_parity(WL.LayerSpec(name="dit_fc2_w4a8", M=sp.M, K=sp.K, N=sp.N, kb=sp.kb, nb=[0, sp.N], dual=True,
                                 code="int8", x_dtype=sp.x_dtype, x_kind=sp.x_kind, w_kind=sp.w_kind, seed=sp.seed,
                                 cal_rows=sp.cal_rows, x_seg_std=list(sp.x_seg_std)))


def test_w4a8_calls_reject_bad_arguments_before_launch():
    X = torch.zeros((16, 16400), dtype=torch.bfloat16, device=DEV)
    n0 = B.segquant_launch_count()
    with pytest.raises(B.SegquantError) as e:
        B.segquant_quantize_per_row(X, B.SegTable([0, 16400], [0, 8]), False)       # longer than a block holds
    assert e.value.status == 5
    seg2 = B.SegTable([0, 128], [0, 32, 64])
    z = torch.zeros((16, 128), dtype=torch.uint8, device=DEV)
    one = torch.ones(64, device=DEV)
    with pytest.raises(B.SegquantError) as e:
        B.segquant_w4a8_gemm(z, None, torch.zeros((64, 128), dtype=torch.uint8, device=DEV), seg2, one, None, one, None,
                             B.new_workspace(DEV))
    assert e.value.status == 3                                                      # output segments: not with per-channel scales
    assert B.segquant_launch_count() == n0
