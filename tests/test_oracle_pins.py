"""Pins for the CPU oracle: each test checks the oracle against something that is not the
oracle -- a library routine of torch/numpy on CPU, a closed form, an invariant, brute force on
tiny inputs, or the numbers the paper prints (Sec. 4.3.1 range example).  No GPU involved."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def gelu(x):
    return 0.5 * x * (1.0 + np.vectorize(math.erf)(x / math.sqrt(2.0)))


# --------------------------------------------------------------- library quantizer pins

def torch_dual_codes(X, kb, s_pos, s_neg, qmax=127.0, qmin_abs=128.0):
    """Sec. 4.3.2 Q_dual + polarity split written with torch CPU library ops (fp32 divide, round
    half to even, clamp), independent of the C oracle."""
    X = torch.from_numpy(np.asarray(X, np.float32))
    sp = torch.zeros(X.shape[1]); sn = torch.zeros(X.shape[1])
    for p in range(len(kb) - 1):
        sp[kb[p]:kb[p + 1]] = float(s_pos[p]); sn[kb[p]:kb[p + 1]] = float(s_neg[p])
    xp = torch.clamp(X, min=0.0)      # X_+ = max(X,0)
    xn = torch.clamp(X, max=0.0)      # X_- = min(X,0)
    cp = torch.clamp(torch.round(xp / sp), 0, qmax)
    cn = torch.clamp(torch.round(xn / sn), -qmin_abs, 0)
    return cp.numpy().astype(np.int8), cn.numpy().astype(np.int8)


def torch_sym_codes(X, kb, s, qmax=127.0):
    X = torch.from_numpy(np.asarray(X, np.float32))
    sv = torch.zeros(X.shape[1])
    for p in range(len(kb) - 1):
        sv[kb[p]:kb[p + 1]] = float(s[p])
    return torch.clamp(torch.round(X / sv), -qmax, qmax).numpy().astype(np.int8)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_int8_dual_codes_match_library_quantizer(seed):
    r = rng(seed)
    K = 96
    kb = [0, 32, 96]
    X = gelu(r.normal(0, 1.5, (50, K))).astype(np.float32)
    X[0, :8] = [0.0, -0.0, 1e-30, -1e-30, 1e6, -1e6, 0.5, -0.5]       # zeros, denormal-ish, clamp cases
    s_pos = np.array([0.011, 0.023], np.float32)
    s_neg = np.array([0.0013, 0.0021], np.float32)
    cp, cn = O.quantize_act(X, kb, s_pos, s_neg)
    tp, tn = torch_dual_codes(X, kb, s_pos, s_neg)
    assert np.array_equal(cp, tp)
    assert np.array_equal(cn, tn)


def test_int8_ties_round_half_to_even():
    # x/s exactly on .5 boundaries with a power-of-two scale: 0.5->0, 1.5->2, 2.5->2, -0.5->0, -1.5->-2 ...
    s = np.array([0.25], np.float32)
    halves = np.arange(-20, 21, dtype=np.float32) + 0.5
    X = (halves * 0.25).reshape(1, -1).astype(np.float32)
    c, _ = O.quantize_act(X, [0, X.shape[1]], s)
    expect = np.array([float(round(h)) for h in halves])       # Python round() is half-to-even
    assert np.array_equal(c[0].astype(np.float64), expect)
    assert np.array_equal(c, torch_sym_codes(X, [0, X.shape[1]], s))


def test_int8_single_codes_match_library_quantizer():
    r = rng(5)
    X = r.normal(0, 3, (40, 64)).astype(np.float32)
    kb = [0, 16, 48, 64]
    s = np.array([0.02, 0.05, 0.011], np.float32)
    c, none = O.quantize_act(X, kb, s)
    assert none is None
    assert np.array_equal(c, torch_sym_codes(X, kb, s))


def test_weight_codes_match_library_quantizer():
    r = rng(6)
    N, K = 24, 40
    kb, nb = [0, 8, 40], [0, 8, 16, 24]
    W = r.normal(0, 0.02, (N, K)).astype(np.float32)
    s_w = O.calib_weight(W, kb, nb)
    Wq = O.quantize_weight(W, kb, nb, s_w)
    for p, q in itertools.product(range(2), range(3)):
        blk = W[nb[q]:nb[q + 1], kb[p]:kb[p + 1]]
        s = np.float32(np.abs(blk).max()) / np.float32(127.0)
        assert s_w[p, q] == s
        ref = torch.clamp(torch.round(torch.from_numpy(blk) / float(s)), -127, 127).numpy()
        assert np.array_equal(Wq[nb[q]:nb[q + 1], kb[p]:kb[p + 1]], ref.astype(np.int8))
        assert np.abs(Wq[nb[q]:nb[q + 1], kb[p]:kb[p + 1]]).max() == 127   # the extremum maps to the range end


# --------------------------------------------------------------- structural invariants

def test_polarity_split_invariants():
    r = rng(7)
    X = gelu(r.normal(0, 2, (64, 128))).astype(np.float32)
    kb = [0, 128]
    s_pos, s_neg = O.calib_act(X, kb, dual=True)
    cp, cn = O.quantize_act(X, kb, s_pos, s_neg)
    assert cp.min() >= 0 and cp.max() <= 127
    assert cn.max() <= 0 and cn.min() >= -128
    assert np.all((cp.astype(int) * cn.astype(int)) == 0)            # disjoint support (X_+ and X_-)
    assert np.all(cn[X >= 0] == 0) and np.all(cp[X < 0] == 0)
    # calibrated on the same data: both extrema land on the ends of their half-range
    assert cp.max() == 127 and cn.min() == -128
    # monotone in x
    order = np.argsort(X.ravel(), kind="stable")
    combined = (cp.astype(int) + cn.astype(int)).ravel()[order]
    neg_sorted = cn.ravel()[order][X.ravel()[order] < 0]
    pos_sorted = cp.ravel()[order][X.ravel()[order] >= 0]
    assert np.all(np.diff(neg_sorted.astype(int)) >= 0) and np.all(np.diff(pos_sorted.astype(int)) >= 0)
    assert combined.shape == order.shape


def test_on_grid_inputs_reconstruct_exactly():
    r = rng(8)
    kb = [0, 16, 48]
    s_pos = np.array([2.0 ** -5, 2.0 ** -3], np.float32)
    s_neg = np.array([2.0 ** -9, 2.0 ** -8], np.float32)
    codes = r.integers(-128, 128, (32, 48))
    X = np.zeros_like(codes, dtype=np.float32)
    for p in range(2):
        sl = slice(kb[p], kb[p + 1])
        X[:, sl] = np.where(codes[:, sl] >= 0, codes[:, sl] * s_pos[p], codes[:, sl] * s_neg[p])
    cp, cn = O.quantize_act(X, kb, s_pos, s_neg)
    assert np.array_equal(cp.astype(int) + cn.astype(int), codes)
    assert np.array_equal(cp.astype(int), np.maximum(codes, 0))
    assert np.array_equal(cn.astype(int), np.minimum(codes, 0))


def test_half_step_error_bound_inside_calibrated_range():
    r = rng(9)
    X = gelu(r.normal(0, 1.5, (200, 64))).astype(np.float32)
    kb = [0, 64]
    s_pos, s_neg = O.calib_act(X, kb, dual=True)
    cp, cn = O.quantize_act(X, kb, s_pos, s_neg)
    rec = cp.astype(np.float64) * float(s_pos[0]) + cn.astype(np.float64) * float(s_neg[0])
    step = np.where(X >= 0, float(s_pos[0]), float(s_neg[0]))
    assert np.all(np.abs(rec - X.astype(np.float64)) <= 0.5 * step * (1 + 1e-6))


# --------------------------------------------------------------- calibration (Sec. 4.3.2 scale formula)

def test_calibration_closed_form_and_single_segment_is_whole_tensor():
    r = rng(10)
    X = gelu(r.normal(0, 1, (64, 96))).astype(np.float32)
    s_pos, s_neg = O.calib_act(X, [0, 96], dual=True)
    assert s_pos[0] == np.float32(X.max()) / np.float32(127.0)
    assert s_neg[0] == np.float32(-X.min()) / np.float32(128.0)
    s, none = O.calib_act(X, [0, 96], dual=False)
    assert none is None and s[0] == np.float32(np.abs(X).max()) / np.float32(127.0)
    kb = [0, 32, 96]
    sp, sn = O.calib_act(X, kb, dual=True)
    for p in range(2):
        blk = X[:, kb[p]:kb[p + 1]]
        assert sp[p] == np.float32(blk.max()) / np.float32(127.0)
        assert sn[p] == np.float32(-blk.min()) / np.float32(128.0)


def test_calibration_degenerate_ranges_give_unit_scale():
    X = np.abs(rng(11).normal(0, 1, (8, 32))).astype(np.float32)      # no negatives at all
    sp, sn = O.calib_act(X, [0, 32], dual=True)
    assert sn[0] == 1.0 and sp[0] > 0
    cp, cn = O.quantize_act(X, [0, 32], sp, sn)
    assert np.all(cn == 0)
    Z = np.zeros((4, 32), np.float32)
    sp, sn = O.calib_act(Z, [0, 32], dual=True)
    assert sp[0] == 1.0 and sn[0] == 1.0
    assert O.calib_weight(Z, [0, 32], [0, 4])[0, 0] == 1.0


def test_paper_range_example_sec_4_3_1():
    vals = {}
    for line in open(os.path.join(GOLDEN, "sec431_range_example.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    hi, lo = np.float32(vals["max_pos"]), np.float32(vals["min_neg"])
    X = np.linspace(lo, hi, 4096, dtype=np.float32).reshape(64, 64)
    X[0, 0], X[-1, -1] = lo, hi
    sp, sn = O.calib_act(X, [0, 64], dual=True)
    assert sp[0] == hi / np.float32(127.0) and sn[0] == -lo / np.float32(128.0)
    s1, _ = O.calib_act(X, [0, 64], dual=False)
    assert s1[0] == hi / np.float32(127.0)
    # one global scale: the whole negative range collapses onto codes -9..0 (0.26/(3.5/127) = 9.43)
    c1, _ = O.quantize_act(X, [0, 64], s1)
    assert c1.min() == -9 and c1.max() == 127
    # dual scale: negatives use their full half-range
    cp, cn = O.quantize_act(X, [0, 64], sp, sn)
    assert cn.min() == -128 and cp.max() == 127
    assert len(np.unique(cn[X < 0])) > 100 and len(np.unique(c1[X < 0])) == 10


# --------------------------------------------------------------- e4m3 (pinned to torch's cast)

def test_e4m3_decode_matches_torch_and_roundtrip():
    codes = np.arange(256, dtype=np.uint8)
    ours = O.e4m3_decode(codes)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    finite = ~np.isnan(ref)
    assert finite.sum() == 254
    assert np.array_equal(ours[finite], ref[finite]) and np.all(np.isnan(ours[~finite]))
    assert ours[0x7E] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6
    enc = O.e4m3_encode(ours[finite].astype(np.float32))
    expect = codes[finite].copy()
    expect[expect == 0x80] = 0x00                                      # -0 is written as +0
    assert np.array_equal(enc, expect)


def test_e4m3_encode_matches_torch_cast():
    r = rng(12)
    v = np.concatenate([
        r.normal(0, 1, 20000), r.normal(0, 100, 20000), r.uniform(-2 ** -5, 2 ** -5, 20000),
        r.uniform(-460, 460, 5000),
    ]).astype(np.float32)
    # all midpoints between adjacent representable values (ties) and their fp32 neighbours
    grid = np.sort(O.e4m3_decode(np.array([c for c in range(0x7F)], np.uint8)))
    mids = ((grid[1:] + grid[:-1]) / 2).astype(np.float32)
    ties = np.concatenate([mids, np.nextafter(mids, np.float32(1e9)), np.nextafter(mids, np.float32(-1e9))])
    v = np.concatenate([v, ties, -ties]).astype(np.float32)
    v = np.clip(v, -448.0, 448.0)
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    ref[ref == 0x80] = 0x00
    assert np.array_equal(O.e4m3_encode(v), ref)
    assert O.e4m3_encode(np.array([1e9, -1e9, 449.0], np.float32)).tolist() == [0x7E, 0xFE, 0x7E]


def test_e4m3_activation_codes_match_library_cast():
    r = rng(13)
    X = gelu(r.standard_t(4, (32, 64))).astype(np.float32)
    kb = [0, 32, 64]
    sp, sn = O.calib_act(X[:8], kb, True, q_max=448.0, q_min_abs=448.0)   # few rows: runtime exceeds the range
    cp, cn = O.quantize_act(X, kb, sp, sn, code="e4m3")
    Xt = torch.from_numpy(X)
    spv = torch.zeros(64); snv = torch.zeros(64)
    for p in range(2):
        spv[kb[p]:kb[p + 1]] = float(sp[p]); snv[kb[p]:kb[p + 1]] = float(sn[p])
    tp = torch.clamp(torch.clamp(Xt, min=0) / spv, 0, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    tn = torch.clamp(torch.clamp(Xt, max=0) / snv, -448, 0).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    tp[tp == 0x80] = 0; tn[tn == 0x80] = 0
    assert np.array_equal(cp, tp) and np.array_equal(cn, tn)
    assert (cp == 0x7E).any()                                           # the clamp was exercised


def test_e4m3_single_scale_activation_codes_match_library_cast():
    """Single-scale branch of the e4m3 activation quantizer (Sec. 3 quantizer with z = 0, Table 1 "8/8 (fp)"):
    one signed code matrix, clip to [-448, 448], against torch's float8 cast of the fp32 quotient."""
    r = rng(31)
    X = r.standard_t(4, (40, 96)).astype(np.float32)
    X[0, :6] = [0.0, -0.0, 1e-30, -1e-30, 1e6, -1e6]
    kb = [0, 32, 96]
    s, _ = O.calib_act(X[:6], kb, False, q_max=448.0, q_min_abs=448.0)    # few rows: runtime exceeds the range
    c, none = O.quantize_act(X, kb, s, None, code="e4m3")
    assert none is None
    sv = torch.zeros(96)
    for p in range(2):
        sv[kb[p]:kb[p + 1]] = float(s[p])
    t = torch.clamp(torch.from_numpy(X) / sv, -448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    t[t == 0x80] = 0
    assert np.array_equal(c, t)
    assert (c == 0x7E).any() and (c == 0xFE).any()                       # both ends of the clip were exercised
    assert ((c & 0x80) != 0).any()                                       # negative codes exist (not clipped to [0, 448])


def test_e4m3_weight_codes_match_library_cast_per_block():
    """FP8 weight codes, one scale per (K-segment, N-segment) block (Sec. 4.2.2: every W_i is quantized
    separately; Sec. 3 quantizer): each block against torch's float8 cast of W / s_w[p][q].  P = 2 and Q = 3
    with P != Q and blocks of very different ranges, so that a transposed scale index cannot pass."""
    r = rng(32)
    kb, nb = [0, 24, 64], [0, 8, 20, 28]
    W = r.normal(0, 0.02, (28, 64)).astype(np.float32)
    for p in range(2):
        for q in range(3):
            W[nb[q]:nb[q + 1], kb[p]:kb[p + 1]] *= 3.0 ** (p * 3 + q)
    s_w = O.calib_weight(W, kb, nb, w_max=448.0)
    assert s_w.shape == (2, 3) and len(np.unique(s_w)) == 6
    Wq = O.quantize_weight(W, kb, nb, s_w, code="e4m3")
    for p in range(2):
        for q in range(3):
            blk = torch.from_numpy(W[nb[q]:nb[q + 1], kb[p]:kb[p + 1]].copy())
            assert np.float32(blk.abs().max()) / np.float32(448.0) == s_w[p, q]
            t = torch.clamp(blk / float(s_w[p, q]), -448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
            t[t == 0x80] = 0
            assert np.array_equal(Wq[nb[q]:nb[q + 1], kb[p]:kb[p + 1]], t)
            assert (t & 0x7F).max() == 0x7E                               # the block's extremum sits on 448


# --------------------------------------------------------------- accumulators

def test_int8_accumulators_brute_force_tiny():
    r = rng(14)
    M, N, K = 3, 4, 10
    kb = [0, 4, 10]
    Xq = r.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = r.integers(-127, 128, (N, K)).astype(np.int8)
    acc = O.accumulate(Xq, Wq, kb)
    for p in range(2):
        for m in range(M):
            for n in range(N):
                s = 0
                for k in range(kb[p], kb[p + 1]):
                    s += int(Xq[m, k]) * int(Wq[n, k])
                assert acc[p, m, n] == s


def test_int8_accumulators_match_int64_matmul_and_extremes():
    r = rng(15)
    M, N, K = 37, 29, 200
    kb = [0, 64, 200]
    Xq = r.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = r.integers(-127, 128, (N, K)).astype(np.int8)
    Xq[0, :] = -128; Wq[0, :] = -127                                   # largest-magnitude products
    acc = O.accumulate(Xq, Wq, kb)
    for p in range(2):
        ref = Xq[:, kb[p]:kb[p + 1]].astype(np.int64) @ Wq[:, kb[p]:kb[p + 1]].astype(np.int64).T
        assert np.array_equal(acc[p].astype(np.int64), ref)
    assert acc[0, 0, 0] == 64 * 128 * 127


def test_e4m3_accumulators_match_decoded_matmul():
    r = rng(16)
    M, N, K = 9, 7, 64
    kb = [0, 32, 64]
    Xq = r.integers(0, 0x7F, (M, K)).astype(np.uint8) | (r.integers(0, 2, (M, K)).astype(np.uint8) << 7)
    Wq = r.integers(0, 0x7F, (N, K)).astype(np.uint8) | (r.integers(0, 2, (N, K)).astype(np.uint8) << 7)
    acc = O.accumulate(Xq, Wq, kb, code="e4m3")
    xf = torch.from_numpy(Xq.copy()).view(torch.float8_e4m3fn).double().numpy()
    wf = torch.from_numpy(Wq.copy()).view(torch.float8_e4m3fn).double().numpy()
    for p in range(2):
        ref = xf[:, kb[p]:kb[p + 1]] @ wf[:, kb[p]:kb[p + 1]].T
        assert np.allclose(acc[p], ref, rtol=1e-13, atol=0)


# --------------------------------------------------------------- SegLinear compositions (Sec. 4.2.2)

def per_tensor_layer(X, W, dual):
    """An unsegmented per-tensor W8A8 layer with its own arithmetic (torch/numpy library ops only):
    min/max scales, codes, int64 matmul, fp64 recovery (App. A symmetric case, Sec. 4.3.2 dual case)."""
    X = np.asarray(X, np.float32); W = np.asarray(W, np.float32)
    s_w = np.float32(np.abs(W).max()) / np.float32(127.0)
    Wq = torch.clamp(torch.round(torch.from_numpy(W) / float(s_w)), -127, 127).numpy().astype(np.int64)
    if dual:
        sp = np.float32(max(X.max(), 0)) / np.float32(127.0)
        sn = np.float32(max(-X.min(), 0)) / np.float32(128.0)
        cp, cn = torch_dual_codes(X, [0, X.shape[1]], [sp], [sn])
        return (float(sp) * float(s_w)) * (cp.astype(np.int64) @ Wq.T) + (float(sn) * float(s_w)) * (cn.astype(np.int64) @ Wq.T)
    s = np.float32(np.abs(X).max()) / np.float32(127.0)
    c = torch_sym_codes(X, [0, X.shape[1]], [s])
    return (float(s) * float(s_w)) * (c.astype(np.int64) @ Wq.T)


def oracle_layer(X, W, kb, nb, dual, bias=None, code="int8"):
    qm = (127.0, 128.0) if code == "int8" else (448.0, 448.0)
    s_pos, s_neg = O.calib_act(X, kb, dual, q_max=qm[0], q_min_abs=qm[1])
    s_w = O.calib_weight(W, kb, nb, w_max=qm[0])
    Wq = O.quantize_weight(W, kb, nb, s_w, code=code)
    return O.layer_forward(X, Wq, O.SegTable(kb, nb), s_pos, s_neg, s_w, bias, code=code), (s_pos, s_neg, s_w, Wq)


@pytest.mark.parametrize("dual", [False, True])
def test_single_segment_reduces_to_per_tensor_layer(dual):
    r = rng(17)
    X = gelu(r.normal(0, 1, (20, 48))).astype(np.float32)
    W = r.normal(0, 0.02, (12, 48)).astype(np.float32)
    res, _ = oracle_layer(X, W, [0, 48], [0, 12], dual)
    assert np.allclose(res.y64, per_tensor_layer(X, W, dual), rtol=1e-14, atol=0)


@pytest.mark.parametrize("dual", [False, True])
def test_output_segmented_is_concat_of_independent_layers(dual):
    r = rng(18)
    X = gelu(r.normal(0, 1, (16, 40))).astype(np.float32)
    nb = [0, 8, 24, 30]
    W = r.normal(0, 0.02, (30, 40)).astype(np.float32)
    W[8:24] *= 7.0
    res, _ = oracle_layer(X, W, [0, 40], nb, dual)
    ref = np.concatenate([per_tensor_layer(X, W[nb[q]:nb[q + 1]], dual) for q in range(3)], axis=1)
    assert np.allclose(res.y64, ref, rtol=1e-14, atol=0)


@pytest.mark.parametrize("dual", [False, True])
def test_input_segmented_is_sum_of_independent_layers(dual):
    r = rng(19)
    kb = [0, 16, 24, 56]
    X = gelu(r.normal(0, 1, (16, 56))).astype(np.float32)
    X[:, 16:24] *= 6.0
    W = r.normal(0, 0.02, (10, 56)).astype(np.float32)
    res, _ = oracle_layer(X, W, kb, [0, 10], dual)
    ref = sum(per_tensor_layer(X[:, kb[p]:kb[p + 1]], W[:, kb[p]:kb[p + 1]], dual) for p in range(3))
    assert np.allclose(res.y64, ref, rtol=1e-13, atol=1e-18)


# --------------------------------------------------------------- DualScale identities (Sec. 4.3.2, App. A)

def test_equal_dual_scales_reduce_to_symmetric():
    r = rng(20)
    X = r.normal(0, 1, (24, 64)).astype(np.float32)
    W = r.normal(0, 0.02, (16, 64)).astype(np.float32)
    kb, nb = [0, 32, 64], [0, 16]
    s, _ = O.calib_act(X, kb, dual=False)
    s_w = O.calib_weight(W, kb, nb)
    Wq = O.quantize_weight(W, kb, nb, s_w)
    seg = O.SegTable(kb, nb)
    sym = O.layer_forward(X, Wq, seg, s, None, s_w)
    dual = O.layer_forward(X, Wq, seg, s, s.copy(), s_w, q_max=127.0, q_min_abs=127.0)
    assert np.array_equal(dual.c_pos.astype(int) + dual.c_neg.astype(int), sym.c_pos.astype(int))
    assert np.array_equal(dual.acc_pos.astype(np.int64) + dual.acc_neg, sym.acc_pos)
    assert np.allclose(dual.y64, sym.y64, rtol=1e-13, atol=1e-18)


def test_recombination_equals_brute_force_dot_of_dequantized_operands():
    r = rng(21)
    M, N, K = 5, 6, 24
    kb, nb = [0, 8, 24], [0, 2, 6]
    X = gelu(r.normal(0, 1.5, (M, K))).astype(np.float32)
    W = r.normal(0, 0.02, (N, K)).astype(np.float32)
    bias = r.normal(0, 0.1, N).astype(np.float32)
    res, (sp, sn, s_w, Wq) = oracle_layer(X, W, kb, nb, True, bias)
    for m in range(M):
        for n in range(N):
            q = 0 if n < 2 else 1
            tot = float(bias[n])
            for k in range(K):
                p = 0 if k < 8 else 1
                xdq = float(sp[p]) * int(res.c_pos[m, k]) + float(sn[p]) * int(res.c_neg[m, k])
                wdq = float(s_w[p, q]) * int(Wq[n, k])
                tot += xdq * wdq
            assert math.isclose(res.y64[m, n], tot, rel_tol=1e-12, abs_tol=1e-15)


@pytest.mark.parametrize("dual", [False, True])
def test_sum_of_absolute_terms_equals_brute_force(dual):
    """The oracle also reports, per output, sum over (segment, polarity) of |term| + |bias|: the magnitude
    against which an fp32 evaluation of the recombination is judged in the GPU parity tests (it sets their
    tolerance, so it is pinned like a result).  Brute force on a tiny layer with terms of both signs."""
    r = rng(33)
    M, N, K = 4, 5, 24
    kb, nb = [0, 8, 24], [0, 2, 5]
    X = gelu(r.normal(0, 1.5, (M, K))).astype(np.float32)
    W = r.normal(0, 0.02, (N, K)).astype(np.float32)
    bias = r.normal(0, 0.1, N).astype(np.float32)
    res, (sp, sn, s_w, Wq) = oracle_layer(X, W, kb, nb, dual, bias)
    for m in range(M):
        for n in range(N):
            q = 0 if n < 2 else 1
            tot = abs(float(bias[n]))
            for p in range(2):
                ap = sum(int(res.c_pos[m, k]) * int(Wq[n, k]) for k in range(kb[p], kb[p + 1]))
                tot += abs(float(sp[p]) * float(s_w[p, q]) * ap)
                if dual:
                    an = sum(int(res.c_neg[m, k]) * int(Wq[n, k]) for k in range(kb[p], kb[p + 1]))
                    tot += abs(float(sn[p]) * float(s_w[p, q]) * an)
            assert math.isclose(res.y_abs[m, n], tot, rel_tol=1e-12, abs_tol=0)
    assert np.all(res.y_abs >= np.abs(res.y64) * (1 - 1e-12))
    assert (res.y_abs > np.abs(res.y64) * 1.5).any()                    # terms do cancel somewhere
    none_bias = O.layer_forward(X, Wq, O.SegTable(kb, nb), sp, sn, s_w, None)
    assert np.allclose(none_bias.y_abs, res.y_abs - np.abs(bias.astype(np.float64))[None, :], rtol=1e-12, atol=1e-18)


def per_tensor_layer_e4m3(X, W, dual):
    """Unsegmented per-tensor FP8 layer from torch library ops only: abs-max / 448 scales, float8 casts,
    fp64 matmul of the decoded codes (exact), fp64 recovery."""
    X = torch.from_numpy(np.asarray(X, np.float32)); W = torch.from_numpy(np.asarray(W, np.float32))
    f8 = lambda t: t.to(torch.float8_e4m3fn).double()
    s_w = np.float32(W.abs().max()) / np.float32(448.0)
    Wd = f8(torch.clamp(W / float(s_w), -448, 448))
    if dual:
        sp = np.float32(max(float(X.max()), 0)) / np.float32(448.0)
        sn = np.float32(max(-float(X.min()), 0)) / np.float32(448.0)
        xp = f8(torch.clamp(torch.clamp(X, min=0) / float(sp), 0, 448))
        xn = f8(torch.clamp(torch.clamp(X, max=0) / float(sn), -448, 0))
        return ((float(sp) * float(s_w)) * (xp @ Wd.T) + (float(sn) * float(s_w)) * (xn @ Wd.T)).numpy()
    s = np.float32(X.abs().max()) / np.float32(448.0)
    return ((float(s) * float(s_w)) * (f8(torch.clamp(X / float(s), -448, 448)) @ Wd.T)).numpy()


@pytest.mark.parametrize("dual", [False, True])
def test_e4m3_layer_compositions(dual):
    """The FP8 layer through the same reductions as the int8 one: one segment = per-tensor layer,
    output-segmented = concatenation, input-segmented = sum of independent per-tensor layers (Sec. 4.2.2)."""
    r = rng(34)
    X = gelu(r.standard_t(4, (12, 56))).astype(np.float32)
    W = r.normal(0, 0.02, (30, 56)).astype(np.float32)
    W[8:24] *= 7.0
    res, _ = oracle_layer(X, W, [0, 56], [0, 30], dual, code="e4m3")
    assert np.allclose(res.y64, per_tensor_layer_e4m3(X, W, dual), rtol=1e-13, atol=1e-18)
    nb = [0, 8, 24, 30]
    res, _ = oracle_layer(X, W, [0, 56], nb, dual, code="e4m3")
    ref = np.concatenate([per_tensor_layer_e4m3(X, W[nb[q]:nb[q + 1]], dual) for q in range(3)], axis=1)
    assert np.allclose(res.y64, ref, rtol=1e-13, atol=1e-18)
    kb = [0, 16, 24, 56]
    X2 = X.copy(); X2[:, 16:24] *= 6.0
    res, _ = oracle_layer(X2, W, kb, [0, 30], dual, code="e4m3")
    ref = sum(per_tensor_layer_e4m3(X2[:, kb[p]:kb[p + 1]], W[:, kb[p]:kb[p + 1]], dual) for p in range(3))
    assert np.allclose(res.y64, ref, rtol=1e-12, atol=1e-18)


def test_power_of_two_scales_and_on_grid_inputs_give_exact_linear_layer():
    r = rng(22)
    M, N, K = 12, 10, 32
    kb, nb = [0, 16, 32], [0, 4, 10]
    sp = np.array([2.0 ** -4, 2.0 ** -2], np.float32)
    sn = np.array([2.0 ** -8, 2.0 ** -7], np.float32)
    s_w = np.array([[2.0 ** -9, 2.0 ** -7], [2.0 ** -8, 2.0 ** -10]], np.float32)
    cx = r.integers(-128, 128, (M, K)); cw = r.integers(-127, 128, (N, K))
    X = np.zeros((M, K), np.float32); W = np.zeros((N, K), np.float32)
    for p in range(2):
        ks = slice(kb[p], kb[p + 1])
        X[:, ks] = np.where(cx[:, ks] >= 0, cx[:, ks] * sp[p], cx[:, ks] * sn[p])
        for q in range(2):
            W[nb[q]:nb[q + 1], ks] = cw[nb[q]:nb[q + 1], ks] * s_w[p, q]
    bias = (r.integers(-8, 8, N) / 16.0).astype(np.float32)
    Wq = O.quantize_weight(W, kb, nb, s_w)
    assert np.array_equal(Wq, cw)
    res = O.layer_forward(X, Wq, O.SegTable(kb, nb), sp, sn, s_w, bias)
    exact = X.astype(np.float64) @ W.astype(np.float64).T + bias
    assert np.array_equal(res.y64, exact)


def test_output_error_within_closed_form_bound():
    r = rng(23)
    M, N, K = 16, 12, 64
    X = gelu(r.normal(0, 1.5, (M, K))).astype(np.float32)
    W = r.normal(0, 0.02, (N, K)).astype(np.float32)
    res, (sp, sn, s_w, Wq) = oracle_layer(X, W, [0, K], [0, N], True)
    exact = X.astype(np.float64) @ W.astype(np.float64).T
    ex = np.where(X >= 0, float(sp[0]), float(sn[0])) / 2           # |x - x_dq| <= step/2
    ew = float(s_w[0, 0]) / 2
    bound = ex @ np.abs(W.astype(np.float64)).T + (np.abs(X.astype(np.float64)) + ex) @ np.full((K, N), ew)
    assert np.all(np.abs(res.y64 - exact) <= bound * (1 + 1e-9))


# --------------------------------------------------------------- directions the paper reports

def rel_fnorm(y, exact):
    return np.linalg.norm(y - exact) / np.linalg.norm(exact)


def test_dual_scale_lowers_error_on_polarity_asymmetric_input():
    # App. B "Dual Scale Sensitivity Analysis": at strict min/max, DualScale < standard.
    r = rng(24)
    X = gelu(r.normal(0, 1.5, (128, 256))).astype(np.float32)
    W = r.normal(0, 0.02, (64, 256)).astype(np.float32)
    exact = X.astype(np.float64) @ W.astype(np.float64).T
    single, _ = oracle_layer(X, W, [0, 256], [0, 64], False)
    dual, _ = oracle_layer(X, W, [0, 256], [0, 64], True)
    assert rel_fnorm(dual.y64, exact) < rel_fnorm(single.y64, exact)


def test_segmentation_lowers_error_on_heteroscedastic_segments():
    # Sec. 5 single-layer table: segment-wise quantization lowers the F-norm error.
    r = rng(25)
    X = r.normal(0, 1, (128, 128)).astype(np.float32)
    X[:, 64:] *= 8.0
    W = r.normal(0, 0.02, (96, 128)).astype(np.float32)
    W[32:64] *= 10.0
    exact = X.astype(np.float64) @ W.astype(np.float64).T
    unseg, _ = oracle_layer(X, W, [0, 128], [0, 96], False)
    seg, _ = oracle_layer(X, W, [0, 64, 128], [0, 32, 64, 96], False)
    assert rel_fnorm(seg.y64, exact) < rel_fnorm(unseg.y64, exact)


# --------------------------------------------------------------- bf16 rounding helper

def test_bf16_rounding_matches_torch_on_fp32_inputs_and_ties():
    r = rng(26)
    v = np.concatenate([r.normal(0, 1, 5000), r.normal(0, 1e-3, 2000), r.normal(0, 1e4, 2000)]).astype(np.float32)
    # exact ties: bf16 value + half ulp
    base = torch.from_numpy(v[:2000].copy()).to(torch.bfloat16).float().numpy()
    ulp = np.abs(base) * 2.0 ** -8
    exp2 = 2.0 ** np.floor(np.log2(np.abs(base) + 1e-38))
    ties = (base + np.sign(base) * exp2 * 2.0 ** -8).astype(np.float32)
    v = np.concatenate([v, ties])
    ref = torch.from_numpy(v.copy()).to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint16)
    assert np.array_equal(O.bf16_bits(v.astype(np.float64)), ref)
    assert ulp.shape == base.shape
    # a value that double rounding (fp64 -> fp32 -> bf16) would get wrong: just above a bf16 tie
    tie = 1.0 + 2.0 ** -8
    assert O.bf16_bits(np.array([tie + 2.0 ** -40]))[0] == 0x3F81
    assert O.bf16_bits(np.array([tie]))[0] == 0x3F80                  # tie -> even
    assert np.float32(tie + 2.0 ** -40) == np.float32(tie)            # fp32 cannot see the difference


# --------------------------------------------------------------- zero-point (asymmetric) comparison scheme, App. A

def torch_asym_codes(X, kb, s, z):
    X = torch.from_numpy(np.asarray(X, np.float32))
    sv = torch.zeros(X.shape[1]); zv = torch.zeros(X.shape[1])
    for p in range(len(kb) - 1):
        sv[kb[p]:kb[p + 1]] = float(s[p]); zv[kb[p]:kb[p + 1]] = float(z[p])
    return torch.clamp(torch.round(X / sv) + zv, -128, 127).numpy().astype(np.int8)


def test_asym_calibration_closed_form_and_range_ends():
    r = rng(40)
    kb = [0, 16, 48, 64]
    X = gelu(r.normal(0, 1.5, (40, 64))).astype(np.float32)
    X[:, 16:48] = np.abs(X[:, 16:48]) + 0.25                       # a segment without negative values
    X[:, 48:] = 0.0                                                # an all-zero segment
    s, z = O.calib_act_asym(X, kb)
    lo, hi = min(float(X[:, :16].min()), 0.0), max(float(X[:, :16].max()), 0.0)
    assert s[0] == (np.float32(hi) - np.float32(lo)) / np.float32(255.0)
    assert z[0] == int(-128 - np.round(np.float32(lo) / s[0]))
    assert s[1] == np.float32(X[:, 16:48].max()) / np.float32(255.0) and z[1] == -128     # range [0, max]
    assert s[2] == 1.0 and z[2] == 0
    c = O.quantize_act_asym(X, kb, s, z)
    i_lo, i_hi = np.unravel_index(np.argmin(X[:, :16]), (40, 16)), np.unravel_index(np.argmax(X[:, :16]), (40, 16))
    assert c[i_lo] == -128 and c[i_hi] in (126, 127)               # the ends of the range sit on the ends of the code range
    assert np.all(c[:, 48:] == 0)
    # inside the calibrated range the reconstruction s (c - z) is within half a step
    for p in range(2):
        ks = slice(kb[p], kb[p + 1])
        rec = float(s[p]) * (c[:, ks].astype(np.float64) - int(z[p]))
        assert np.all(np.abs(rec - X[:, ks]) <= float(s[p]) / 2 * (1 + 1e-6))


def test_asym_codes_match_library_quantizer():
    r = rng(41)
    kb = [0, 24, 64]
    X = gelu(r.standard_t(4, (60, 64))).astype(np.float32)
    s, z = O.calib_act_asym(X[:6], kb)                              # few rows: run-time values exceed the range
    assert len(set(z.tolist())) == 2
    X[0, :6] = [0.0, -0.0, 1e30, -1e30, 2.5 * s[0], -0.5 * s[0]]    # clip far outside, exact ties
    c = O.quantize_act_asym(X, kb, s, z)
    assert np.array_equal(c, torch_asym_codes(X, kb, s, z))
    assert (c == 127).any() and (c == -128).any()


def asym_layer(X, W, kb, nb, bias=None):
    s_x, z_x = O.calib_act_asym(X, kb)
    s_w = O.calib_weight(W, kb, nb)
    Wq = O.quantize_weight(W, kb, nb, s_w)
    return O.layer_forward_asym(X, Wq, O.SegTable(kb, nb), s_x, z_x, s_w, bias), (s_x, z_x, s_w, Wq)


def test_asym_recovery_equals_brute_force_with_both_zero_points():
    r = rng(42)
    M, N, K = 5, 6, 24
    kb, nb = [0, 8, 24], [0, 2, 6]
    P, Q = 2, 2
    Xq = r.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = r.integers(-128, 128, (N, K)).astype(np.int8)
    s_x = np.array([0.011, 0.37], np.float32); z_x = np.array([-77, 13], np.int32)
    s_w = np.array([[0.002, 0.0031], [0.0007, 0.0013]], np.float32); z_w = np.array([[5, -9], [-3, 21]], np.int32)
    bias = r.normal(0, 0.1, N).astype(np.float32)
    acc = O.accumulate(Xq, Wq, kb)
    xsum, wsum = O.segment_sums(Xq, kb), O.segment_sums(Wq, kb)
    for p in range(P):
        assert np.array_equal(xsum[p], Xq[:, kb[p]:kb[p + 1]].astype(np.int64).sum(axis=1))
        assert np.array_equal(wsum[p], Wq[:, kb[p]:kb[p + 1]].astype(np.int64).sum(axis=1))
    y, ya = O.dequant_asym(acc, xsum, wsum, kb, nb, s_x, z_x, s_w, z_w, bias)
    for m in range(M):
        for n in range(N):
            q = 0 if n < 2 else 1
            tot, tot_abs = float(bias[n]), abs(float(bias[n]))
            for k in range(K):
                p = 0 if k < 8 else 1
                tot += float(s_x[p]) * (int(Xq[m, k]) - int(z_x[p])) * float(s_w[p, q]) * (int(Wq[n, k]) - int(z_w[p, q]))
            for p in range(P):
                c = float(s_x[p]) * float(s_w[p, q])
                kp = kb[p + 1] - kb[p]
                tot_abs += abs(c * int(acc[p, m, n])) + abs(c * int(z_x[p]) * int(wsum[p, n])) + \
                    abs(c * int(z_w[p, q]) * int(xsum[p, m])) + abs(c * kp * int(z_x[p]) * int(z_w[p, q]))
            assert math.isclose(y[m, n], tot, rel_tol=1e-11, abs_tol=1e-13)
            assert math.isclose(ya[m, n], tot_abs, rel_tol=1e-12)


def test_asym_with_zero_zero_points_is_the_symmetric_recovery():
    r = rng(43)
    kb, nb = [0, 32, 64], [0, 8, 16]
    X = r.normal(0, 1, (12, 64)).astype(np.float32)
    W = r.normal(0, 0.02, (16, 64)).astype(np.float32)
    s, _ = O.calib_act(X, kb, dual=False)
    s_w = O.calib_weight(W, kb, nb)
    Wq = O.quantize_weight(W, kb, nb, s_w)
    bias = r.normal(0, 0.1, 16).astype(np.float32)
    sym = O.layer_forward(X, Wq, O.SegTable(kb, nb), s, None, s_w, bias)
    z0 = np.zeros(2, np.int32)
    asym = O.layer_forward_asym(X, Wq, O.SegTable(kb, nb), s, z0, s_w, bias)
    assert np.array_equal(asym.codes, sym.c_pos) and np.array_equal(asym.acc, sym.acc_pos)
    assert np.array_equal(asym.y64, sym.y64) and np.allclose(asym.y_abs, sym.y_abs, rtol=1e-14)
    assert np.array_equal(asym.bias_folded, bias.astype(np.float64))


def test_asym_folded_bias_gives_the_unfolded_recovery():
    r = rng(44)
    kb, nb = [0, 16, 56], [0, 8, 24, 30]
    X = gelu(r.normal(0, 1.5, (14, 56))).astype(np.float32)
    X[:, 16:] *= 4.0
    W = r.normal(0, 0.02, (30, 56)).astype(np.float32)
    W[8:24] *= 5.0
    bias = r.normal(0, 0.1, 30).astype(np.float32)
    res, (s_x, z_x, s_w, Wq) = asym_layer(X, W, kb, nb, bias)
    assert (z_x != 0).all()
    # symmetric recovery of the same accumulators with the folded bias (the form the GPU path runs)
    folded = O.dequant(res.acc.astype(np.float64), None, nb, s_x, None, s_w, None) + res.bias_folded[None, :]
    assert np.allclose(folded, res.y64, rtol=1e-11, atol=1e-13)
    # the fold itself, term by term
    for n in (0, 9, 29):
        q = 0 if n < 8 else (1 if n < 24 else 2)
        t = float(bias[n]) - sum(float(s_x[p]) * float(s_w[p, q]) * int(z_x[p]) *
                                 int(Wq[n, kb[p]:kb[p + 1]].astype(np.int64).sum()) for p in range(2))
        assert math.isclose(res.bias_folded[n], t, rel_tol=1e-12, abs_tol=1e-15)
    # and the layer approximates the real one within the half-step bound of both operands
    exact = X.astype(np.float64) @ W.astype(np.float64).T + bias
    assert np.abs(res.y64 - exact).max() < 0.05 * np.abs(exact).max()


def test_zero_point_lowers_error_on_polarity_asymmetric_input_like_dual_scale():
    # App. A: the asymmetric scheme "can improve accuracy when data distributions are significantly shifted";
    # Sec. 4.3.1: even so its uniform bins resolve the narrow negative range worse than two scales do.
    r = rng(45)
    X = gelu(r.normal(0, 1.5, (128, 256))).astype(np.float32)
    W = r.normal(0, 0.02, (64, 256)).astype(np.float32)
    exact = X.astype(np.float64) @ W.astype(np.float64).T
    single, _ = oracle_layer(X, W, [0, 256], [0, 64], False)
    dual, _ = oracle_layer(X, W, [0, 256], [0, 64], True)
    asym, _ = asym_layer(X, W, [0, 256], [0, 64])
    assert rel_fnorm(asym.y64, exact) < rel_fnorm(single.y64, exact)
    assert rel_fnorm(dual.y64, exact) < rel_fnorm(single.y64, exact)


# --------------------------------------------------------------- act-to-linear segment: activation and multiplier

def test_activation_functions_match_library_and_identities():
    import scipy.special
    h = np.concatenate([np.linspace(-12, 12, 4801), rng(46).normal(0, 3, 2000)])
    L = O.lib()
    silu = np.array([L.sqo_silu(float(v)) for v in h])
    gel = np.array([L.sqo_gelu(float(v)) for v in h])
    ht = torch.from_numpy(h)
    assert np.allclose(silu, torch.nn.functional.silu(ht).numpy(), rtol=1e-13, atol=1e-300)
    assert np.allclose(gel, h * scipy.special.ndtr(h), rtol=1e-12, atol=1e-300)        # GELU(h) = h Phi(h)
    assert np.allclose(gel, torch.nn.functional.gelu(ht).numpy(), rtol=1e-9, atol=1e-14)
    # odd-part identities: f(h) - f(-h) = h for both functions
    for f in (L.sqo_silu, L.sqo_gelu):
        for v in (0.3, 1.0, 2.5, 7.0):
            assert math.isclose(f(v) - f(-v), v, rel_tol=1e-14)
        assert f(0.0) == 0.0
    assert math.isclose(L.sqo_silu(1.0), 1.0 / (1.0 + math.exp(-1.0)), rel_tol=1e-15)
    assert math.isclose(L.sqo_gelu(1.0), 0.5 * (1.0 + math.erf(1.0 / math.sqrt(2.0))), rel_tol=1e-15)
    assert L.sqo_silu(-5.0) < 0 and L.sqo_gelu(-5.0) < 0 and abs(L.sqo_gelu(-5.0)) < 2e-6


@pytest.mark.parametrize("act", ["silu", "gelu"])
def test_activation_is_rounded_once_to_the_stored_dtype(act):
    h = torch.from_numpy(rng(47).normal(0, 2.5, 4000).astype(np.float32)).to(torch.bfloat16).float().numpy()
    out, exact = O.activation(h, act, "bf16")
    bits = out.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0)                                      # bf16 values
    assert np.array_equal((bits >> 16).astype(np.uint16), O.bf16_bits(exact))  # = the pinned fp64 -> bf16 rounding
    ulp = 2.0 ** (np.floor(np.log2(np.abs(exact) + 1e-300)) - 7)
    assert np.all(np.abs(out - exact) <= ulp / 2)
    out32, exact32 = O.activation(h, act, "f32")
    assert np.array_equal(out32, exact32.astype(np.float32)) and np.array_equal(exact32, exact)


def test_gated_gelu_against_library_and_identities():
    """GEGLU (App. B): value half times GELU(gate half).  Pinned to torch's fp64 GELU on the chunked halves, to the
    identity a(v, g) - a(v, -g) = v g, to a(v, 0) = 0 and a(1, g) = GELU(g), and to which half is the gate."""
    r = rng(49)
    M, K = 7, 24
    H = torch.from_numpy(r.normal(0, 2.0, (M, 2 * K)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    out, exact = O.activation_gated(H, "f32")
    value, gate = torch.from_numpy(H).double().chunk(2, dim=1)
    want = (value * torch.nn.functional.gelu(gate)).numpy()
    assert exact.shape == (M, K) and np.allclose(exact, want, rtol=1e-9, atol=1e-14)
    assert np.array_equal(out, exact.astype(np.float32))
    L = O.lib()
    for v, g in [(0.7, 1.3), (-2.0, 0.4), (3.0, -2.5)]:
        assert math.isclose(L.sqo_geglu(v, g) - L.sqo_geglu(v, -g), v * g, rel_tol=1e-13)
        assert L.sqo_geglu(v, 0.0) == 0.0
        assert L.sqo_geglu(1.0, g) == L.sqo_gelu(g)
    # the gate is the SECOND half: a large negative gate closes the unit whatever the value half holds
    Hc = H.copy()
    Hc[:, K:] = -30.0
    assert np.all(np.abs(O.activation_gated(Hc, "f32")[1]) < 1e-100)
    Hc = H.copy()
    Hc[:, :K] = -30.0
    assert np.all(np.abs(O.activation_gated(Hc, "f32")[1])[H[:, K:] > 0.5] > 1e-3)
    # rows do not mix
    out1, _ = O.activation_gated(H[3:4], "f32")
    assert np.array_equal(out1[0], out[3])


def test_gated_gelu_is_rounded_once_to_the_stored_dtype():
    H = torch.from_numpy(rng(50).normal(0, 2.5, (40, 128)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    out, exact = O.activation_gated(H, "bf16")
    bits = out.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0)
    assert np.array_equal((bits >> 16).astype(np.uint16), O.bf16_bits(exact))
    # rounding GELU(gate) to bf16 first and the product again (two roundings) gives different values somewhere
    g16 = O.activation(H[:, 64:], "gelu", "bf16")[0].astype(np.float64)
    twice = O.bf16_bits(H[:, :64].astype(np.float64) * g16)
    assert np.any(twice != (bits >> 16).astype(np.uint16))


def test_smoothing_multiplier_is_one_fp32_multiply():
    r = rng(48)
    X = r.normal(0, 1, (9, 40)).astype(np.float32)
    m = r.uniform(0.1, 4.0, 40).astype(np.float32)
    assert np.array_equal(O.smooth(X, m), X * m[None, :])
    assert O.smooth(X, m).dtype == np.float32


# --------------------------------------------------------------- W4A8: per-channel 4-bit weights, per-token scales

def test_per_row_scales_and_codes_match_closed_form_and_library_quantizer():
    r = rng(50)
    kb = [0, 24, 64]
    X = gelu(r.normal(0, 1.5, (20, 64))).astype(np.float32)
    X[3] = 0.0                                                      # an all-zero token
    X[4, :24] = np.abs(X[4, :24])                                   # a token without negative values in segment 0
    for dual in (False, True):
        s_pos, s_neg, c_pos, c_neg = O.quantize_per_row(X, kb, dual)
        for m in range(20):
            for p in range(2):
                seg = X[m, kb[p]:kb[p + 1]]
                if dual:
                    hi, lo = max(float(seg.max()), 0.0), max(float(-seg.min()), 0.0)
                    assert s_pos[m, p] == (np.float32(hi) / np.float32(127.0) if hi > 0 else 1.0)
                    assert s_neg[m, p] == (np.float32(lo) / np.float32(128.0) if lo > 0 else 1.0)
                else:
                    a = float(np.abs(seg).max())
                    assert s_pos[m, p] == (np.float32(a) / np.float32(127.0) if a > 0 else 1.0)
            # the row's codes are those of the library quantizer with the row's own scales
            if dual:
                tp, tn = torch_dual_codes(X[m:m + 1], kb, s_pos[m], s_neg[m])
                assert np.array_equal(c_pos[m:m + 1], tp) and np.array_equal(c_neg[m:m + 1], tn)
            else:
                assert np.array_equal(c_pos[m:m + 1], torch_sym_codes(X[m:m + 1], kb, s_pos[m]))
        # every token uses its full range: the row extremum sits on the end of the code range
        assert np.all(np.abs(c_pos[[0, 1, 2, 5]].astype(int)).max(axis=1) == 127)
    # 4-bit weights: the same quantizer with q_max = 7
    W = r.normal(0, 0.02, (12, 64)).astype(np.float32)
    s_w, _, Wq, _ = O.quantize_per_row(W, kb, False, q_max=7.0, q_min_abs=7.0)
    assert Wq.min() == -7 and Wq.max() == 7
    for n in range(12):
        assert np.array_equal(Wq[n:n + 1], torch_sym_codes(W[n:n + 1], kb, s_w[n], qmax=7.0))
        assert s_w[n, 1] == np.float32(np.abs(W[n, 24:]).max()) / np.float32(7.0)


def test_w4_pack_roundtrip_and_nibble_order():
    r = rng(51)
    Wq = r.integers(-8, 8, (9, 32)).astype(np.int8)
    packed = O.pack_w4(Wq)
    assert packed.shape == (9, 16)
    assert np.array_equal(O.unpack_w4(packed), Wq)
    one = np.zeros((1, 4), np.int8); one[0] = [1, -1, 7, -8]
    assert O.pack_w4(one).tolist() == [[0xF1, 0x87]]                  # even code in the low nibble, two's complement


@pytest.mark.parametrize("dual", [False, True])
def test_w4a8_recombination_equals_brute_force_and_exact_on_grid(dual):
    r = rng(52)
    M, N, K = 5, 6, 24
    kb = [0, 8, 24]
    X = gelu(r.normal(0, 1.5, (M, K))).astype(np.float32)
    W = r.normal(0, 0.02, (N, K)).astype(np.float32)
    bias = r.normal(0, 0.1, N).astype(np.float32)
    s_w, _, Wq, _ = O.quantize_per_row(W, kb, False, q_max=7.0, q_min_abs=7.0)
    res = O.layer_forward_w4a8(X, O.unpack_w4(O.pack_w4(Wq)), s_w, kb, dual, bias)
    for m in range(M):
        for n in range(N):
            tot, tot_abs = float(bias[n]), abs(float(bias[n]))
            for p in range(2):
                ks = range(kb[p], kb[p + 1])
                ap = sum(int(res.c_pos[m, k]) * int(Wq[n, k]) for k in ks)
                t = float(res.s_pos[m, p]) * float(s_w[n, p]) * ap
                tot += t; tot_abs += abs(t)
                if dual:
                    an = sum(int(res.c_neg[m, k]) * int(Wq[n, k]) for k in ks)
                    u = float(res.s_neg[m, p]) * float(s_w[n, p]) * an
                    tot += u; tot_abs += abs(u)
            assert math.isclose(res.y64[m, n], tot, rel_tol=1e-12, abs_tol=1e-15)
            assert math.isclose(res.y_abs[m, n], tot_abs, rel_tol=1e-12)
    # the layer approximates X W^T + b within the half-step bounds of both operands
    exact = X.astype(np.float64) @ W.astype(np.float64).T + bias
    ex = np.zeros((M, K)); ew = np.zeros((N, K))
    for p in range(2):
        ks = slice(kb[p], kb[p + 1])
        sp = res.s_pos[:, p:p + 1].astype(np.float64)
        sn = res.s_neg[:, p:p + 1].astype(np.float64) if dual else sp
        ex[:, ks] = np.where(X[:, ks] >= 0, sp, sn) / 2
        ew[:, ks] = s_w[:, p:p + 1].astype(np.float64) / 2
    bound = ex @ np.abs(W.astype(np.float64)).T + (np.abs(X.astype(np.float64)) + ex) @ ew.T
    assert np.all(np.abs(res.y64 - exact) <= bound * (1 + 1e-9))
    # power-of-two scales and on-grid operands: exact
    cx = r.integers(-127, 128, (M, K)); cw = r.integers(-7, 8, (N, K))
    cx[:, 0] = 127; cx[:, 8] = -127 if not dual else 127; cw[:, 0] = 7; cw[:, 8] = -7
    if dual:
        cx[:, 1] = -128; cx[:, 9] = -128
    Xg = np.where(cx >= 0, cx * 2.0 ** -5, cx * (2.0 ** -9 if dual else 2.0 ** -5)).astype(np.float32)
    Wg = (cw * 2.0 ** -6).astype(np.float32)
    s_wg, _, Wqg, _ = O.quantize_per_row(Wg, kb, False, q_max=7.0, q_min_abs=7.0)
    assert np.array_equal(Wqg, cw) and np.all(s_wg == 2.0 ** -6)
    resg = O.layer_forward_w4a8(Xg, Wqg, s_wg, kb, dual, None)
    assert np.array_equal(resg.c_pos.astype(int) + (resg.c_neg.astype(int) if dual else 0), cx)
    assert np.array_equal(resg.y64, Xg.astype(np.float64) @ Wg.astype(np.float64).T)


def test_per_token_scales_lower_error_against_one_scale_for_all_tokens():
    # tokens whose magnitudes differ by orders of magnitude: one scale for all of them leaves the small tokens
    # a handful of codes, a scale per token gives every token the full range
    r = rng(53)
    X = r.normal(0, 1, (64, 128)).astype(np.float32) * (10.0 ** r.uniform(-2.0, 1.3, (64, 1))).astype(np.float32)
    s_tok, _, c_tok, _ = O.quantize_per_row(X, [0, 128], False)
    s_all, _ = O.calib_act(X, [0, 128], False)
    c_all, _ = O.quantize_act(X, [0, 128], s_all)
    row_err = lambda rec: np.linalg.norm(rec - X, axis=1) / np.linalg.norm(X, axis=1)
    e_tok = row_err(s_tok.astype(np.float64) * c_tok)
    e_all = row_err(float(s_all[0]) * c_all.astype(np.float64))
    assert np.all(e_tok <= e_all * 1.0001) and np.median(e_tok) < 0.2 * np.median(e_all)
    # and through a layer with 8-bit per-channel weights the output error follows
    W = r.normal(0, 0.02, (32, 128)).astype(np.float32)
    exact = X.astype(np.float64) @ W.astype(np.float64).T
    s_w, _, Wq, _ = O.quantize_per_row(W, [0, 128], False)
    y_tok = O.layer_forward_w4a8(X, Wq, s_w, [0, 128], False).y64
    y_all, _ = O.dequant_per_token(O.accumulate(c_all, Wq, [0, 128]), None, np.full((64, 1), s_all[0], np.float32), None, s_w)
    out_err = lambda y: np.linalg.norm(y - exact, axis=1) / np.linalg.norm(exact, axis=1)
    assert np.median(out_err(y_tok)) < 0.5 * np.median(out_err(y_all))
