"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.
Bit-exact scales, codes and int32 accumulators; fp32 epilogue within 1e-5 relative; bf16 within
1 ulp; e4m3 accumulators within 1e-3 relative."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2507_14811_b200 import binding as B
from paper_2507_14811_b200 import workloads as WL
from paper_2507_14811_b200.layer import SegQuantLinear

from parity_util import (QRANGE, check_bf16_output, check_fp32_output, oracle_scales, to_f32_np)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def custom_spec(name, M, K, N, kb, nb, dual, code, x_dtype="bf16", x_kind="normal+gelu", seed=7, cal_rows=32,
                x_seg_std=None, w_kind="plain"):
    return WL.LayerSpec(name=name, M=M, K=K, N=N, kb=kb, nb=nb, dual=dual, code=code, x_dtype=x_dtype,
                        x_kind=x_kind, w_kind=w_kind, seed=seed, cal_rows=cal_rows, x_seg_std=x_seg_std or [])


def run_parity(spec, rows=None, flags=0, tile_n=0, cta_group=0, segment_mode=0, split=False):
    """Full element-by-element parity of one layer.  rows: optional subset of rows the oracle computes.
    split: give the layer the larger workspace, with which the bf16 call may split tiles along K."""
    data = WL.make_layer(spec)
    qmin_sym = bool(flags & B.SQ_FLAG_QMIN_SYM)
    s_pos, s_neg, s_w, Wq, (qmax, qmin_abs) = oracle_scales(data, qmin_sym)

    B.segquant_set_tuning(tile_n, 0, cta_group, segment_mode)
    try:
        layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, spec.dual, spec.code, DEV, flags)
        if split:
            layer.allow_split_tiles(spec.M)
        g_pos, g_neg = layer.calibrate(data.X_cal)
        # --- scales: bit-exact
        assert np.array_equal(layer.s_w.cpu().numpy().reshape(spec.P, spec.Q), s_w)
        assert np.array_equal(g_pos.cpu().numpy(), s_pos)
        if spec.dual:
            assert np.array_equal(g_neg.cpu().numpy(), s_neg)
        # --- weight codes: bit-exact
        assert np.array_equal(layer.Wq.cpu().numpy().view(Wq.dtype), Wq)

        Xd = data.X.to(DEV)
        Y32, c_pos, c_neg, dump = layer.forward_steps(Xd, y_dtype=torch.float32, dump_acc=True)
        Ybf = layer.forward(Xd)                       # the one-call path, bf16 output
        layer.check_status()
        torch.cuda.synchronize()
        if split:
            # partial sums went through the workspace, every tile counter is back at zero, and a second call
            # (which finds the slots of the first) gives the same bytes; so does the unsplit kernel for int8
            ws = layer.workspace[B.workspace_bytes():]
            assert int(ws.count_nonzero()) > 0, "the layer did not split any tile"
            n_tiles = -(-spec.M // 256) * -(-spec.N // (128 if spec.dual else 256))
            assert int(ws[:8 * n_tiles].count_nonzero()) == 0
            assert torch.equal(layer.forward(Xd), Ybf)
            B.segquant_set_tuning(tile_n, 0, cta_group, 7)
            Y_whole = layer.forward(Xd)
            layer.check_status()
            if spec.code == "int8":
                assert torch.equal(Y_whole, Ybf)
            else:
                assert (Y_whole.float() - Ybf.float()).abs().max() <= 0.02 * Ybf.float().abs().max()
    finally:
        B.segquant_set_tuning(0, 0, 0, 0)

    sel = np.arange(spec.M) if rows is None else np.asarray(rows)
    Xs = to_f32_np(data.X)[sel]
    res = O.layer_forward(Xs, Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w, to_f32_np(data.bias),
                          code=spec.code, q_max=qmax, q_min_abs=qmin_abs)
    # --- activation codes: bit-exact
    dt = np.int8 if spec.code == "int8" else np.uint8
    assert np.array_equal(c_pos.cpu().numpy().view(dt)[sel], res.c_pos)
    if spec.dual:
        assert np.array_equal(c_neg.cpu().numpy().view(dt)[sel], res.c_neg)
    # --- accumulators
    acc_extra = 0.0
    npol = 2 if spec.dual else 1
    acc = dump.cpu().numpy().reshape(spec.P, npol, spec.M, spec.N)[:, :, sel]
    nacc = spec.P * npol
    if spec.code == "int8":
        assert np.array_equal(acc[:, 0], res.acc_pos)
        if spec.dual:
            assert np.array_equal(acc[:, 1], res.acc_neg)
        y64, y_abs = res.y64, res.y_abs
    else:
        # e4m3: tensor-core fp32 accumulation against exact sums; judged against the sum of |products|
        mag = lambda c: (np.asarray(c, np.uint8) & 0x7F)
        q_of_n = np.searchsorted(np.asarray(spec.nb), np.arange(spec.N), side="right") - 1
        for pol, (cx, ref) in enumerate([(res.c_pos, res.acc_pos), (res.c_neg, res.acc_neg)][:npol]):
            abs_sum = O.accumulate(mag(cx), mag(Wq), spec.kb, code="e4m3")
            err = np.abs(acc[:, pol].astype(np.float64) - ref)
            allow = 1e-3 * np.abs(ref) + 1e-5 * abs_sum
            assert np.all(err <= allow), \
                f"e4m3 accumulator error {np.max(err / np.maximum(abs_sum, 1e-30)):.3g} of sum|prod|"
            if split:      # the split kernel adds fp32 partial sums: its accumulators get the same allowance again
                s_act = (s_pos, s_neg)[pol].astype(np.float64)
                c = s_act[:, None] * s_w.reshape(spec.P, spec.Q).astype(np.float64)[:, q_of_n]      # [P, N]
                acc_extra = acc_extra + (c[:, None, :] * allow).sum(0)
        # epilogue is judged on the accumulators the GPU produced
        a_pos = acc[:, 0].astype(np.float64)
        a_neg = acc[:, 1].astype(np.float64) if spec.dual else None
        y64, y_abs = O.dequant(a_pos, a_neg, spec.nb, s_pos, s_neg, s_w, to_f32_np(data.bias), with_abs=True)
    # --- epilogue
    check_fp32_output(Y32[torch.as_tensor(sel, device=DEV)], y64, y_abs, nacc)
    check_bf16_output(Ybf[torch.as_tensor(sel, device=DEV)], y64, y_abs, nacc, extra=acc_extra)
    return res


# ------------------------------------------------------------------ small shapes, every element

def test_config_tiny_qkv_full_parity():
    run_parity(WL.WORKLOADS["tiny_qkv"][0])


@pytest.mark.parametrize("case", [
    # name, M, K, N, kb, nb, dual, code
    ("ragged_m_single", 300, 256, 256, [0, 256], [0, 256], False, "int8"),
    ("ragged_everything_dual", 129, 208, 200, [0, 96, 208], [0, 64, 200], True, "int8"),
    ("one_row", 1, 128, 64, [0, 128], [0, 64], True, "int8"),
    ("k_tail_16", 70, 48, 40, [0, 48], [0, 8, 40], True, "int8"),
    ("four_k_segments_dual", 260, 512, 192, [0, 128, 224, 384, 512], [0, 192], True, "int8"),
    ("eight_k_segments_dual", 150, 512, 96, [0, 64, 128, 192, 256, 320, 384, 448, 512], [0, 96], True, "int8"),
    ("sixteen_k_segments_single", 140, 1024, 72, list(range(0, 1025, 64)), [0, 72], False, "int8"),
    ("six_n_segments", 257, 384, 768, [0, 384], [0, 128, 256, 384, 512, 640, 768], True, "int8"),
    ("uneven_n_segments", 200, 256, 520, [0, 256], [0, 8, 264, 520], False, "int8"),
    ("multi_tile_long_k", 384, 2304, 512, [0, 2304], [0, 512], True, "int8"),
    ("e4m3_single", 200, 256, 256, [0, 256], [0, 256], False, "e4m3"),
    ("e4m3_dual_seg", 260, 384, 320, [0, 128, 384], [0, 64, 320], True, "e4m3"),
])
def test_small_shapes_full_parity(case):
    name, M, K, N, kb, nb, dual, code = case
    run_parity(custom_spec(name, M, K, N, kb, nb, dual, code, x_seg_std=[1.0 + 2 * i for i in range(len(kb) - 1)]))


@pytest.mark.parametrize("cta_group", [1, 2])
@pytest.mark.parametrize("tile_n", [32, 64, 128, 256])
def test_every_tile_width(tile_n, cta_group):
    run_parity(custom_spec("tile", 200, 384, 520, [0, 384], [0, 256, 520], False, "int8"), tile_n=tile_n,
               cta_group=cta_group)


@pytest.mark.parametrize("cta_group", [1, 2])
@pytest.mark.parametrize("tile_n", [64, 128, 256])
def test_every_tile_width_dual(tile_n, cta_group):
    run_parity(custom_spec("tile_dual", 300, 640, 776, [0, 640], [0, 776], True, "int8"), tile_n=tile_n,
               cta_group=cta_group)


@pytest.mark.parametrize("case", [
    # name, M, K, N, nb, code: single-scale layers whose bf16 output takes the 256 x 512 tiles (an even number of
    # 256-column tiles): exact, a second half of 8 columns, ragged rows, several N-segments, both code types
    ("wide_exact", 256, 256, 512, [0, 512], "int8"),
    ("wide_tail8", 300, 384, 776, [0, 256, 776], "int8"),
    ("wide_ragged", 700, 400, 1000, [0, 160, 480, 1000], "int8"),
    ("wide_e4m3", 260, 256, 1536, [0, 1536], "e4m3"),
    ("wide_many", 520, 128, 2560, [0, 2560], "int8"),
])
def test_wide_single_scale_tiles(case):
    name, M, K, N, nb, code = case
    run_parity(custom_spec(name, M, K, N, [0, K], nb, False, code, x_kind="normal", seed=51), tile_n=256, cta_group=2,
               segment_mode=5)
    # the same layer with 256 x 256 tiles gives the same bytes
    spec = custom_spec(name, M, K, N, [0, K], nb, False, code, x_kind="normal", seed=51)
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, False, code, DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    try:
        B.segquant_set_tuning(256, 0, 2, 5)
        Y_wide = layer.forward(Xd)
        B.segquant_set_tuning(256, 0, 2, 4)
        Y_narrow = layer.forward(Xd)
        layer.check_status()
        torch.cuda.synchronize()
    finally:
        B.segquant_set_tuning(0, 0, 0, 0)
    assert torch.equal(Y_wide, Y_narrow)


@pytest.mark.parametrize("case", [
    # layers with one K-segment whose K loops are cut across CTA pairs (the larger workspace; forced here): fewer
    # tiles than pairs (every tile shared by several pairs), a few more tiles than pairs, ragged M / N / K,
    # a K of two blocks (most pairs get one block or none), several N-segments, both code types and polarities
    ("split_few_tiles_dual", 512, 4608, 256, [0, 256], True, "int8"),
    ("split_one_tile_single", 200, 9216, 256, [0, 256], False, "int8"),
    ("split_ragged_dual", 1300, 1072, 392, [0, 128, 392], True, "int8"),
    ("split_ragged_single", 2100, 2000, 776, [0, 512, 776], False, "int8"),
    ("split_short_k", 2560, 256, 1280, [0, 1280], True, "int8"),
    ("split_e4m3_dual", 700, 3072, 384, [0, 384], True, "e4m3"),
    ("split_e4m3_single", 520, 2048, 520, [0, 520], False, "e4m3"),
])
def test_split_tiles(case):
    name, M, K, N, nb, dual, code = case
    run_parity(custom_spec(name, M, K, N, [0, K], nb, dual, code, seed=71), segment_mode=6, split=True)


@pytest.mark.parametrize("cta_group", [1, 2])
@pytest.mark.parametrize("case", [
    # the CTA-pair tile is 256 rows: M at, just below and just above its multiples; a second CTA with no rows
    ("pair_exact", 512, 256, 256, [0, 256], [0, 256], True, "int8"),
    ("pair_plus_one", 257, 256, 264, [0, 128, 256], [0, 264], True, "int8"),
    ("pair_second_cta_empty", 120, 256, 136, [0, 256], [0, 136], False, "int8"),
    ("pair_many_tiles", 1100, 384, 1032, [0, 384], [0, 512, 1032], False, "int8"),
    ("pair_e4m3", 640, 512, 520, [0, 256, 512], [0, 520], True, "e4m3"),
])
def test_cta_pair_edges(case, cta_group):
    name, M, K, N, kb, nb, dual, code = case
    run_parity(custom_spec(name, M, K, N, kb, nb, dual, code), cta_group=cta_group)


@pytest.mark.parametrize("segment_mode", [1, 2])
@pytest.mark.parametrize("case", [
    # layers with several K-segments, with all accumulators resident in tensor memory (1) and with the
    # segments passing through it one after the other (2)
    ("two_k_dual", 300, 512, 384, [0, 256, 512], [0, 384], True, "int8"),
    ("three_k_single_uneven", 260, 416, 264, [0, 96, 160, 416], [0, 136, 264], False, "int8"),
    ("four_k_dual_e4m3", 520, 1024, 256, [0, 256, 512, 768, 1024], [0, 128, 256], True, "e4m3"),
    ("eight_k_single_one_row_tile", 100, 1024, 520, list(range(0, 1025, 128)), [0, 520], False, "int8"),
])
def test_k_segments_resident_and_sequential(case, segment_mode):
    name, M, K, N, kb, nb, dual, code = case
    run_parity(custom_spec(name, M, K, N, kb, nb, dual, code, x_seg_std=[1.0 + 3 * i for i in range(len(kb) - 1)]),
               segment_mode=segment_mode)


@pytest.mark.parametrize("dual", [False, True])
def test_many_small_k_segments(dual):
    """24 K-segments of 64 codes (the head-merge reshape in front of an attention output projection) and
    40 segments of 32: more accumulators than tensor memory could hold at once."""
    run_parity(custom_spec("heads24", 300, 1536, 320, list(range(0, 1537, 64)), [0, 320], dual, "int8",
                           x_seg_std=[0.5 + 0.4 * i for i in range(24)]))
    run_parity(custom_spec("seg40", 140, 1280, 136, list(range(0, 1281, 32)), [0, 64, 136], dual, "int8",
                           x_seg_std=[1.0 + 0.2 * i for i in range(40)]))


@pytest.mark.parametrize("chunks", [1, 3, 8])
def test_pipelined_host_call_equals_the_plain_one(chunks):
    """Pinned-host input and output with the copies on their own streams: same bytes as the one-stream call."""
    spec = custom_spec("pipe", 1500, 384, 520, [0, 128, 384], [0, 256, 520], True, "int8")
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    Xh = data.X.pin_memory()
    x_stage = torch.empty_like(data.X, device=DEV)
    y_stage = torch.empty((spec.M, spec.N), dtype=torch.bfloat16, device=DEV)
    Y_plain = torch.empty((spec.M, spec.N), dtype=torch.bfloat16).pin_memory()
    Y_pipe = torch.full((spec.M, spec.N), 3.0, dtype=torch.bfloat16).pin_memory()
    layer.forward(Xh, Y=Y_plain, x_stage=x_stage, y_stage=y_stage)
    torch.cuda.synchronize()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    layer.forward_pipelined(Xh, Y_pipe, x_stage, y_stage, chunks, s_in, s_out)
    torch.cuda.current_stream().synchronize()          # the compute stream alone is synchronized, as documented
    layer.check_status()
    assert torch.equal(Y_plain, Y_pipe)
    res = O.layer_forward(to_f32_np(data.X), *[oracle_scales(data)[i] for i in (3,)],
                          O.SegTable(spec.kb, spec.nb), *oracle_scales(data)[:3], to_f32_np(data.bias))
    check_bf16_output(Y_pipe, res.y64, res.y_abs, 4)


def _codes_and_output_buffers(spec):
    c_pos = B.new_codes(spec.M, spec.K, DEV)
    c_neg = B.new_codes(spec.M, spec.K, DEV) if spec.dual else None
    return c_pos, c_neg


def test_back_to_back_calls_on_shared_code_buffers_do_not_race():
    """Four quantize -> GEMM rounds on different inputs, issued without any synchronisation, all through the SAME
    code matrices: the launches overlap (programmatic dependent launch), yet every round's output must be the one
    of its own input, i.e. no quantize pass may overwrite codes that the previous GEMM is still reading."""
    spec = custom_spec("b2b", 2300, 512, 768, [0, 512], [0, 256, 768], True, "int8", seed=11)
    data = WL.make_layer(spec)
    s_pos, s_neg, s_w, Wq, _ = oracle_scales(data)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    rounds = 4
    Xs = [torch.roll(data.X, shifts=17 * r, dims=0) * (1.0 + 0.25 * r) for r in range(rounds)]
    Xd = [x.to(DEV) for x in Xs]
    Ys = [torch.empty((spec.M, spec.N), dtype=torch.bfloat16, device=DEV) for _ in range(rounds)]
    c_pos, c_neg = _codes_and_output_buffers(spec)
    torch.cuda.synchronize()
    for r in range(rounds):
        B.segquant_quantize_act(Xd[r], layer.seg, layer.s_pos, layer.s_neg, "int8", 0, c_pos, c_neg)
        B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_neg, layer.s_w,
                                  layer.bias, layer.workspace, Y=Ys[r])
    layer.check_status()
    torch.cuda.synchronize()
    rows = np.arange(0, spec.M, 37)
    for r in range(rounds):
        res = O.layer_forward(to_f32_np(Xs[r])[rows], Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w,
                              to_f32_np(data.bias))
        check_bf16_output(Ys[r][torch.as_tensor(rows, device=DEV)], res.y64, res.y_abs, 2)


@pytest.mark.parametrize("wl,idx", [("dit_xl2", 0), ("dit_xl2", 1), ("sdxl_skip", 0)])
def test_repeated_full_size_launches_are_bitwise_identical(wl, idx):
    """Forty back-to-back launches of a full-size benchmark layer (many tiles per CTA pair, so every hand-over
    between the MMA issuer and the epilogue warps happens thousands of times) give the same bytes every time."""
    spec = WL.WORKLOADS[wl][idx]
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, spec.dual, spec.code, DEV)
    layer.calibrate(data.X_cal)
    c_pos, c_neg = B.segquant_quantize_act(data.X.to(DEV), layer.seg, layer.s_pos, layer.s_neg, spec.code)
    Ys = [torch.empty((spec.M, spec.N), dtype=torch.bfloat16, device=DEV) for _ in range(3)]

    def gemm(Y):
        if spec.dual:
            B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, spec.code, layer.s_pos, layer.s_neg,
                                      layer.s_w, layer.bias, layer.workspace, Y=Y)
        else:
            B.segquant_seglinear_gemm(c_pos, layer.Wq, layer.seg, spec.code, layer.s_pos, layer.s_w, layer.bias,
                                      layer.workspace, Y=Y)
    gemm(Ys[0])
    torch.cuda.synchronize()
    for r in range(20):
        gemm(Ys[1])
        gemm(Ys[2])
        if r % 5 == 4:
            torch.cuda.synchronize()
            assert torch.equal(Ys[1], Ys[0]) and torch.equal(Ys[2], Ys[0]), f"launch {2 * r} differs"
            Ys[1].zero_()
            Ys[2].zero_()
    layer.check_status()


def test_calls_can_be_captured_in_a_cuda_graph_and_replayed():
    """quantize -> GEMM captured once into a CUDA graph (the calls allocate nothing and query nothing that a
    capture forbids); two replays on changed input contents give the outputs of eager calls."""
    spec = custom_spec("graph", 700, 384, 520, [0, 128, 384], [0, 256, 520], True, "int8", seed=12)
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    X_in = Xd.clone()
    c_pos, c_neg = _codes_and_output_buffers(spec)
    Y = torch.empty((spec.M, spec.N), dtype=torch.bfloat16, device=DEV)

    def calls():
        B.segquant_quantize_act(X_in, layer.seg, layer.s_pos, layer.s_neg, "int8", 0, c_pos, c_neg)
        B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_neg, layer.s_w,
                                  layer.bias, layer.workspace, Y=Y)

    calls()                                            # eager: loads the kernels, sets their attributes
    torch.cuda.synchronize()
    Y_eager0 = Y.clone()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream, capture_error_mode="relaxed"):
            calls()
    torch.cuda.current_stream().wait_stream(stream)
    Y.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(Y, Y_eager0)
    X_in.copy_(torch.flip(Xd, dims=[0]) * 0.5)
    graph.replay()
    torch.cuda.synchronize()
    Y_graph1 = Y.clone()
    calls()
    layer.check_status()
    torch.cuda.synchronize()
    assert torch.equal(Y_graph1, Y)
    assert not torch.equal(Y_graph1, Y_eager0)


def _random_case(i):
    rs = np.random.default_rng(1000 + i)
    P = int(rs.choice([1, 1, 2, 3, 5, 9, 17]))
    Q = int(rs.choice([1, 1, 2, 4, 7]))
    kb = np.concatenate([[0], np.cumsum(rs.integers(1, 6, P)) * 32])          # interior bounds multiples of 32
    if rs.random() < 0.5:
        kb[-1] -= 16                                                           # K a multiple of 16 only
    nb = np.concatenate([[0], np.cumsum(rs.integers(1, 12, Q)) * (8 if rs.random() < 0.5 else 32)])
    M = int(rs.choice([1, 7, 128, 129, 255, 257, 300, 520]))
    return dict(M=M, K=int(kb[-1]), N=int(nb[-1]), kb=[int(v) for v in kb], nb=[int(v) for v in nb],
                dual=bool(rs.random() < 0.6), code=str(rs.choice(["int8", "int8", "e4m3"])))


@pytest.mark.parametrize("i", range(24))
def test_random_shapes_and_segment_tables(i):
    """Seeded random layers: segment counts from 1 to 17 (K) and 1 to 7 (N), bounds at the alignment minima,
    row counts around the 128- and 256-row tile edges, both code types, dual and single."""
    c = _random_case(i)
    run_parity(custom_spec(f"rand{i}", c["M"], c["K"], c["N"], c["kb"], c["nb"], c["dual"], c["code"],
                           x_seg_std=[0.5 + (j % 5) for j in range(len(c["kb"]) - 1)], seed=100 + i))


def test_strided_output_and_code_matrices():
    """Y with a row pitch larger than N (a column slice of a wider buffer) is written only inside its
    N columns, and code matrices with a padded pitch are read correctly."""
    spec = custom_spec("strided", 300, 256, 200, [0, 256], [0, 200], True, "int8")
    data = WL.make_layer(spec)
    s_pos, s_neg, s_w, Wq, (qmax, qmin_abs) = oracle_scales(data)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    wide = torch.full((spec.M, 256), 7.0, dtype=torch.bfloat16, device=DEV)
    Y = wide[:, 8:208]
    c_pos, c_neg = B.segquant_quantize_act(Xd, layer.seg, layer.s_pos, layer.s_neg, "int8")
    B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_neg, layer.s_w,
                              layer.bias, layer.workspace, Y=Y)
    layer.check_status()
    torch.cuda.synchronize()
    assert torch.all(wide[:, :8] == 7.0) and torch.all(wide[:, 208:] == 7.0)
    res = O.layer_forward(to_f32_np(data.X), Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w,
                          to_f32_np(data.bias))
    check_bf16_output(Y.contiguous(), res.y64, res.y_abs, 2)


@pytest.mark.parametrize("col0,pitch", [(0, 328), (8, 328), (16, 328), (4, 328), (0, 324), (24, 1024)])
@pytest.mark.parametrize("dual", [True, False])
def test_output_alignment_and_pitch_variants(col0, pitch, dual):
    """The bf16 output goes out through TMA stores, which need Y and its pitch 16-byte aligned: the interface
    demands exactly that, so a column offset of 4 (8 bytes) or a pitch of 324 (648 bytes) is refused, and
    every accepted placement (16-byte but not 32-byte aligned included) writes exactly the M x N window:
    300 rows end inside a 32-row block, 296 columns end inside a 32-column slab."""
    M, K, N = 300, 384, 296
    spec = custom_spec(f"align{col0}_{pitch}_{int(dual)}", M, K, N, [0, K], [0, 160, N], dual, "int8", seed=77)
    data = WL.make_layer(spec)
    s_pos, s_neg, s_w, Wq, _ = oracle_scales(data)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, dual, "int8", DEV)
    layer.calibrate(data.X_cal)
    wide = torch.full((M + 2, pitch), -3.0, dtype=torch.bfloat16, device=DEV)
    Y = wide[1:M + 1, col0:col0 + N]
    c_pos, c_neg = B.segquant_quantize_act(data.X.to(DEV), layer.seg, layer.s_pos, layer.s_neg, "int8")
    def call():
        if dual:
            B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_neg, layer.s_w,
                                      layer.bias, layer.workspace, Y=Y)
        else:
            B.segquant_seglinear_gemm(c_pos, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_w, layer.bias,
                                      layer.workspace, Y=Y)
    if (col0 * 2) % 16 or (pitch * 2) % 16:
        with pytest.raises(Exception, match="SQ_ERR_ALIGN"):
            call()
        torch.cuda.synchronize()
        assert torch.all(wide == -3.0)
        return
    call()
    layer.check_status()
    torch.cuda.synchronize()
    outside = wide.clone()
    outside[1:M + 1, col0:col0 + N] = -3.0
    assert torch.all(outside == -3.0), "wrote outside the M x N window"
    res = O.layer_forward(to_f32_np(data.X), Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg if dual else None, s_w,
                          to_f32_np(data.bias))
    check_bf16_output(Y.contiguous(), res.y64, res.y_abs, 2 if dual else 1)


@pytest.mark.parametrize("code", ["int8", "e4m3"])
@pytest.mark.parametrize("dual", [True, False])
def test_quantizer_codes_equal_the_division_definition_on_adversarial_values(code, dual):
    """Codes are defined by one IEEE fp32 division, round half to even, clip.  Random mantissas for scale
    and input, quotients spread over and beyond the code range, exact ties, tiny quotients, and scales
    at the extremes of the fp32 range (which take the kernel's division path)."""
    rs = np.random.default_rng(5)
    M, P, seg_len = 1024, 8, 512
    K = P * seg_len
    kb = [i * seg_len for i in range(P + 1)]
    exps = [0, -7, 13, -30, 40, -110, 105, 3]
    sp = (rs.uniform(1.0, 2.0, P) * np.exp2(exps)).astype(np.float32)
    sn = (rs.uniform(1.0, 2.0, P) * np.exp2(exps[::-1])).astype(np.float32)
    qmax, qmin_abs = QRANGE[code]
    X = np.empty((M, K), np.float32)
    for p in range(P):
        blk = rs.uniform(-1.3 * qmax, 1.3 * qmax, (M, seg_len))
        blk[:, :64] = np.round(blk[:, :64]) + 0.5                      # exact ties
        blk[:, 64:96] *= 1e-3                                          # near zero
        blk[:, 96:100] *= 1e6                                          # far outside the range
        s_elem = np.where(blk >= 0, sp[p], sn[p] if dual else sp[p]).astype(np.float64)
        with np.errstate(over="ignore"):
            X[:, kb[p]:kb[p + 1]] = (blk * s_elem).astype(np.float32)
    X[~np.isfinite(X)] = 0.0
    seg = B.SegTable(kb, [0, 8])
    Xd = torch.from_numpy(X).to(DEV)
    c_pos, c_neg = B.segquant_quantize_act(Xd, seg, torch.from_numpy(sp).to(DEV),
                                           torch.from_numpy(sn).to(DEV) if dual else None, code)
    torch.cuda.synchronize()
    r_pos, r_neg = O.quantize_act(X, kb, sp, sn if dual else None, code=code, q_max=qmax, q_min_abs=qmin_abs)
    dt = np.int8 if code == "int8" else np.uint8
    assert np.array_equal(c_pos.cpu().numpy().view(dt), r_pos)
    if dual:
        assert np.array_equal(c_neg.cpu().numpy().view(dt), r_neg)


def test_int32_accumulators_at_the_largest_k_with_extreme_codes():
    """K = 131072 is the largest K the library accepts for int8 codes: with every activation code at +-127 / -128
    and every weight code at +-127 the sums reach 2.13e9, just inside int32.  The code matrices are handed to
    the GEMM directly; rows alternate sign patterns so that both extremes and cancelling sums occur."""
    M, N, K = 136, 64, 131072
    rs = np.random.default_rng(3)
    xq = np.empty((M, K), np.int8)
    xq[0::4] = 127
    xq[1::4] = -128
    xq[2::4] = np.where(np.arange(K) % 2 == 0, 127, -128).astype(np.int8)
    xq[3::4] = rs.integers(-128, 128, (M // 4, K), dtype=np.int8)
    wq = np.empty((N, K), np.int8)
    wq[0::2] = 127
    wq[1::2] = np.where(np.arange(K) % 3 == 0, -127, 127).astype(np.int8)
    ref = xq.astype(np.float64) @ wq.astype(np.float64).T                 # exact: |sum| < 2^53
    assert np.abs(ref).max() > 2.1e9 and np.abs(ref).max() < 2 ** 31
    seg = B.SegTable([0, K], [0, N])
    one = torch.ones(1, device=DEV)
    ws = B.new_workspace(DEV)
    Xd = torch.from_numpy(xq.view(np.uint8)).to(DEV)
    Wd = torch.from_numpy(wq.view(np.uint8)).to(DEV)
    Y, dump = B.segquant_seglinear_gemm(Xd, Wd, seg, "int8", one, one, None, ws, y_dtype=torch.float32, dump_acc=True)
    B.check_device_status(ws)
    torch.cuda.synchronize()
    assert np.array_equal(dump.cpu().numpy()[0].astype(np.float64), ref)
    # K one block beyond the limit is refused on the host
    with pytest.raises(B.SegquantError) as e:
        B.segquant_seglinear_gemm(torch.zeros((8, K + 128), dtype=torch.uint8, device=DEV),
                                  torch.zeros((8, K + 128), dtype=torch.uint8, device=DEV),
                                  B.SegTable([0, K + 128], [0, 8]), "int8", one, one, None, ws)
    assert e.value.status == 2


def test_fp32_input_and_student_t():
    run_parity(custom_spec("f32_in", 160, 256, 128, [0, 128, 256], [0, 128], True, "int8", x_dtype="f32",
                           x_kind="student_t4+silu"))


def test_symmetric_negative_bound_flag():
    spec = custom_spec("qmin_sym", 130, 128, 64, [0, 128], [0, 64], True, "int8")
    res = run_parity(spec, flags=B.SQ_FLAG_QMIN_SYM)
    assert res.c_neg.min() >= -127


def test_runtime_values_beyond_calibrated_range_are_clamped():
    spec = custom_spec("clamp", 256, 128, 64, [0, 128], [0, 64], True, "int8", cal_rows=4, x_kind="student_t4+gelu")
    res = run_parity(spec)
    assert (res.c_pos == 127).sum() > 1


def test_degenerate_all_nonnegative_input():
    # ReLU-like input: the negative path is all zeros and its scale degenerates to 1
    spec = custom_spec("relu_like", 140, 128, 64, [0, 128], [0, 64], True, "int8", x_kind="normal")
    data = WL.make_layer(spec)
    data.X = data.X.abs(); data.X_cal = data.X_cal.abs()
    s_pos, s_neg, s_w, Wq, (qmax, qmin_abs) = oracle_scales(data)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    g_pos, g_neg = layer.calibrate(data.X_cal)
    assert g_neg.cpu().numpy()[0] == 1.0 and np.array_equal(g_pos.cpu().numpy(), s_pos)
    Y, c_pos, c_neg, dump = layer.forward_steps(data.X.to(DEV), y_dtype=torch.float32, dump_acc=True)
    assert int(c_neg.cpu().numpy().view(np.int8).astype(np.int32).__abs__().max()) == 0
    res = O.layer_forward(to_f32_np(data.X), Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w, to_f32_np(data.bias))
    assert np.array_equal(dump.cpu().numpy()[0], res.acc_pos[0])
    assert np.all(dump.cpu().numpy()[1] == 0)
    check_fp32_output(Y, res.y64, res.y_abs, 2)


def test_host_threads_with_their_own_streams_and_workspaces():
    """Two host threads prepare and launch different layers at the same time, each on its own stream with its own
    layer object (workspace included): the library's shared state (tensor-map encoder, per-kernel attributes and
    occupancy caches) is guarded, so both get the bytes of their serial runs."""
    import threading
    specs = [custom_spec("thr_a", 700, 512, 520, [0, 256, 512], [0, 256, 520], True, "int8", seed=81),
             custom_spec("thr_b", 1300, 384, 1032, [0, 384], [0, 1032], False, "e4m3", seed=82)]
    jobs = []
    for sp in specs:
        data = WL.make_layer(sp)
        layer = SegQuantLinear(data.W, data.bias, sp.kb, sp.nb, sp.dual, sp.code, DEV)
        layer.calibrate(data.X_cal)
        Xd = data.X.to(DEV)
        jobs.append((layer, Xd, layer.forward(Xd).clone()))
    torch.cuda.synchronize()
    errors = []

    def work(layer, Xd, want):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for _ in range(40):
                    Y = layer.forward(Xd)
                st.synchronize()
                layer.check_status()
                if not torch.equal(Y, want):
                    errors.append("output differs from the serial run")
        except Exception as e:                      # surfaced in the main thread below
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=j) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


def test_repeated_calls_are_deterministic():
    spec = custom_spec("det", 300, 512, 384, [0, 256, 512], [0, 384], True, "int8")
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    y1 = layer.forward(Xd).clone()
    y2 = layer.forward(Xd).clone()
    assert torch.equal(y1, y2)


# ------------------------------------------------------------------ reduced copies of the benchmark layers

@pytest.mark.parametrize("wl,idx,M,K,N", [
    ("dit_xl2", 0, 300, 384, 768 * 3),      # 6 N-segments, ladder weights, SiLU, dual
    ("dit_xl2", 1, 300, 1536, 384),         # GELU dual, long K
    ("sd3_mmdit", 0, 333, 512, 768),        # 2 K-segments x 3 N-segments, single scale
    ("sd3_mmdit", 2, 270, 2048, 512),
    ("flux", 0, 280, 512, 1024),            # e4m3 single, heavy tails
    ("flux", 1, 280, 2048, 512),            # e4m3 dual
    ("flux", 2, 280, 512, 768 * 3),         # e4m3 dual, 6 N-segments
    ("sdxl_skip", 0, 1000, 1280, 640),      # 2 K-segments, dual, full K and N
])
def test_reduced_benchmark_layers(wl, idx, M, K, N):
    run_parity(WL.small_variant(WL.WORKLOADS[wl][idx], M, K, N))


# ------------------------------------------------------------------ full benchmark sizes, every row

@pytest.mark.parametrize("wl,idx", [("dit_xl2", 0), ("dit_xl2", 1), ("sd3_mmdit", 0), ("sd3_mmdit", 1),
                                    ("sd3_mmdit", 2), ("flux", 0), ("flux", 1), ("flux", 2), ("sdxl_skip", 0),
                                    ("sdxl_sweep", 0), ("sdxl_sweep", 7), ("sd3_heads", 0), ("sd3_heads", 1),
                                    ("sdxl_geglu", 0), ("sdxl_geglu", 1), ("sd3_qkv_768x2", 0),
                                    ("modulation_small_m", 0), ("modulation_small_m", 1), ("modulation_small_m", 2)])
def test_full_size_layers_every_row(wl, idx):
    """Every benchmark layer at its full size, in the launch configuration the benchmark times (automatic tile
    plan): codes, accumulators (dumped by the checking variant of the kernel) and both outputs (fp32 from the
    checking variant, bf16 from the production variant with TMA stores) are compared with the oracle on ALL
    rows, so every tile a persistent CTA pair walks through is covered.  For int8 layers the oracle's own
    accumulators are also cross-checked against an exact fp64 library matmul of its codes."""
    spec = WL.WORKLOADS[wl][idx]
    res = run_parity(spec)
    if spec.code == "int8":
        Wq = oracle_scales(WL.make_layer(spec, M=8))[3]
        wd = torch.from_numpy(Wq.astype(np.float64))
        for p in range(spec.P):
            ks = slice(spec.kb[p], spec.kb[p + 1])
            for codes, acc in [(res.c_pos, res.acc_pos)] + ([(res.c_neg, res.acc_neg)] if spec.dual else []):
                ref = torch.from_numpy(codes[:, ks].astype(np.float64)) @ wd[:, ks].T      # exact: |sum| < 2^53
                assert np.array_equal(ref.numpy(), acc[p].astype(np.float64))


# ------------------------------------------------------------------ host-side errors through the loaded library

def test_argument_errors_are_reported_before_launch():
    spec = custom_spec("err", 64, 128, 64, [0, 128], [0, 64], True, "int8")
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, True, "int8", DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    n0 = B.segquant_launch_count()
    bad_seg = B.SegTable([0, 64, 32, 128], [0, 64])
    with pytest.raises(B.SegquantError) as e:
        B.segquant_quantize_act(Xd, bad_seg, layer.s_pos, layer.s_neg, "int8")
    assert e.value.status == 3
    unaligned = B.SegTable([0, 40, 128], [0, 64])
    c_pos, c_neg = B.segquant_quantize_act(Xd, layer.seg, layer.s_pos, layer.s_neg, "int8")
    n1 = B.segquant_launch_count()
    sp2 = torch.ones(2, device=DEV)
    with pytest.raises(B.SegquantError) as e:
        B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, unaligned, "int8", sp2, sp2, torch.ones(2, device=DEV),
                                  None, layer.workspace)
    assert e.value.status == 4
    with pytest.raises(B.SegquantError) as e:
        B.segquant_dualscale_gemm(c_pos, c_neg, layer.Wq, layer.seg, "int8", layer.s_pos, layer.s_neg, layer.s_w,
                                  None, torch.zeros(16, dtype=torch.uint8, device=DEV))
    assert e.value.status == 8
    assert B.segquant_launch_count() == n1 and n1 == n0 + 1


# ------------------------------------------------------------------ prepared calls (plans)

@pytest.mark.parametrize("case", [
    ("plan_dual", 700, 384, 520, [0, 384], [0, 256, 520], True, "int8"),
    ("plan_single_k_segments", 333, 512, 768, [0, 256, 512], [0, 256, 512, 768], False, "int8"),
    ("plan_e4m3", 300, 256, 264, [0, 256], [0, 264], True, "e4m3"),
])
def test_planned_layer_call_equals_the_checked_call(case):
    """segquant_plan_layer + segquant_plan_run give the bytes of segquant_layer_forward; a replay after the
    input's contents changed gives the new input's output; building and running launch exactly 0 and 2 kernels;
    the run can be captured into a CUDA graph."""
    name, M, K, N, kb, nb, dual, code = case
    spec = custom_spec(name, M, K, N, kb, nb, dual, code, seed=71)
    data = WL.make_layer(spec)
    layer = SegQuantLinear(data.W, data.bias, kb, nb, dual, code, DEV)
    layer.calibrate(data.X_cal)
    Xd = data.X.to(DEV)
    Y_ref = layer.forward(Xd).clone()
    X_in = Xd.clone()
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    n0 = B.segquant_launch_count()
    plan = layer.plan(X_in, Y)
    assert B.segquant_launch_count() == n0                       # building launches nothing
    plan.run()
    assert B.segquant_launch_count() == n0 + 2
    layer.check_status()
    torch.cuda.synchronize()
    assert torch.equal(Y, Y_ref)
    X_in.copy_(torch.flip(Xd, dims=[0]) * 0.5)
    Y_ref2 = layer.forward(X_in).clone()
    Y.zero_()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream, capture_error_mode="relaxed"):
            plan.run()
    torch.cuda.current_stream().wait_stream(stream)
    graph.replay()
    layer.check_status()
    torch.cuda.synchronize()
    assert torch.equal(Y, Y_ref2) and not torch.equal(Y_ref2, Y_ref)
    res = O.layer_forward(to_f32_np(X_in.cpu()), oracle_scales(data)[3], O.SegTable(kb, nb), *oracle_scales(data)[:3],
                          to_f32_np(data.bias), code=code, q_max=QRANGE[code][0], q_min_abs=QRANGE[code][1])
    if code == "int8":
        check_bf16_output(Y, res.y64, res.y_abs, (2 if dual else 1) * (len(kb) - 1))


def test_calibration_beyond_one_grid_is_refused_without_a_launch():
    """A matrix with more columns than the reduction's grid covers (65535 blocks of 256 columns) is refused
    on the host: no kernel is launched and the partials are not touched."""
    K = 65536 * 256
    X = torch.zeros((1, K), dtype=torch.bfloat16, device=DEV)
    ws = B.new_workspace(DEV)
    ws[256:320] = 7
    n0 = B.segquant_launch_count()
    with pytest.raises(B.SegquantError) as e:
        B.segquant_calib_scales(X, B.SegTable([0, K], [0, 8]), "int8", False, True, ws)
    assert e.value.status == 2
    with pytest.raises(B.SegquantError) as e:
        B.segquant_calib_scales_static(X, B.SegTable([0, K], [0, 8]), "int8", False, True)
    assert e.value.status == 2
    torch.cuda.synchronize()
    assert B.segquant_launch_count() == n0 and bool(torch.all(ws[256:320] == 7))
    # one block of columns fewer is accepted
    X2 = X[:, :K - 256]
    s_pos, s_neg = B.segquant_calib_scales(X2, B.SegTable([0, K - 256], [0, 8]), "int8", False, True, ws)
    torch.cuda.synchronize()
    assert float(s_pos[0]) == 1.0 and float(s_neg[0]) == 1.0
