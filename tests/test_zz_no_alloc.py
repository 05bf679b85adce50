"""The allocation-free calibration entry point against the ordinary one.

segquant_calib_scales_static exists for callers that may not allocate device memory (a plugin that
only receives tensors, a process whose device memory belongs to someone else's pool, a no-allocation-
after-start-up policy): it keeps its reduction partials in an array inside the library instead of a
caller-provided workspace.  It has to return bit-identical scales, and because every call shares that
array, a second call right after the first (on other data, with other segment counts) must not see
anything the first one left behind.  This file is named to be collected last, so a run that stops at
the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2507_14811_b200 import binding as B
from paper_2507_14811_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _spec(name, M, K, N, kb, nb, x_kind, seed, x_dtype="bf16", x_seg_std=None):
    return WL.LayerSpec(name=name, M=M, K=K, N=N, kb=kb, nb=nb, dual=True, code="int8", x_dtype=x_dtype,
                        x_kind=x_kind, w_kind="segment_ladder", seed=seed, cal_rows=96, x_seg_std=x_seg_std or [])


def _compare(spec, code):
    data = WL.make_layer(spec)
    seg = B.SegTable(spec.kb, spec.nb)
    ws = B.new_workspace(DEV)
    Xc = data.X_cal.to(DEV).contiguous()
    Wd = data.W.to(DEV).contiguous()
    # outputs are allocated up front: the call under test itself allocates nothing
    out = {k: torch.full((n,), -1.0, dtype=torch.float32, device=DEV)
           for k, n in (("pos", seg.P), ("neg", seg.P), ("one", seg.P), ("w", seg.P * seg.Q))}
    torch.cuda.synchronize()
    for dual in (True, False):
        ref_pos, ref_neg = B.segquant_calib_scales(Xc, seg, code, False, dual, ws)
        got_pos, got_neg = B.segquant_calib_scales_static(Xc, seg, code, False, dual,
                                                          s_pos=out["pos"] if dual else out["one"],
                                                          s_neg=out["neg"] if dual else None)
        torch.cuda.synchronize()
        assert np.array_equal(got_pos.cpu().numpy(), ref_pos.cpu().numpy())
        if dual:
            assert np.array_equal(got_neg.cpu().numpy(), ref_neg.cpu().numpy())
    ref_w, _ = B.segquant_calib_scales(Wd, seg, code, True, False, ws)
    got_w, _ = B.segquant_calib_scales_static(Wd, seg, code, True, False, s_pos=out["w"])
    torch.cuda.synchronize()
    assert np.array_equal(got_w.cpu().numpy(), ref_w.cpu().numpy())
    assert float(got_w.min()) > 0.0


def test_static_calibration_matches_workspace_calibration_twice_in_a_row():
    # first call: many blocks, large values; second call: fewer blocks, much smaller values, so stale
    # partials of the first call would show up as scales that are too large
    _compare(_spec("first", 64, 512, 384, [0, 128, 256, 512], [0, 64, 128, 192, 256, 320, 384],
                   "student_t4+gelu", 11, x_seg_std=[4.0, 9.0, 2.0]), "int8")
    _compare(_spec("second", 64, 256, 128, [0, 256], [0, 128], "normal+silu", 12, x_dtype="f32",
                   x_seg_std=[0.05]), "e4m3")


def test_static_calibration_refuses_more_blocks_than_it_holds():
    # 33 K-segments x 32 N-segments = 1056 weight blocks: a valid table for the workspace version, one more
    # row of blocks than the built-in array holds; refused on the host, before any launch
    n0 = B.segquant_launch_count()
    P, Q = 33, 32
    K, N = 32 * P, 8 * Q
    X = torch.zeros((N, K), dtype=torch.float32, device=DEV)
    seg = B.SegTable(list(range(0, K + 1, 32)), list(range(0, N + 1, 8)))
    with pytest.raises(B.SegquantError) as e:
        B.segquant_calib_scales_static(X, seg, "int8", True, False)
    assert e.value.status == 5
    assert B.segquant_launch_count() == n0
    s_w, _ = B.segquant_calib_scales(X, seg, "int8", True, False, B.new_workspace(DEV))
    torch.cuda.synchronize()
    assert s_w.numel() == P * Q and bool(torch.all(s_w == 1.0))       # all-zero blocks: unit scale


def test_static_calibration_allocates_nothing_and_takes_exactly_its_limit():
    """The reason this entry point exists is that its caller cannot allocate: after one warm-up call (which looks
    up the built-in array's address) a call leaves torch's allocator counters and the device's free memory
    untouched.  And the limit is exact: 32 x 32 = 1024 weight blocks are accepted and give the workspace
    version's scales; an activation table with more K- than N-segments (P > Q) goes through the same array."""
    rs = np.random.default_rng(21)
    P, Q = 32, 32
    K, N = 32 * P, 8 * Q
    W = torch.from_numpy(rs.normal(0, 0.02, (N, K)).astype(np.float32)).to(DEV)
    W *= torch.linspace(0.5, 20.0, N, device=DEV)[:, None]
    seg = B.SegTable(list(range(0, K + 1, 32)), list(range(0, N + 1, 8)))
    out = torch.empty(P * Q, dtype=torch.float32, device=DEV)
    B.segquant_calib_scales_static(W, seg, "int8", True, False, s_pos=out)            # warm-up call
    torch.cuda.synchronize()
    # cumulative allocation and segment counts of torch's allocator, its reserved bytes, the device's free bytes
    snap = lambda: (torch.cuda.memory_stats()["allocation.all.allocated"], torch.cuda.memory_stats()["segment.all.allocated"],
                    torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    before = snap()
    B.segquant_calib_scales_static(W, seg, "int8", True, False, s_pos=out)
    torch.cuda.synchronize()
    assert snap() == before
    ref, _ = B.segquant_calib_scales(W, seg, "int8", True, False, B.new_workspace(DEV))
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), ref.cpu().numpy()) and len(np.unique(out.cpu().numpy())) > 100

    # activations: 40 K-segments, 1 N-segment (P > Q)
    Pa = 40
    X = torch.from_numpy(rs.normal(0, 1, (50, 32 * Pa)).astype(np.float32)).to(DEV)
    X *= torch.linspace(0.1, 30.0, 32 * Pa, device=DEV)[None, :]
    seg_a = B.SegTable(list(range(0, 32 * Pa + 1, 32)), [0, 8])
    sp, sn = torch.empty(Pa, device=DEV), torch.empty(Pa, device=DEV)
    B.segquant_calib_scales_static(X, seg_a, "int8", False, True, s_pos=sp, s_neg=sn)
    rp, rn = B.segquant_calib_scales(X, seg_a, "int8", False, True, B.new_workspace(DEV))
    torch.cuda.synchronize()
    assert torch.equal(sp, rp) and torch.equal(sn, rn)
