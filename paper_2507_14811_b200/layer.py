"""A quantized linear layer object over the C-ABI calls: holds the device buffers a layer needs
(weight codes, scale tables, code scratch, workspace) and issues the calls in the method's order.
All arithmetic happens inside the library's kernels."""
from __future__ import annotations

import torch

from . import binding as B


class SegQuantLinear:
    """SegLinear (per-segment scales over kb / nb) + optional DualScale W8A8 linear layer."""

    def __init__(self, W: torch.Tensor, bias, kb, nb, dual: bool, code: str = "int8", device="cuda", flags: int = 0):
        self.device = torch.device(device)
        self.N, self.K = W.shape
        self.seg = B.SegTable(kb, nb)
        self.dual, self.code, self.flags = dual, code, flags
        self.workspace = B.new_workspace(self.device)
        Wd = W.to(self.device).contiguous()
        # offline: weight scales per (K-segment, N-segment) block, then weight codes
        self.s_w, _ = B.segquant_calib_scales(Wd, self.seg, code, True, False, self.workspace)
        self.Wq = B.segquant_quantize_weight(Wd, self.seg, self.s_w, code)
        self.bias = None if bias is None else bias.to(self.device, torch.float32).contiguous()
        self.s_pos = self.s_neg = None
        self._scratch = None

    def calibrate(self, X_cal: torch.Tensor):
        """Min/max activation scales from a calibration batch (offline)."""
        Xc = X_cal.to(self.device).contiguous()
        self.s_pos, self.s_neg = B.segquant_calib_scales(Xc, self.seg, self.code, False, self.dual,
                                                         self.workspace, self.flags)
        return self.s_pos, self.s_neg

    def allow_split_tiles(self, M: int):
        """Replaces the workspace by the larger one with which the GEMM may split tiles along K for inputs of up
        to M rows (used where the layer's output has too few tiles to fill the GPU; see the C header)."""
        self.workspace = B.new_workspace(self.device, split_for=(M, self.N, self.dual))

    def scratch_for(self, M: int) -> torch.Tensor:
        need = B.layer_scratch_bytes(M, self.K, self.dual)
        if self._scratch is None or self._scratch.numel() < need:
            self._scratch = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._scratch

    def forward(self, X: torch.Tensor, Y: torch.Tensor | None = None, y_dtype=torch.bfloat16,
                x_stage=None, y_stage=None) -> torch.Tensor:
        """X [M,K] (device, or pinned host with x_stage) -> Y [M,N]."""
        M = X.shape[0]
        if Y is None:
            Y = torch.empty((M, self.N), dtype=y_dtype, device=self.device)
        return B.segquant_layer_forward(X, self.Wq, self.seg, self.code, self.s_pos, self.s_neg, self.s_w,
                                        self.bias, Y, self.scratch_for(M), self.workspace,
                                        x_stage=x_stage, y_stage=y_stage, flags=self.flags)

    def plan(self, X: torch.Tensor, Y: torch.Tensor) -> "B.LayerPlan":
        """A prepared call for these device buffers: plan.run() issues the layer's two kernels and nothing else."""
        return B.LayerPlan(X, self.Wq, self.seg, self.code, self.s_pos, self.s_neg, self.s_w, self.bias, Y,
                           self.scratch_for(X.shape[0]), self.workspace, self.flags)

    def forward_pipelined(self, X_host: torch.Tensor, Y_host: torch.Tensor, x_stage, y_stage, chunks, stream_in, stream_out):
        """Pinned-host X -> pinned-host Y with the copies overlapped with the kernels (see the C header)."""
        M = X_host.shape[0]
        return B.segquant_layer_forward_pipelined(X_host, self.Wq, self.seg, self.code, self.s_pos, self.s_neg, self.s_w,
                                                  self.bias, Y_host, self.scratch_for(M), self.workspace, x_stage, y_stage,
                                                  chunks, stream_in, stream_out, flags=self.flags)

    def forward_steps(self, X: torch.Tensor, y_dtype=torch.bfloat16, dump_acc=False):
        """The same path as separate calls, returning the intermediate codes (and raw accumulators)."""
        c_pos, c_neg = B.segquant_quantize_act(X, self.seg, self.s_pos, self.s_neg, self.code, self.flags)
        if self.dual:
            out = B.segquant_dualscale_gemm(c_pos, c_neg, self.Wq, self.seg, self.code, self.s_pos, self.s_neg,
                                            self.s_w, self.bias, self.workspace, y_dtype=y_dtype, dump_acc=dump_acc)
        else:
            out = B.segquant_seglinear_gemm(c_pos, self.Wq, self.seg, self.code, self.s_pos, self.s_w, self.bias,
                                            self.workspace, y_dtype=y_dtype, dump_acc=dump_acc)
        Y, dump = out if dump_acc else (out, None)
        return Y, c_pos, c_neg, dump

    def check_status(self):
        B.check_device_status(self.workspace)


def shard_rows(M: int, rank: int, world: int) -> tuple[int, int]:
    """Row range [r0, r1) of rank `rank` when M rows are split over `world` ranks (rows are
    independent: no exchange step).  Shards differ by at most one row; empty shards are allowed."""
    base, extra = divmod(M, world)
    r0 = rank * base + min(rank, extra)
    return r0, r0 + base + (1 if rank < extra else 0)
