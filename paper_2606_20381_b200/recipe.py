"""The UFP4 linear-layer training step (Sec. 4, Table 1) assembled from the library's calls.

One step of a linear layer Y = X W^T is: quantize X and W (RTNE) and dY (SR), each along both axes in one pass, then
the three products fwd_y = X W^T, bwd_dx = dY W and bwd_dw = dY^T X, each on the pair of variants whose 16-blocks and
RHT run along that product's reduction dimension (Sec. 2.2, last paragraph).  This module only sequences library
calls and owns the buffers; all arithmetic is in libufp4's kernels.
"""
from __future__ import annotations

import torch

from . import binding as ufp4


class _Ufp4Step:
    """The schedule shared by the dense and the MoE-grouped layer: six calls, in sequence on one stream or ordered
    only by their data dependences on three.  Subclasses provide the buffers and the calls `_quantize_x/_w/_g` and
    `_gemm(which, workspace, stream)`."""

    overlap = False

    def _init_schedule(self, need_bytes: int, device, overlap: bool):
        self.workspace = torch.empty(max(need_bytes, 16), dtype=torch.uint8, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        # overlap: the three products run on three streams (each with its own workspace), so that the operand
        # preparation of one product and the tails of the quantizer launches fill SMs another kernel leaves idle
        self.overlap = overlap
        if overlap:
            self.workspaces = [self.workspace] + [torch.empty_like(self.workspace) for _ in range(2)]
            self.side = [torch.cuda.Stream(device=device) for _ in range(2)]
            self.ev = {k: torch.cuda.Event() for k in ("start", "x", "w", "g", "dx", "dw")}

    def _qkw(self, stream):
        return dict(axis=ufp4.AXIS_BOTH, rht_block=self.rht_block, grid=self.grid, scale_fmt=self.scale_fmt,
                    seed_rht=self.seed_rht, dev_status=self.dev_status, stream=stream)

    def quantize(self, X, W, dY, stream=None, reuse_w: bool = False):
        self._quantize_x(X, stream)
        if not reuse_w:
            self._quantize_w(W, stream)
        self._quantize_g(dY, stream)

    def gemms(self, stream=None):
        for which in ("fwd_y", "bwd_dx", "bwd_dw"):
            self._gemm(which, self.workspace, stream)

    def step(self, X, W, dY, stream=None, join: bool = True, reuse_w: bool = False):
        """reuse_w: W has not changed since the last step (micro-batches of one optimizer step): its two quantized
        variants are kept and only X and dY are quantized (RTNE of the same W gives the same codes)."""
        if self.overlap:
            return self.step_overlapped(X, W, dY, stream, join, reuse_w)
        self.quantize(X, W, dY, stream, reuse_w)
        self.gemms(stream)
        return self.Y, self.dX, self.dW

    def step_overlapped(self, X, W, dY, stream=None, join: bool = True, reuse_w: bool = False):
        """The same six calls as step(), ordered only by their data dependences: X, W and fwd_y on the caller's stream,
        dY and bwd_dx on a second, bwd_dw on a third; the caller's stream joins both at the end (join=False leaves
        that to a later join() call, so that independent layers overlap too)."""
        s0 = torch.cuda.current_stream() if stream is None else stream
        s1, s2 = self.side
        ev = self.ev
        ev["start"].record(s0)
        s1.wait_event(ev["start"])
        self._quantize_g(dY, s1)
        ev["g"].record(s1)
        # separate calls here: with the three streams busy, other kernels already fill a launch's last wave, and one call for
        # X and W would make bwd_dw wait for W as well (measured: 0.893 instead of 0.882 ms per step)
        self._quantize_x(X, s0)
        ev["x"].record(s0)
        if not reuse_w:
            self._quantize_w(W, s0)
        ev["w"].record(s0)
        self._gemm("fwd_y", self.workspaces[0], s0)
        s1.wait_event(ev["w"])
        self._gemm("bwd_dx", self.workspaces[1], s1)
        ev["dx"].record(s1)
        s2.wait_event(ev["g"])
        s2.wait_event(ev["x"])
        self._gemm("bwd_dw", self.workspaces[2], s2)
        ev["dw"].record(s2)
        if join:
            self.join(s0)
        return self.Y, self.dX, self.dW

    def join(self, stream=None):
        """Make the caller's stream wait for the side streams of the last step_overlapped()."""
        if self.overlap:
            s0 = torch.cuda.current_stream() if stream is None else stream
            s0.wait_event(self.ev["dx"])
            s0.wait_event(self.ev["dw"])


class Ufp4Linear(_Ufp4Step):
    """Preallocated buffers and the 3-quantize + 3-GEMM step for one dense layer (T tokens, K in, N out)."""

    def __init__(self, tokens: int, in_features: int, out_features: int, device="cuda", grid: int = ufp4.GRID_INT4,
                 scale_fmt: int = ufp4.SCALE_FP32, path: int = ufp4.PATH_AUTO, rht_block: int = 16,
                 seed_rht: int = 1, seed_sr: int = 2, out_bf16: bool = False, overlap: bool = False,
                 tensor_scales=None):
        """tensor_scales: (ts_X, ts_W, ts_dY), the per-tensor FP32 scales of the two-level E4M3 format (floats or
        one-element device tensors); each must bound its tensor's rotated values, ts >= 4 amax / (g_max 448)."""
        T, K, N = tokens, in_features, out_features
        self.T, self.K, self.N = T, K, N
        self.grid, self.scale_fmt, self.path, self.rht_block = grid, scale_fmt, path, rht_block
        self.seed_rht, self.seed_sr = seed_rht, seed_sr
        if scale_fmt == ufp4.SCALE_E4M3_TENSOR and tensor_scales is None:
            raise ValueError("E4M3_TENSOR needs tensor_scales = (ts_X, ts_W, ts_dY)")
        tsx, tsw, tsg = tensor_scales if scale_fmt == ufp4.SCALE_E4M3_TENSOR else (None, None, None)
        a = lambda r, k, ts: ufp4.alloc_qtensor(r, k, grid, scale_fmt, device, ts)
        self.Xr, self.Xc = a(T, K, tsx), a(K, T, tsx)
        self.Wr, self.Wc = a(N, K, tsw), a(K, N, tsw)
        self.Gr, self.Gc = a(T, N, tsg), a(N, T, tsg)
        dt = torch.bfloat16 if out_bf16 else torch.float32
        self.Y = torch.empty(T, N, dtype=dt, device=device)
        self.dX = torch.empty(T, K, dtype=dt, device=device)
        self.dW = torch.empty(N, K, dtype=dt, device=device)
        need = max(ufp4.gemm_workspace_bytes(self.Xr, self.Wr, path), ufp4.gemm_workspace_bytes(self.Gr, self.Wc, path),
                   ufp4.gemm_workspace_bytes(self.Gc, self.Xc, path))
        self._init_schedule(need, device, overlap)

    def _qitem(self, which, t):
        """The keyword arguments of one of the layer's three quantizer calls (for ufp4.quantize_multi)."""
        kw = dict(x=t, axis=ufp4.AXIS_BOTH, rht_block=self.rht_block, grid=self.grid, scale_fmt=self.scale_fmt, seed_rht=self.seed_rht)
        if which == "x":
            return dict(kw, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc)
        if which == "w":
            return dict(kw, rounding=ufp4.ROUND_RTNE, out_row=self.Wr, out_col=self.Wc)
        return dict(kw, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc)

    def quantize(self, X, W, dY, stream=None, reuse_w: bool = False):
        """The layer's quantizer calls on one stream, as one ufp4_quantize_multi: X, W and dY are independent tensors, so each
        kernel's thread blocks may fill the last wave of the one before it (11 % less time than three separate calls on the
        dense layer pair)."""
        items = [self._qitem("x", X)] + ([] if reuse_w else [self._qitem("w", W)]) + [self._qitem("g", dY)]
        ufp4.quantize_multi(items, dev_status=self.dev_status, stream=stream)

    def _quantize_x(self, X, stream):
        ufp4.quantize(X, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc, **self._qkw(stream))

    def _quantize_w(self, W, stream):
        ufp4.quantize(W, rounding=ufp4.ROUND_RTNE, out_row=self.Wr, out_col=self.Wc, **self._qkw(stream))

    def _quantize_g(self, dY, stream):
        ufp4.quantize(dY, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc, **self._qkw(stream))

    def _gemm(self, which, workspace, stream):
        a, b, out, layout = {"fwd_y": (self.Xr, self.Wr, self.Y, ufp4.FWD_Y), "bwd_dx": (self.Gr, self.Wc, self.dX, ufp4.BWD_DX),
                             "bwd_dw": (self.Gc, self.Xc, self.dW, ufp4.BWD_DW)}[which]
        ufp4.gemm(a, b, out=out, layout=layout, path=self.path, workspace=workspace, dev_status=self.dev_status, stream=stream)

    @property
    def flops(self) -> int:
        return 3 * 2 * self.T * self.K * self.N

    @property
    def quantize_elements(self) -> int:
        return self.T * self.K + self.N * self.K + self.T * self.N


class Ufp4MoE(_Ufp4Step):
    """The same step for an MoE expert layer: rows of X / dY grouped by expert (offsets), weights [E][F][H]."""

    def __init__(self, offsets_host: torch.Tensor, hidden: int, ffn: int, device="cuda", grid: int = ufp4.GRID_INT4,
                 scale_fmt: int = ufp4.SCALE_FP32, path: int = ufp4.PATH_AUTO, rht_block: int = 16, seed_rht: int = 1,
                 seed_sr: int = 2, out_bf16: bool = False, counts: torch.Tensor | None = None, overlap: bool = False):
        self.counts = counts
        self.offsets_host = offsets_host.to(torch.int64).contiguous()
        self.offsets_dev = self.offsets_host.to(device)
        E, R, H, F = offsets_host.numel() - 1, int(offsets_host[-1]), hidden, ffn
        self.E, self.R, self.H, self.F = E, R, H, F
        self.grid, self.scale_fmt, self.path, self.rht_block = grid, scale_fmt, path, rht_block
        self.seed_rht, self.seed_sr = seed_rht, seed_sr
        a = lambda r, k: ufp4.alloc_qtensor(r, k, grid, scale_fmt, device)
        self.Xr, self.Xc = a(R, H), a(H, R)
        self.Wr, self.Wc = a(E * F, H), a(E * H, F)
        self.Gr, self.Gc = a(R, F), a(F, R)
        dt = torch.bfloat16 if out_bf16 else torch.float32
        self.Y = torch.empty(R, F, dtype=dt, device=device)
        self.dX = torch.empty(R, H, dtype=dt, device=device)
        self.dW = torch.empty(E * F, H, dtype=dt, device=device)
        need = max(ufp4.gemm_workspace_bytes(self.Xr, self.Wr, path), ufp4.gemm_workspace_bytes(self.Gr, self.Wc, path),
                   ufp4.gemm_workspace_bytes(self.Gc, self.Xc, path))
        self._init_schedule(need, device, overlap)

    def _quantize_x(self, X, stream):
        ufp4.quantize(X, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc, **self._qkw(stream))

    def _quantize_w(self, W, stream):
        ufp4.quantize_batched(W.view(self.E, self.F, self.H), rounding=ufp4.ROUND_RTNE, out_row=self.Wr, out_col=self.Wc,
                              **self._qkw(stream))

    def _quantize_g(self, dY, stream):
        ufp4.quantize(dY, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc, **self._qkw(stream))

    def _gemm(self, which, workspace, stream):
        a, b, out, layout, gn = {"fwd_y": (self.Xr, self.Wr, self.Y, ufp4.FWD_Y, self.F),
                                 "bwd_dx": (self.Gr, self.Wc, self.dX, ufp4.BWD_DX, self.H),
                                 "bwd_dw": (self.Gc, self.Xc, self.dW, ufp4.BWD_DW, self.F)}[which]
        ufp4.gemm_grouped(a, b, self.offsets_dev, self.offsets_host, gn, layout, out=out, path=self.path, workspace=workspace,
                          dev_status=self.dev_status, stream=stream)

    @property
    def flops(self) -> int:
        """Useful flops: unpadded routed rows only (padded rows if the counts were not given)."""
        rows = int(self.counts.sum()) if self.counts is not None else self.R
        return 3 * 2 * rows * self.H * self.F

    @property
    def quantize_elements(self) -> int:
        return self.R * self.H + self.E * self.F * self.H + self.R * self.F
