"""The UFP4 linear-layer training step (Sec. 4, Table 1) assembled from the library's calls.

One step of a linear layer Y = X W^T is: quantize X and W (RTNE) and dY (SR), each along both axes in one pass, then
the three products fwd_y = X W^T, bwd_dx = dY W and bwd_dw = dY^T X, each on the pair of variants whose 16-blocks and
RHT run along that product's reduction dimension (Sec. 2.2, last paragraph).  This module only sequences library
calls and owns the buffers; all arithmetic is in libufp4's kernels.
"""
from __future__ import annotations

import torch

from . import binding as ufp4


class Ufp4Linear:
    """Preallocated buffers and the 3-quantize + 3-GEMM step for one dense layer (T tokens, K in, N out)."""

    def __init__(self, tokens: int, in_features: int, out_features: int, device="cuda", grid: int = ufp4.GRID_INT4,
                 scale_fmt: int = ufp4.SCALE_FP32, path: int = ufp4.PATH_AUTO, rht_block: int = 16,
                 seed_rht: int = 1, seed_sr: int = 2, out_bf16: bool = False, overlap: bool = False):
        T, K, N = tokens, in_features, out_features
        self.T, self.K, self.N = T, K, N
        self.grid, self.scale_fmt, self.path, self.rht_block = grid, scale_fmt, path, rht_block
        self.seed_rht, self.seed_sr = seed_rht, seed_sr
        a = lambda r, k: ufp4.alloc_qtensor(r, k, grid, scale_fmt, device)
        self.Xr, self.Xc = a(T, K), a(K, T)
        self.Wr, self.Wc = a(N, K), a(K, N)
        self.Gr, self.Gc = a(T, N), a(N, T)
        dt = torch.bfloat16 if out_bf16 else torch.float32
        self.Y = torch.empty(T, N, dtype=dt, device=device)
        self.dX = torch.empty(T, K, dtype=dt, device=device)
        self.dW = torch.empty(N, K, dtype=dt, device=device)
        need = max(ufp4.gemm_workspace_bytes(self.Xr, self.Wr, path), ufp4.gemm_workspace_bytes(self.Gr, self.Wc, path),
                   ufp4.gemm_workspace_bytes(self.Gc, self.Xc, path))
        self.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        # overlap: the three products run on three streams (each with its own workspace), so that the operand
        # preparation of one product and the tails of the quantizer launches fill SMs another kernel leaves idle
        self.overlap = overlap
        if overlap:
            self.workspaces = [self.workspace] + [torch.empty_like(self.workspace) for _ in range(2)]
            self.side = [torch.cuda.Stream(device=device) for _ in range(2)]
            self.ev = {k: torch.cuda.Event() for k in ("start", "x", "w", "g", "dx", "dw")}

    # number of kernel launches one call makes (for the benchmark's launch count)
    launches_quantize = 3

    def quantize(self, X, W, dY, stream=None):
        kw = dict(axis=ufp4.AXIS_BOTH, rht_block=self.rht_block, grid=self.grid, scale_fmt=self.scale_fmt,
                  seed_rht=self.seed_rht, dev_status=self.dev_status, stream=stream)
        ufp4.quantize(X, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc, **kw)
        ufp4.quantize(W, rounding=ufp4.ROUND_RTNE, out_row=self.Wr, out_col=self.Wc, **kw)
        ufp4.quantize(dY, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc, **kw)

    def gemms(self, stream=None):
        kw = dict(path=self.path, workspace=self.workspace, dev_status=self.dev_status, stream=stream)
        ufp4.gemm(self.Xr, self.Wr, out=self.Y, layout=ufp4.FWD_Y, **kw)
        ufp4.gemm(self.Gr, self.Wc, out=self.dX, layout=ufp4.BWD_DX, **kw)
        ufp4.gemm(self.Gc, self.Xc, out=self.dW, layout=ufp4.BWD_DW, **kw)

    def step(self, X, W, dY, stream=None, join: bool = True):
        if self.overlap:
            return self.step_overlapped(X, W, dY, stream, join)
        self.quantize(X, W, dY, stream)
        self.gemms(stream)
        return self.Y, self.dX, self.dW

    def step_overlapped(self, X, W, dY, stream=None, join: bool = True):
        """The same six calls as step(), ordered only by their data dependences: X, W and fwd_y on the caller's stream,
        dY and bwd_dx on a second, bwd_dw on a third; the caller's stream joins both at the end (join=False leaves
        that to a later join() call, so that independent layers overlap too)."""
        s0 = torch.cuda.current_stream() if stream is None else stream
        s1, s2 = self.side
        ev = self.ev
        qkw = dict(axis=ufp4.AXIS_BOTH, rht_block=self.rht_block, grid=self.grid, scale_fmt=self.scale_fmt,
                   seed_rht=self.seed_rht, dev_status=self.dev_status)
        gkw = dict(path=self.path, dev_status=self.dev_status)
        ev["start"].record(s0)
        s1.wait_event(ev["start"])
        ufp4.quantize(dY, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc, stream=s1, **qkw)
        ev["g"].record(s1)
        ufp4.quantize(X, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc, stream=s0, **qkw)
        ev["x"].record(s0)
        ufp4.quantize(W, rounding=ufp4.ROUND_RTNE, out_row=self.Wr, out_col=self.Wc, stream=s0, **qkw)
        ev["w"].record(s0)
        ufp4.gemm(self.Xr, self.Wr, out=self.Y, layout=ufp4.FWD_Y, workspace=self.workspaces[0], stream=s0, **gkw)
        s1.wait_event(ev["w"])
        ufp4.gemm(self.Gr, self.Wc, out=self.dX, layout=ufp4.BWD_DX, workspace=self.workspaces[1], stream=s1, **gkw)
        ev["dx"].record(s1)
        s2.wait_event(ev["g"])
        s2.wait_event(ev["x"])
        ufp4.gemm(self.Gc, self.Xc, out=self.dW, layout=ufp4.BWD_DW, workspace=self.workspaces[2], stream=s2, **gkw)
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

    @property
    def flops(self) -> int:
        return 3 * 2 * self.T * self.K * self.N

    @property
    def quantize_elements(self) -> int:
        return self.T * self.K + self.N * self.K + self.T * self.N


class Ufp4MoE:
    """The same step for an MoE expert layer: rows of X / dY grouped by expert (offsets), weights [E][F][H]."""

    def __init__(self, offsets_host: torch.Tensor, hidden: int, ffn: int, device="cuda", grid: int = ufp4.GRID_INT4,
                 scale_fmt: int = ufp4.SCALE_FP32, path: int = ufp4.PATH_AUTO, rht_block: int = 16, seed_rht: int = 1,
                 seed_sr: int = 2, out_bf16: bool = False, counts: torch.Tensor | None = None):
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
        self.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)

    def quantize(self, X, W, dY, stream=None):
        kw = dict(axis=ufp4.AXIS_BOTH, rht_block=self.rht_block, grid=self.grid, scale_fmt=self.scale_fmt,
                  seed_rht=self.seed_rht, dev_status=self.dev_status, stream=stream)
        ufp4.quantize(X, rounding=ufp4.ROUND_RTNE, out_row=self.Xr, out_col=self.Xc, **kw)
        ufp4.quantize_batched(W.view(self.E, self.F, self.H), rounding=ufp4.ROUND_RTNE, out_row=self.Wr,
                              out_col=self.Wc, **kw)
        ufp4.quantize(dY, rounding=ufp4.ROUND_SR, seed_sr=self.seed_sr, out_row=self.Gr, out_col=self.Gc, **kw)

    def gemms(self, stream=None):
        kw = dict(path=self.path, workspace=self.workspace, dev_status=self.dev_status, stream=stream)
        ufp4.gemm_grouped(self.Xr, self.Wr, self.offsets_dev, self.offsets_host, self.F, ufp4.FWD_Y, out=self.Y, **kw)
        ufp4.gemm_grouped(self.Gr, self.Wc, self.offsets_dev, self.offsets_host, self.H, ufp4.BWD_DX, out=self.dX, **kw)
        ufp4.gemm_grouped(self.Gc, self.Xc, self.offsets_dev, self.offsets_host, self.F, ufp4.BWD_DW, out=self.dW, **kw)

    overlap = False     # the grouped step runs its calls in sequence on one stream

    def step(self, X, W, dY, stream=None, join: bool = True):
        self.quantize(X, W, dY, stream)
        self.gemms(stream)
        return self.Y, self.dX, self.dW

    def join(self, stream=None):
        pass

    @property
    def flops(self) -> int:
        """Useful flops: unpadded routed rows only (padded rows if the counts were not given)."""
        rows = int(self.counts.sum()) if self.counts is not None else self.R
        return 3 * 2 * rows * self.H * self.F

    @property
    def quantize_elements(self) -> int:
        return self.R * self.H + self.E * self.F * self.H + self.R * self.F
