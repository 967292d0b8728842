"""The one-piece FP16 tensor-core path (UFP4_PATH_FP16) for operands with E4M3 block scales times a per-tensor FP32 scale:
level x E4M3 value is exact in FP16, so one MMA per K step gives the product within the usual bound, without a row
reference and without an exponent window.  Operands are quantized by the oracle; the oracle's FP64 product decides."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs
from test_gpu_gemm import grouped_reference

pytestmark = pytest.mark.gpu


def _ts(x: torch.Tensor, gmax: float) -> float:
    """A per-tensor scale that bounds the rotated values: amax / (g_max 448) with the factor 4 the 16-point RHT allows."""
    return float(np.float32(4 * x.float().abs().max().item() / (gmax * 448)))


def _quantize(x, axis, grid, gmax, **extra):
    return oracle_quantize(x, axis, rht_block=16, grid=grid, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=3,
                           tensor_scale=_ts(x, gmax), **extra)


def test_the_fp16_path_takes_e4m3_tensor_scales_only():
    X, W = inputs.normal_bf16(64, 64, 1.0, seed=1), inputs.normal_bf16(32, 64, 0.02, seed=2)
    A, B = to_device(_quantize(X, oracle.AXIS_ROW, oracle.GRID_INT4, 7)), to_device(_quantize(W, oracle.AXIS_ROW, oracle.GRID_INT4, 7))
    assert ufp4.gemm_path_taken(A, B, ufp4.PATH_FP16) == (ufp4.PATH_FP16, 2)
    assert ufp4.gemm_path_name(A, B, ufp4.PATH_FP16) == "fp16"
    assert ufp4.gemm_workspace_bytes(A, B, ufp4.PATH_FP16) < ufp4.gemm_workspace_bytes(A, B, ufp4.PATH_SPLIT)
    P = to_device(oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=3))
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm(A, P, path=ufp4.PATH_FP16)
    assert e.value.status == -5
    assert ufp4.gemm_path_taken(A, P, ufp4.PATH_AUTO)[0] == ufp4.PATH_SPLIT


@pytest.mark.parametrize("grids", [(oracle.GRID_INT4, oracle.GRID_INT4), (oracle.GRID_E1M2, oracle.GRID_E2M1)])
@pytest.mark.parametrize("shape", [(256, 256, 256), (200, 72, 176), (1, 1, 16), (130, 260, 144), (384, 520, 1040),
                                   (1024, 1536, 2048), (640, 256, 8192)])
def test_shapes_and_grids(shape, grids):
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=21 + M)
    W = inputs.normal_bf16(N, K, 0.02, seed=22 + N)
    gmax = {oracle.GRID_INT4: 7.0, oracle.GRID_E1M2: 1.75, oracle.GRID_E2M1: 6.0}
    A = _quantize(X, oracle.AXIS_ROW, grids[0], gmax[grids[0]])
    B = _quantize(W, oracle.AXIS_ROW, grids[1], gmax[grids[1]])
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_FP16, dev_status=status)
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, f"fp16 path {shape} grids {grids}")
    # the same through AUTO, into a padded BF16 buffer
    out = torch.full((M, (N + 15) // 8 * 8), 7.0, dtype=torch.bfloat16, device="cuda")
    ufp4.gemm(to_device(A), to_device(B), out=out[:, :N])
    assert_gemm_close(out[:, :N].float().cpu().numpy(), ref, S, "bf16 out", bf16_out=True)
    assert torch.all(out[:, N:] == 7.0)
    # and it agrees with the two-piece path on the same operands
    two = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_SPLIT)
    assert_gemm_close(two.cpu().numpy(), ref, S, "two-piece path on the same operands")


def test_tiny_layer_all_three_products():
    X, W, dY = inputs.tiny_layer(0)
    q = lambda t, ax, **kw: _quantize(t, ax, oracle.GRID_INT4, 7, **kw)
    sr = dict(rounding=oracle.ROUND_SR, seed_sr=2)
    cases = {"fwd_y": (q(X, oracle.AXIS_ROW), q(W, oracle.AXIS_ROW), ufp4.FWD_Y),
             "bwd_dx": (q(dY, oracle.AXIS_ROW, **sr), q(W, oracle.AXIS_COL), ufp4.BWD_DX),
             "bwd_dw": (q(dY, oracle.AXIS_COL, **sr), q(X, oracle.AXIS_COL), ufp4.BWD_DW)}
    for name, (A, B, layout) in cases.items():
        ref, S = oracle.gemm(A, B)
        got = ufp4.gemm(to_device(A), to_device(B), layout=layout, path=ufp4.PATH_FP16)
        assert_gemm_close(got.cpu().numpy(), ref, S, name)


def test_extreme_block_scales_need_no_window():
    """Blocks 2^40 apart inside one row: every E4M3 block value fits FP16 next to every other, nothing is flushed."""
    M, N, K = 128, 64, 256
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(9))
    x[:, :16] *= 2.0 ** 20
    x[:, 16:32] *= 2.0 ** -20
    X = x.to(torch.bfloat16)
    W = inputs.normal_bf16(N, K, 1.0, seed=10)
    kw = dict(rht_block=0, grid=oracle.GRID_INT4, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=3)
    # a tensor scale small enough that the tiny blocks keep non-zero E4M3 scales while the large ones saturate at 448
    A = oracle_quantize(X, oracle.AXIS_ROW, tensor_scale=2.0 ** -14, **kw)
    B = oracle_quantize(W, oracle.AXIS_ROW, tensor_scale=_ts(W, 7), **kw)
    assert A.scales.max() == 0x7E and 0 < A.scales[A.scales > 0].min() < 0x20     # 448 saturated next to tiny E4M3 scales
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_FP16, dev_status=status)
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, "extreme block scales")


def test_grouped_products():
    """Four experts, one of them empty, rows and reduction grouped."""
    offsets = [0, 128, 128, 384, 512]
    E, H, F = 4, 96, 80
    X = inputs.heavy_tailed_activations(512, H, seed=31)
    W = inputs.normal_bf16(E * F, H, 0.02, seed=32)
    dY = inputs.normal_bf16(512, F, 1e-4, seed=33)
    tsw = _ts(W, 7)
    kw = dict(rht_block=16, grid=oracle.GRID_INT4, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=1)
    Xr, Xc = (oracle_quantize(X, a, tensor_scale=_ts(X, 7), **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Gr, Gc = (oracle_quantize(dY, a, rounding=oracle.ROUND_SR, seed_sr=2, tensor_scale=_ts(dY, 7), **kw)
              for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Wr = oracle_quantize(W, oracle.AXIS_ROW, tensor_scale=tsw, **kw)
    parts = [oracle_quantize(W[e * F:(e + 1) * F], oracle.AXIS_COL, tensor_scale=tsw, **kw) for e in range(E)]
    Wc = oracle.QTensor(np.concatenate([p.codes for p in parts]), np.concatenate([p.scales for p in parts]),
                        oracle.GRID_INT4, oracle.SCALE_E4M3_TENSOR, parts[0].tensor_scale)
    off_h = torch.tensor(offsets, dtype=torch.int64)
    off_d = off_h.cuda()
    for name, (A, B, layout, gn) in {"fwd_y": (Xr, Wr, ufp4.FWD_Y, F), "bwd_dx": (Gr, Wc, ufp4.BWD_DX, H),
                                     "bwd_dw": (Gc, Xc, ufp4.BWD_DW, F)}.items():
        ref, S = grouped_reference(A, B, offsets, gn, layout)
        got = ufp4.gemm_grouped(to_device(A), to_device(B), off_d, off_h, gn, layout, path=ufp4.PATH_FP16).cpu().numpy()
        assert_gemm_close(got, ref, S, f"grouped {name}")
