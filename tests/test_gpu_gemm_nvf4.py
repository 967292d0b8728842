"""The native-FP4 tensor-core path (UFP4_PATH_NVF4: kind::mxf4nvf4, one UE4M3 scale per 16 elements applied by the tensor
core) for operands with E4M3 block scales times a per-tensor FP32 scale.  An E2M1 tensor is the hardware's operand as it
stands; a uniform code is split into two E2M1 values (q / 2 = hi + lo) and the product taken plane by plane.  Operands are
quantized by the oracle; the oracle's FP64 product decides."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs

pytestmark = pytest.mark.gpu

GMAX = {oracle.GRID_INT4: 7.0, oracle.GRID_E1M2: 1.75, oracle.GRID_E2M1: 6.0}


def _ts(x: torch.Tensor, gmax: float) -> float:
    """A per-tensor scale that bounds the rotated values: amax / (g_max 448) with the factor 4 the 16-point RHT allows."""
    return float(np.float32(4 * x.float().abs().max().item() / (gmax * 448)))


def _quantize(x, axis, grid, **extra):
    return oracle_quantize(x, axis, rht_block=16, grid=grid, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=3,
                           tensor_scale=_ts(x, GMAX[grid]), **extra)


def test_path_selection():
    X, W = inputs.normal_bf16(64, 64, 1.0, seed=1), inputs.normal_bf16(32, 64, 0.02, seed=2)
    Au, Bu = to_device(_quantize(X, oracle.AXIS_ROW, oracle.GRID_INT4)), to_device(_quantize(W, oracle.AXIS_ROW, oracle.GRID_INT4))
    Ae, Be = to_device(_quantize(X, oracle.AXIS_ROW, oracle.GRID_E2M1)), to_device(_quantize(W, oracle.AXIS_ROW, oracle.GRID_E2M1))
    assert ufp4.gemm_path_taken(Au, Bu, ufp4.PATH_NVF4) == (ufp4.PATH_NVF4, 2) and ufp4.gemm_path_name(Au, Bu, ufp4.PATH_NVF4) == "nvf4"
    for a, b in ((Au, Bu), (Ae, Be), (Au, Be)):          # four, one, two MMAs per step: AUTO's path for plain products
        assert ufp4.gemm_path_taken(a, b, ufp4.PATH_AUTO)[0] == ufp4.PATH_NVF4
    # E2M1 tensors need no planes: only the scale units
    assert ufp4.gemm_workspace_bytes(Ae, Be, ufp4.PATH_NVF4) < ufp4.gemm_workspace_bytes(Au, Bu, ufp4.PATH_NVF4)
    P = to_device(oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=3))
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm(Au, P, path=ufp4.PATH_NVF4)
    assert e.value.status == -5


@pytest.mark.parametrize("grids", [(oracle.GRID_INT4, oracle.GRID_INT4), (oracle.GRID_E1M2, oracle.GRID_E2M1),
                                   (oracle.GRID_E2M1, oracle.GRID_INT4), (oracle.GRID_E2M1, oracle.GRID_E2M1)])
@pytest.mark.parametrize("shape", [(256, 256, 256), (200, 72, 176), (1, 1, 16), (130, 260, 144), (384, 520, 1040),
                                   (1024, 1536, 2048), (640, 256, 8192), (2304, 2560, 160)])
def test_shapes_and_grids(shape, grids):
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=21 + M)
    W = inputs.normal_bf16(N, K, 0.02, seed=22 + N)
    A = _quantize(X, oracle.AXIS_ROW, grids[0])
    B = _quantize(W, oracle.AXIS_ROW, grids[1])
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_NVF4, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, f"nvf4 path {shape} grids {grids}")
    out = torch.full((M, (N + 15) // 8 * 8), 7.0, dtype=torch.bfloat16, device="cuda")
    ufp4.gemm(to_device(A), to_device(B), out=out[:, :N], path=ufp4.PATH_NVF4)
    assert_gemm_close(out[:, :N].float().cpu().numpy(), ref, S, "bf16 out", bf16_out=True)
    assert torch.all(out[:, N:] == 7.0)


def test_every_uniform_code_splits_into_two_e2m1_values():
    """All 15 codes (and INT4's -8, which the quantizer never writes) against all of them, with unit scales: the product of
    the planes is the integer product."""
    K = 256
    qa = np.zeros((16, K), dtype=np.int64)
    qb = np.zeros((16, K), dtype=np.int64)
    for i in range(16):
        qa[i, :] = i - 8
        qb[i, :] = np.resize(np.arange(-8, 8), K)
    def qt(q):
        n = (q & 0xF).astype(np.uint8)
        codes = torch.from_numpy((n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)).cuda()
        scales = torch.full((q.shape[0], K // 16), 0x38, dtype=torch.uint8, device="cuda")      # E4M3 1.0
        return ufp4.QTensor(codes, scales, ufp4.GRID_INT4, ufp4.SCALE_E4M3_TENSOR, K, tensor_scale=torch.ones(1, device="cuda"))
    got = ufp4.gemm(qt(qa), qt(qb), path=ufp4.PATH_NVF4).cpu().numpy()
    assert np.array_equal(got, (qa @ qb.T).astype(np.float32))


def test_tiny_layer_all_three_products():
    X, W, dY = inputs.tiny_layer(0)
    for grid in (oracle.GRID_INT4, oracle.GRID_E2M1):
        q = lambda t, ax, **kw: _quantize(t, ax, grid, **kw)
        sr = dict(rounding=oracle.ROUND_SR, seed_sr=2)
        cases = {"fwd_y": (q(X, oracle.AXIS_ROW), q(W, oracle.AXIS_ROW), ufp4.FWD_Y),
                 "bwd_dx": (q(dY, oracle.AXIS_ROW, **sr), q(W, oracle.AXIS_COL), ufp4.BWD_DX),
                 "bwd_dw": (q(dY, oracle.AXIS_COL, **sr), q(X, oracle.AXIS_COL), ufp4.BWD_DW)}
        for name, (A, B, layout) in cases.items():
            ref, S = oracle.gemm(A, B)
            got = ufp4.gemm(to_device(A), to_device(B), layout=layout, path=ufp4.PATH_NVF4)
            assert_gemm_close(got.cpu().numpy(), ref, S, f"{name} grid {grid}")


def test_extreme_block_scales_need_no_window():
    """Blocks 2^40 apart inside one row, E4M3 scales from the subnormal bytes up to the saturated 448: the hardware applies
    each block's own scale, nothing is flushed."""
    M, N, K = 128, 64, 256
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(9))
    x[:, :16] *= 2.0 ** 20
    x[:, 16:32] *= 2.0 ** -20
    X = x.to(torch.bfloat16)
    W = inputs.normal_bf16(N, K, 1.0, seed=10)
    kw = dict(rht_block=0, grid=oracle.GRID_INT4, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=3)
    A = oracle_quantize(X, oracle.AXIS_ROW, tensor_scale=2.0 ** -14, **kw)
    B = oracle_quantize(W, oracle.AXIS_ROW, tensor_scale=_ts(W, 7), **kw)
    assert A.scales.max() == 0x7E and 0 < A.scales[A.scales > 0].min() < 0x08      # 448 next to subnormal E4M3 scales
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_NVF4, dev_status=status)
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, "extreme block scales")


def test_grouped_products_are_refused():
    X, W = inputs.normal_bf16(256, 64, 1.0, seed=1), inputs.normal_bf16(2 * 48, 64, 0.02, seed=2)
    A, B = to_device(_quantize(X, oracle.AXIS_ROW, oracle.GRID_INT4)), to_device(_quantize(W, oracle.AXIS_ROW, oracle.GRID_INT4))
    off = torch.tensor([0, 128, 256], dtype=torch.int64)
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_grouped(A, B, off.cuda(), off, 48, ufp4.FWD_Y, path=ufp4.PATH_NVF4)
    assert e.value.status == -5


@pytest.mark.parametrize("grid", [oracle.GRID_INT4, oracle.GRID_E1M2, oracle.GRID_E2M1])
def test_tiny_layer_step_with_two_level_scales(grid):
    """The tiny single-layer check in its two-level scale format (E4M3 per block, FP32 per tensor), through the recipe class:
    the six quantized tensors bit-equal to the oracle's, the three products (AUTO: the FP4 path) within the bound."""
    from helpers import assert_qtensor_equal
    from paper_2606_20381_b200.recipe import Ufp4Linear
    X, W, dY = inputs.tiny_layer(0)
    ts = tuple(_ts(t, GMAX[grid]) for t in (X, W, dY))
    step = Ufp4Linear(X.shape[0], X.shape[1], W.shape[0], grid=grid, scale_fmt=ufp4.SCALE_E4M3_TENSOR, tensor_scales=ts)
    Y, dX, dW = step.step(X.cuda(), W.cuda(), dY.cuda())
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == 0
    kw = dict(rht_block=16, grid=grid, scale_fmt=oracle.SCALE_E4M3_TENSOR, seed_rht=1)
    sr = dict(rounding=oracle.ROUND_SR, seed_sr=2)
    ref = {"Xr": oracle_quantize(X, oracle.AXIS_ROW, tensor_scale=ts[0], **kw), "Xc": oracle_quantize(X, oracle.AXIS_COL, tensor_scale=ts[0], **kw),
           "Wr": oracle_quantize(W, oracle.AXIS_ROW, tensor_scale=ts[1], **kw), "Wc": oracle_quantize(W, oracle.AXIS_COL, tensor_scale=ts[1], **kw),
           "Gr": oracle_quantize(dY, oracle.AXIS_ROW, tensor_scale=ts[2], **kw, **sr),
           "Gc": oracle_quantize(dY, oracle.AXIS_COL, tensor_scale=ts[2], **kw, **sr)}
    for key in ref:
        assert_qtensor_equal(getattr(step, key), ref[key], f"{key} grid {grid}")
    assert ufp4.gemm_path_name(step.Xr, step.Wr) == "nvf4"
    for out, a, b, name in ((Y, "Xr", "Wr", "fwd_y"), (dX, "Gr", "Wc", "bwd_dx"), (dW, "Gc", "Xc", "bwd_dw")):
        c, s = oracle.gemm(ref[a], ref[b])
        assert_gemm_close(out.cpu().numpy(), c, s, f"{name} grid {grid}")
