"""The hardware-block-scaled tensor-core path (UFP4_PATH_MX: kind::mxf8f6f4, one UE8M0 scale per 32 elements applied by
the tensor core): parity with the oracle's FP64 product on oracle-quantized operands, for 1 x 32 E8M0 tensors (exact by
construction: nothing is ever flushed, whatever the spread of a row's scales) and for 1 x 16 POW2 tensors (the gap inside a
32-group is folded into the elements)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs
from test_gpu_gemm import grouped_reference

pytestmark = pytest.mark.gpu


def test_mx_is_taken_on_request_and_auto_keeps_the_folded_path():
    X, W = inputs.normal_bf16(64, 64, 1.0, seed=1), inputs.normal_bf16(32, 64, 0.02, seed=2)
    kw = dict(rht_block=16, seed_rht=3)
    A32 = to_device(oracle_quantize(X, oracle.AXIS_ROW, scale_fmt=oracle.SCALE_E8M0_B32, **kw))
    B32 = to_device(oracle_quantize(W, oracle.AXIS_ROW, scale_fmt=oracle.SCALE_E8M0_B32, **kw))
    B16 = to_device(oracle_quantize(W, oracle.AXIS_ROW, scale_fmt=oracle.SCALE_POW2, **kw))
    BF = to_device(oracle_quantize(W, oracle.AXIS_ROW, scale_fmt=oracle.SCALE_FP32, **kw))
    assert ufp4.gemm_path_taken(A32, B32, ufp4.PATH_MX) == (ufp4.PATH_MX, 2) and ufp4.gemm_path_name(A32, B32, ufp4.PATH_MX) == "mx"
    assert ufp4.gemm_path_taken(A32, B32, ufp4.PATH_AUTO)[0] == ufp4.PATH_TENSOR
    assert ufp4.gemm_path_taken(A32, B16, ufp4.PATH_AUTO)[0] == ufp4.PATH_TENSOR
    assert ufp4.gemm_path_taken(A32, B16, ufp4.PATH_MX)[0] == ufp4.PATH_MX
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm(A32, BF, path=ufp4.PATH_MX)
    assert e.value.status == -5


@pytest.mark.parametrize("fmt", [oracle.SCALE_E8M0_B32, oracle.SCALE_POW2])
@pytest.mark.parametrize("grids", [(oracle.GRID_INT4, oracle.GRID_INT4), (oracle.GRID_E1M2, oracle.GRID_E2M1)])
@pytest.mark.parametrize("shape", [(256, 256, 256), (128, 256, 128), (200, 72, 160), (1, 1, 32), (130, 260, 192),
                                   (384, 520, 1056), (1024, 1536, 2048), (640, 300, 8192),
                                   (2304, 2560, 160)])                     # more tiles than resident CTA pairs
def test_shapes_grids_and_scale_formats(shape, grids, fmt):
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=21 + M)
    W = inputs.normal_bf16(N, K, 0.02, seed=22 + N)
    kw = dict(rht_block=16, scale_fmt=fmt, seed_rht=5)
    A = oracle_quantize(X, oracle.AXIS_ROW, grid=grids[0], **kw)
    B = oracle_quantize(W, oracle.AXIS_ROW, grid=grids[1], **kw)
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_MX, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, f"mx {shape} grids {grids} fmt {fmt}")
    out = torch.full((M, (N + 15) // 8 * 8), 7.0, dtype=torch.bfloat16, device="cuda")
    ufp4.gemm(to_device(A), to_device(B), out=out[:, :N], path=ufp4.PATH_MX)
    assert_gemm_close(out[:, :N].float().cpu().numpy(), ref, S, "bf16 out", bf16_out=True)
    assert torch.all(out[:, N:] == 7.0)


def test_k_multiple_of_16_only_for_pow2_scales():
    M, N, K = 192, 136, 176                       # K / 16 odd: the last 32-group holds one block
    X, W = inputs.heavy_tailed_activations(M, K, seed=3), inputs.normal_bf16(N, K, 0.02, seed=4)
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=5)
    A, B = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)
    ref, S = oracle.gemm(A, B)
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_MX)
    assert_gemm_close(got.cpu().numpy(), ref, S, "K = 176")


def test_a_row_whose_scales_spread_over_2_to_the_30_is_exact_here_and_flagged_on_the_folded_path():
    """One row holds 32-groups 2^30 apart.  With one hardware scale per group every group is exact; the folded 8-bit path,
    whose elements carry their exponent relative to the row's largest block, has to flush the small ones and says so."""
    M, N, K = 128, 64, 256
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(9))
    x[:, :32] *= 2.0 ** 15
    x[:, 32:64] *= 2.0 ** -15
    X = x.to(torch.bfloat16)
    W = inputs.normal_bf16(N, K, 1.0, seed=10)
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_E8M0_B32, seed_rht=5)
    A, B = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_MX, dev_status=status)
    assert int(status.item()) == 0
    assert_gemm_close(got.cpu().numpy(), ref, S, "2^30 spread, hardware scales")
    # each small group on its own: exact as well (the large group does not mask them)
    sub = oracle.QTensor(A.codes[:, 16:32].copy(), A.scales[:, 2:4].copy(), A.grid, A.scale_fmt)
    subB = oracle.QTensor(B.codes[:, 16:32].copy(), B.scales[:, 2:4].copy(), B.grid, B.scale_fmt)
    r2, s2 = oracle.gemm(sub, subB)
    g2 = ufp4.gemm(to_device(sub), to_device(subB), path=ufp4.PATH_MX)
    assert_gemm_close(g2.cpu().numpy(), r2, s2, "the small group alone")
    ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_TENSOR, dev_status=status)
    assert int(status.item()) & ufp4.DEV_EXP_WINDOW


def test_pow2_blocks_far_below_their_neighbour_are_flushed_and_reported():
    M, N, K = 128, 64, 64
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(11))
    x[:, 16:32] *= 2.0 ** -20                         # second half of the first 32-group: 2^20 below the first half
    X, W = x.to(torch.bfloat16), inputs.normal_bf16(N, K, 1.0, seed=12)
    kw = dict(rht_block=0, scale_fmt=oracle.SCALE_POW2, seed_rht=5)
    A, B = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_MX, dev_status=status)
    assert int(status.item()) & ufp4.DEV_EXP_WINDOW
    assert_gemm_close(got.cpu().numpy(), ref, S, "flushed blocks are far below the bound")    # 2^-20 of a term


def test_reduction_grouped_product():
    offsets = [0, 128, 128, 384, 512]
    H, F = 96, 80
    X = inputs.heavy_tailed_activations(512, H, seed=31)
    dY = inputs.normal_bf16(512, F, 1e-4, seed=33)
    kw = dict(rht_block=16, grid=oracle.GRID_INT4, scale_fmt=oracle.SCALE_E8M0_B32, seed_rht=1)
    Xc = oracle_quantize(X, oracle.AXIS_COL, **kw)
    Gc = oracle_quantize(dY, oracle.AXIS_COL, rounding=oracle.ROUND_SR, seed_sr=2, **kw)
    off_h = torch.tensor(offsets, dtype=torch.int64)
    ref, S = grouped_reference(Gc, Xc, offsets, F, ufp4.BWD_DW)
    got = ufp4.gemm_grouped(to_device(Gc), to_device(Xc), off_h.cuda(), off_h, F, ufp4.BWD_DW, path=ufp4.PATH_MX)
    assert_gemm_close(got.cpu().numpy(), ref, S, "bwd_dw grouped")
    assert torch.all(got[F:2 * F] == 0)
    Xr = oracle_quantize(X, oracle.AXIS_ROW, **kw)
    Wr = oracle_quantize(inputs.normal_bf16(4 * F, H, 0.02, seed=32), oracle.AXIS_ROW, **kw)
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_grouped(to_device(Xr), to_device(Wr), off_h.cuda(), off_h, F, ufp4.FWD_Y, path=ufp4.PATH_MX)
    assert e.value.status == -5
    # AUTO serves the row-grouped product of 1 x 32 tensors on the folded path
    assert ufp4.gemm_grouped(to_device(Xr), to_device(Wr), off_h.cuda(), off_h, F, ufp4.FWD_Y).shape == (512, F)
