"""Parity of the CUDA GEMMs with the CPU oracle: |C_gpu - C_oracle| <= 1e-5 * sum_k |a_k b_k| per element.

Operands are quantized by the ORACLE and uploaded, so the GEMM check does not depend on the CUDA quantizer."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, assert_qtensor_equal, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs

pytestmark = pytest.mark.gpu


def three_products(X, W, dY, grid, scale_fmt=oracle.SCALE_FP32, seed_rht=1, seed_sr=2, rht_block=16):
    """The operands of fwd_y, bwd_dx and bwd_dw per the recipe: RTNE for X and W, SR for dY (Table 1)."""
    kw = dict(rht_block=rht_block, grid=grid, scale_fmt=scale_fmt, seed_rht=seed_rht)
    Xr, Xc = (oracle_quantize(X, a, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Wr, Wc = (oracle_quantize(W, a, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Gr, Gc = (oracle_quantize(dY, a, rounding=oracle.ROUND_SR, seed_sr=seed_sr, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    return {"fwd_y": (Xr, Wr, ufp4.FWD_Y), "bwd_dx": (Gr, Wc, ufp4.BWD_DX), "bwd_dw": (Gc, Xc, ufp4.BWD_DW)}


@pytest.mark.parametrize("path", [ufp4.PATH_EXACT, ufp4.PATH_PROMOTE, ufp4.PATH_SPLIT])
@pytest.mark.parametrize("grid", [oracle.GRID_INT4, oracle.GRID_E1M2, oracle.GRID_E2M1])
def test_tiny_layer_all_three_products(grid, path):
    X, W, dY = inputs.tiny_layer(0)
    for name, (A, B, layout) in three_products(X, W, dY, grid).items():
        ref, S = oracle.gemm(A, B)
        got = ufp4.gemm(to_device(A), to_device(B), layout=layout, path=path).cpu().numpy()
        assert got.shape == ref.shape
        assert_gemm_close(got, ref, S, f"{name} grid {grid}")
        # against the unquantized product: same rotation on both operands, so only quantization error remains
    exact = X.double().numpy() @ W.double().numpy().T
    A, B, _ = three_products(X, W, dY, oracle.GRID_INT4)["fwd_y"]
    got = ufp4.gemm(to_device(A), to_device(B), path=path).cpu().numpy()
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.2


@pytest.mark.parametrize("path", [ufp4.PATH_EXACT, ufp4.PATH_PROMOTE, ufp4.PATH_SPLIT])
@pytest.mark.parametrize("scale_fmt", [oracle.SCALE_FP32, oracle.SCALE_POW2, oracle.SCALE_E4M3_TENSOR])
def test_ragged_shapes_and_scale_formats_exact_path(scale_fmt, path):
    M, N, K = 200, 72, 176
    X = inputs.heavy_tailed_activations(M, K, seed=21)
    W = inputs.normal_bf16(N, K, 0.02, seed=22)
    kw = dict(rht_block=16, scale_fmt=scale_fmt, seed_rht=5)
    kwx, kww = dict(kw), dict(kw)
    if scale_fmt == oracle.SCALE_E4M3_TENSOR:
        kwx["tensor_scale"] = float(np.float32(4 * X.float().abs().max().item() / (7 * 448)))
        kww["tensor_scale"] = float(np.float32(4 * W.float().abs().max().item() / (6 * 448)))
    A = oracle_quantize(X, oracle.AXIS_ROW, grid=oracle.GRID_INT4, **kwx)
    B = oracle_quantize(W, oracle.AXIS_ROW, grid=oracle.GRID_E2M1, **kww)        # mixed grids are allowed
    ref, S = oracle.gemm(A, B)
    got = ufp4.gemm(to_device(A), to_device(B), path=path).cpu().numpy()
    assert_gemm_close(got, ref, S, f"ragged fmt {scale_fmt}")
    out = torch.full((M, 80), 7.0, dtype=torch.bfloat16, device="cuda")        # BF16 output into a padded buffer
    ufp4.gemm(to_device(A), to_device(B), out=out[:, :N], path=path)
    assert_gemm_close(out[:, :N].float().cpu().numpy(), ref, S, "bf16 out", bf16_out=True)
    assert torch.all(out[:, N:] == 7.0)


@pytest.mark.parametrize("path", [ufp4.PATH_PROMOTE, ufp4.PATH_SPLIT])
@pytest.mark.parametrize("shape", [(130, 260, 144), (384, 512, 1040), (1, 1, 16), (128, 128, 4096), (1024, 1536, 2048),
                                   (2600, 1100, 528)])
def test_fp32_scale_tensor_core_paths_shapes(shape, path):
    """The two tensor-core paths for FP32 scales (block promotion; FP16 two-piece operands) over ragged, multi-tile and
    long-K shapes; the last shape gives the persistent CTA pairs several tiles each."""
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=21)
    W = inputs.normal_bf16(N, K, 0.02, seed=22)
    A = oracle_quantize(X, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_FP32, seed_rht=5)
    B = oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_FP32, seed_rht=5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = ufp4.gemm(to_device(A), to_device(B), path=path, dev_status=status)
    assert int(status.item()) == 0
    if M * N <= 1 << 19:
        ref, S = oracle.gemm(A, B)
        assert_gemm_close(out.cpu().numpy(), ref, S, f"path {path} {shape}")
    else:
        rng = np.random.default_rng(7)
        im, in_ = rng.integers(0, M, 20000), rng.integers(0, N, 20000)
        c, s = oracle.gemm_sampled(A, B, im, in_)
        assert_gemm_close(out.cpu().numpy()[im, in_], c, s, f"path {path} sampled {shape}")
    assert torch.equal(out, ufp4.gemm(to_device(A), to_device(B), path=path))
    assert ufp4.gemm_path_name(to_device(A), to_device(B), ufp4.PATH_AUTO) == "split"


def test_integer_and_one_hot_operands():
    rng = np.random.default_rng(3)
    qa = rng.integers(-7, 8, size=(64, 64)).astype(np.float32)
    qb = rng.integers(-7, 8, size=(64, 64)).astype(np.float32)
    qa[:, ::16] = 7
    qb[:, ::16] = -7
    A = oracle_quantize(torch.from_numpy(qa).bfloat16(), oracle.AXIS_ROW, rht_block=0)
    B = oracle_quantize(torch.from_numpy(qb).bfloat16(), oracle.AXIS_ROW, rht_block=0)
    got = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_EXACT).cpu().numpy()
    assert np.array_equal(got, (qa.astype(np.int64) @ qb.astype(np.int64).T).astype(np.float32))


def grouped_reference(A, B, offsets, group_n, layout):
    G = len(offsets) - 1
    if layout == ufp4.BWD_DW:
        C = np.zeros((G * A.rows, B.rows))
        S = np.zeros_like(C)
        da, db = oracle.dequantize(A), oracle.dequantize(B)
        for g in range(G):
            k0, k1 = offsets[g], offsets[g + 1]
            if k1 > k0:
                c, s = oracle.gemm_f64(da[:, k0:k1], db[:, k0:k1])
                C[g * A.rows:(g + 1) * A.rows], S[g * A.rows:(g + 1) * A.rows] = c, s
        return C, S
    C = np.zeros((A.rows, group_n))
    S = np.zeros_like(C)
    da, db = oracle.dequantize(A), oracle.dequantize(B)
    for g in range(G):
        r0, r1 = offsets[g], offsets[g + 1]
        if r1 > r0:
            C[r0:r1], S[r0:r1] = oracle.gemm_f64(da[r0:r1], db[g * group_n:(g + 1) * group_n])
    return C, S


def test_grouped_products_small():
    """Four experts, one of them empty; hidden 96, expert FFN 80."""
    offsets = [0, 128, 128, 384, 512]
    E, H, F = 4, 96, 80
    X = inputs.heavy_tailed_activations(512, H, seed=31)
    W = inputs.normal_bf16(E * F, H, 0.02, seed=32)
    dY = inputs.normal_bf16(512, F, 1e-4, seed=33)
    kw = dict(rht_block=16, grid=oracle.GRID_INT4, seed_rht=1)
    Xr, Xc = (oracle_quantize(X, a, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Gr, Gc = (oracle_quantize(dY, a, rounding=oracle.ROUND_SR, seed_sr=2, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Wr = oracle_quantize(W, oracle.AXIS_ROW, **kw)
    parts = [oracle_quantize(W[e * F:(e + 1) * F], oracle.AXIS_COL, **kw) for e in range(E)]
    Wc = oracle.QTensor(np.concatenate([p.codes for p in parts]), np.concatenate([p.scales for p in parts]),
                        oracle.GRID_INT4, oracle.SCALE_FP32)
    off_h = torch.tensor(offsets, dtype=torch.int64)
    off_d = off_h.cuda()
    cases = {"fwd_y": (Xr, Wr, ufp4.FWD_Y, F), "bwd_dx": (Gr, Wc, ufp4.BWD_DX, H), "bwd_dw": (Gc, Xc, ufp4.BWD_DW, F)}
    for name, (A, B, layout, gn) in cases.items():
        ref, S = grouped_reference(A, B, offsets, gn, layout)
        for path in (ufp4.PATH_EXACT, ufp4.PATH_PROMOTE, ufp4.PATH_SPLIT):
            got = ufp4.gemm_grouped(to_device(A), to_device(B), off_d, off_h, gn, layout, path=path).cpu().numpy()
            assert got.shape == ref.shape, name
            assert_gemm_close(got, ref, S, f"grouped {name} path {path}")
    # the empty group's dW is exactly zero
    got = ufp4.gemm_grouped(to_device(Gc), to_device(Xc), off_d, off_h, F, ufp4.BWD_DW, path=ufp4.PATH_EXACT)
    assert torch.all(got[F:2 * F] == 0)


def test_split_path_exponent_window_and_extreme_scales():
    """FP16 two-piece operands: block scales spanning 2^20 inside a row stay within the bound, a spread beyond the
    window (2^26) is reported, and rows whose scales sit near the ends of the quantizer's range (2^-100, 2^100) work."""
    M, N, K = 160, 272, 256
    rng = np.random.default_rng(9)
    x = rng.standard_normal((M, K)).astype(np.float32)
    for b in range(K // 16):
        x[:, 16 * b:16 * b + 16] *= 2.0 ** (-(b % 11) * 2)
    x[3] *= 2.0 ** -90                           # tiny row: scales near 2^-100
    x[5] *= 2.0 ** 100                           # huge row
    w = rng.standard_normal((N, K)).astype(np.float32)
    w[7] *= 2.0 ** -20                           # products stay inside FP32's range: 2^-110 .. 2^100
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_FP32, seed_rht=1)
    A = oracle_quantize(torch.from_numpy(x).bfloat16(), oracle.AXIS_ROW, **kw)
    B = oracle_quantize(torch.from_numpy(w).bfloat16(), oracle.AXIS_ROW, grid=oracle.GRID_E1M2, **kw)
    ref, S = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_SPLIT, dev_status=status)
    assert int(status.item()) == 0
    assert_gemm_close(out.cpu().numpy(), ref, S, "2^20 spread, extreme rows")
    x[5] *= 2.0 ** -100
    x[:, :16] *= 2.0 ** 30                       # one block 2^30 above the rest: the small blocks leave the window
    A = oracle_quantize(torch.from_numpy(x).bfloat16(), oracle.AXIS_ROW, **kw)
    ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_SPLIT, dev_status=status)
    assert int(status.item()) & ufp4.DEV_EXP_WINDOW


@pytest.mark.parametrize("grid", [ufp4.GRID_E2M1_MAX4, ufp4.GRID_E2M1_MAX2])
def test_range_restricted_e2m1_operands_on_every_path(grid):
    """Sec. 5.4's range-restricted E2M1 (max_fpx = 4 / 2): quantized on the GPU, bit-equal to the oracle, and read by
    every GEMM path as the E2M1 codes they are."""
    M, N, K = 200, 136, 320
    X = inputs.heavy_tailed_activations(M, K, seed=61)
    W = inputs.normal_bf16(N, K, 0.02, seed=62)
    for scale_fmt, paths in ((oracle.SCALE_POW2, (ufp4.PATH_TENSOR, ufp4.PATH_SPLIT, ufp4.PATH_EXACT)),
                             (oracle.SCALE_FP32, (ufp4.PATH_SPLIT, ufp4.PATH_PROMOTE, ufp4.PATH_EXACT, ufp4.PATH_AUTO))):
        kw = dict(rht_block=16, grid=grid, scale_fmt=scale_fmt, seed_rht=1)
        A, _ = ufp4.quantize(X.cuda(), axis=ufp4.AXIS_ROW, **kw)
        B, _ = ufp4.quantize(W.cuda(), axis=ufp4.AXIS_ROW, **kw)
        Ao, Bo = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)
        assert_qtensor_equal(A, Ao, "A")
        assert_qtensor_equal(B, Bo, "B")
        ref, S = oracle.gemm(Ao, Bo)
        for path in paths:
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = ufp4.gemm(A, B, path=path, dev_status=status)
            assert int(status.item()) == 0
            assert_gemm_close(out.cpu().numpy(), ref, S, f"grid {grid} fmt {scale_fmt} path {path}")
