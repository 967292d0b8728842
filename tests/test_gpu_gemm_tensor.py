"""Parity of the tensor-core GEMM path (power-of-two block scales folded into E5M2 operands) with the CPU oracle.

Operands are quantized by the ORACLE and uploaded.  Tolerance: |C_gpu - C_oracle| <= 1e-5 * sum_k |a_k b_k|."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs
from test_gpu_gemm import grouped_reference, three_products

pytestmark = pytest.mark.gpu


def run_tensor(A, B, **kw):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = ufp4.gemm(to_device(A), to_device(B), path=ufp4.PATH_TENSOR, dev_status=status, **kw)
    torch.cuda.synchronize()
    return out, int(status.item())


def test_single_tile_integer_operands():
    """One 128 x 256 x 128 tile, all scales 1: the result is an exact integer matrix product."""
    rng = np.random.default_rng(1)
    qa = rng.integers(-7, 8, size=(128, 128)).astype(np.float32)
    qb = rng.integers(-7, 8, size=(256, 128)).astype(np.float32)
    qa[:, ::16] = 7
    qb[:, ::16] = -7
    A = oracle_quantize(torch.from_numpy(qa).bfloat16(), oracle.AXIS_ROW, rht_block=0, scale_fmt=oracle.SCALE_POW2)
    B = oracle_quantize(torch.from_numpy(qb).bfloat16(), oracle.AXIS_ROW, rht_block=0, scale_fmt=oracle.SCALE_POW2)
    assert np.all(A.scales == 1) and np.all(B.scales == 1)
    out, status = run_tensor(A, B)
    assert status == 0
    assert np.array_equal(out.cpu().numpy(), (qa.astype(np.int64) @ qb.astype(np.int64).T).astype(np.float32))


@pytest.mark.parametrize("grid", [oracle.GRID_INT4, oracle.GRID_E1M2, oracle.GRID_E2M1])
def test_tiny_layer_all_three_products(grid):
    X, W, dY = inputs.tiny_layer(0)
    for name, (A, B, layout) in three_products(X, W, dY, grid, scale_fmt=oracle.SCALE_POW2).items():
        ref, S = oracle.gemm(A, B)
        out, status = run_tensor(A, B, layout=layout)
        assert status == 0
        assert_gemm_close(out.cpu().numpy(), ref, S, f"{name} grid {grid}")


@pytest.mark.parametrize("shape", [(200, 72, 176), (130, 260, 144), (384, 512, 1040), (1, 1, 16), (128, 256, 4096)])
def test_ragged_shapes(shape):
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=21)
    W = inputs.normal_bf16(N, K, 0.02, seed=22)
    A = oracle_quantize(X, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=5)
    B = oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=5, grid=oracle.GRID_E2M1)
    ref, S = oracle.gemm(A, B)
    out, status = run_tensor(A, B)
    assert status == 0
    assert_gemm_close(out.cpu().numpy(), ref, S, f"ragged {shape}")
    Np = (N + 7) // 8 * 8 + 8
    buf = torch.full((M, Np), 7.0, dtype=torch.bfloat16, device="cuda")
    out, status = run_tensor(A, B, out=buf[:, :N])
    assert_gemm_close(buf[:, :N].float().cpu().numpy(), ref, S, "bf16 out", bf16_out=True)
    assert torch.all(buf[:, N:] == 7.0)


def test_matches_exact_path_on_many_tiles_and_is_deterministic():
    """1024 x 1536 x 2048: more tiles than one wave of a few SMs, several k-blocks per tile; the tensor path must agree
    with the oracle on sampled entries and with itself across runs bit for bit."""
    M, N, K = 1024, 1536, 2048
    X = inputs.heavy_tailed_activations(M, K, seed=23)
    W = inputs.normal_bf16(N, K, 0.02, seed=24)
    A = oracle_quantize(X, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    B = oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    out, status = run_tensor(A, B)
    assert status == 0
    rng = np.random.default_rng(7)
    im, in_ = rng.integers(0, M, 20000), rng.integers(0, N, 20000)
    c, s = oracle.gemm_sampled(A, B, im, in_)
    assert_gemm_close(out.cpu().numpy()[im, in_], c, s, "sampled")
    out2, _ = run_tensor(A, B)
    assert torch.equal(out, out2)


def test_wide_exponent_spread_inside_a_row():
    """Block scales spanning 2^20 inside one row stay exact; a spread beyond the window is reported, not hidden."""
    M, N, K = 128, 256, 256
    rng = np.random.default_rng(9)
    x = rng.standard_normal((M, K)).astype(np.float32)
    for b in range(K // 16):
        x[:, 16 * b:16 * b + 16] *= 2.0 ** (-(b % 11) * 2)
    w = rng.standard_normal((N, K)).astype(np.float32)
    A = oracle_quantize(torch.from_numpy(x).bfloat16(), oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    B = oracle_quantize(torch.from_numpy(w).bfloat16(), oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    ref, S = oracle.gemm(A, B)
    out, status = run_tensor(A, B)
    assert status == 0
    assert_gemm_close(out.cpu().numpy(), ref, S, "2^20 spread")
    x[:, :16] *= 2.0 ** 30                       # one block 2^30 above the rest: the small blocks leave the window
    A = oracle_quantize(torch.from_numpy(x).bfloat16(), oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    out, status = run_tensor(A, B)
    assert status & ufp4.DEV_EXP_WINDOW


def test_grouped_products_small():
    offsets = [0, 128, 128, 384, 512]
    E, H, F = 4, 96, 80
    X = inputs.heavy_tailed_activations(512, H, seed=31)
    W = inputs.normal_bf16(E * F, H, 0.02, seed=32)
    dY = inputs.normal_bf16(512, F, 1e-4, seed=33)
    kw = dict(rht_block=16, grid=oracle.GRID_INT4, seed_rht=1, scale_fmt=oracle.SCALE_POW2)
    Xr, Xc = (oracle_quantize(X, a, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Gr, Gc = (oracle_quantize(dY, a, rounding=oracle.ROUND_SR, seed_sr=2, **kw) for a in (oracle.AXIS_ROW, oracle.AXIS_COL))
    Wr = oracle_quantize(W, oracle.AXIS_ROW, **kw)
    parts = [oracle_quantize(W[e * F:(e + 1) * F], oracle.AXIS_COL, **kw) for e in range(E)]
    Wc = oracle.QTensor(np.concatenate([p.codes for p in parts]), np.concatenate([p.scales for p in parts]),
                        oracle.GRID_INT4, oracle.SCALE_POW2)
    off_h = torch.tensor(offsets, dtype=torch.int64)
    off_d = off_h.cuda()
    cases = {"fwd_y": (Xr, Wr, ufp4.FWD_Y, F), "bwd_dx": (Gr, Wc, ufp4.BWD_DX, H), "bwd_dw": (Gc, Xc, ufp4.BWD_DW, F)}
    for name, (A, B, layout, gn) in cases.items():
        ref, S = grouped_reference(A, B, offsets, gn, layout)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        got = ufp4.gemm_grouped(to_device(A), to_device(B), off_d, off_h, gn, layout, path=ufp4.PATH_TENSOR,
                                dev_status=status).cpu().numpy()
        assert int(status.item()) == 0
        assert_gemm_close(got, ref, S, f"grouped {name}")
    got = ufp4.gemm_grouped(to_device(Gc), to_device(Xc), off_d, off_h, F, ufp4.BWD_DW, path=ufp4.PATH_TENSOR)
    assert torch.all(got[F:2 * F] == 0)


@pytest.mark.parametrize("grid", [oracle.GRID_INT4, oracle.GRID_E1M2, oracle.GRID_E2M1])
@pytest.mark.parametrize("path", [ufp4.PATH_TENSOR, ufp4.PATH_PROMOTE, ufp4.PATH_SPLIT, ufp4.PATH_EXACT])
def test_every_nibble_code_on_every_path(grid, path):
    """Hand-made operands holding all 16 nibble codes (also the ones the quantizer never emits: INT4 0x8 = -8, the
    negative zero of the sign | magnitude grids) with scales spread over the exponent window, zero scales included."""
    rng = np.random.default_rng(7)
    M, N, K = 96, 80, 256

    def operand(rows):
        codes = rng.integers(0, 256, size=(rows, K // 2), dtype=np.uint8)
        codes[0, :8] = np.arange(8, dtype=np.uint8) * 0x22          # every code twice in row 0: 0x00, 0x22, ..., 0xEE
        codes[0, 8:16] = np.arange(8, 16, dtype=np.uint8) * 0x11
        scales = np.ldexp(1.0, rng.integers(-10, 11, size=(rows, K // 16))).astype(np.float32)
        scales[rng.random(scales.shape) < 0.1] = 0.0
        return oracle.QTensor(codes, scales, grid, oracle.SCALE_POW2)

    A, B = operand(M), operand(N)
    c_ref, s_ref = oracle.gemm(A, B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = ufp4.gemm(to_device(A), to_device(B), path=path, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_gemm_close(out.cpu().numpy(), c_ref, s_ref, f"grid {grid} path {path}")


def test_row_grouped_product_long_reduction_on_cta_pairs():
    """Row-grouped products with K >= 4096 run on CTA pairs whose 256-row tiles are laid out group by group: groups of
    128 (mod 256) rows (half-filled last tile), an empty group, a ragged N; every row must come from its own expert."""
    offsets = [0, 128, 128, 512, 768, 1408]
    E, H, F = 5, 4096, 200
    X = inputs.heavy_tailed_activations(offsets[-1], H, seed=41)
    W = inputs.normal_bf16(E * F, H, 0.02, seed=42)
    kw = dict(rht_block=16, grid=oracle.GRID_INT4, seed_rht=1, scale_fmt=oracle.SCALE_POW2)
    Xr = oracle_quantize(X, oracle.AXIS_ROW, **kw)
    Wr = oracle_quantize(W, oracle.AXIS_ROW, **kw)
    off_h = torch.tensor(offsets, dtype=torch.int64)
    ref, S = grouped_reference(Xr, Wr, offsets, F, ufp4.FWD_Y)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((offsets[-1], F), 7.0, dtype=torch.float32, device="cuda")
    ufp4.gemm_grouped(to_device(Xr), to_device(Wr), off_h.cuda(), off_h, F, ufp4.FWD_Y, path=ufp4.PATH_TENSOR,
                      dev_status=status, out=out)
    assert int(status.item()) == 0
    assert_gemm_close(out.cpu().numpy(), ref, S, "row-grouped, pairs")
