"""Parity of the CUDA quantizer with the CPU oracle: codes, scales and SR draws bit-exact, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_qtensor_equal, oracle_quantize
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs

pytestmark = pytest.mark.gpu

GRIDS = [ufp4.GRID_INT4, ufp4.GRID_E1M2, ufp4.GRID_E2M1, ufp4.GRID_E2M1_MAX4, ufp4.GRID_E2M1_MAX2]


def run_both(x, axis, **kw):
    """Quantize on the GPU (axis BOTH/ROW/COL) and with the oracle; compare every output."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ts = kw.get("tensor_scale")
    row, col = ufp4.quantize(x.cuda(), axis=axis, dev_status=status, **kw)
    okw = dict(kw)
    if ts is not None:
        okw["tensor_scale"] = float(ts)
    if row is not None:
        assert_qtensor_equal(row, oracle_quantize(x, oracle.AXIS_ROW, **okw), f"row variant {kw}")
    if col is not None:
        assert_qtensor_equal(col, oracle_quantize(x, oracle.AXIS_COL, **okw), f"col variant {kw}")
    assert int(status.item()) == 0
    return row, col


def test_tiny_layer_recipe():
    """The tiny single-layer check: UFP4 settings of Table 1 (RTNE for X and W, SR for dY, RHT 16, FP32 scales) and
    the same with the E2M1 grid."""
    X, W, dY = inputs.tiny_layer(0)
    for grid in (ufp4.GRID_INT4, ufp4.GRID_E1M2, ufp4.GRID_E2M1):
        for t in (X, W):
            run_both(t, ufp4.AXIS_BOTH, rht_block=16, grid=grid, rounding=ufp4.ROUND_RTNE, seed_rht=1)
        run_both(dY, ufp4.AXIS_BOTH, rht_block=16, grid=grid, rounding=ufp4.ROUND_SR, seed_rht=1, seed_sr=2)


@pytest.mark.parametrize("grid", GRIDS)
@pytest.mark.parametrize("rounding", [ufp4.ROUND_RTNE, ufp4.ROUND_SR])
@pytest.mark.parametrize("scale_fmt", [ufp4.SCALE_FP32, ufp4.SCALE_POW2, ufp4.SCALE_E4M3_TENSOR])
@pytest.mark.parametrize("rht_block", [0, 16])
def test_all_variants_on_a_ragged_multi_tile_matrix(grid, rounding, scale_fmt, rht_block):
    x = inputs.spiky_normal(272, 400, seed=5)          # 3 x 4 tiles of 128 with ragged edges in both directions
    kw = dict(rht_block=rht_block, grid=grid, rounding=rounding, scale_fmt=scale_fmt, seed_rht=3, seed_sr=11)
    if scale_fmt == ufp4.SCALE_E4M3_TENSOR:
        gmax = {ufp4.GRID_INT4: 7.0, ufp4.GRID_E1M2: 1.75, ufp4.GRID_E2M1: 6.0, ufp4.GRID_E2M1_MAX4: 4.0,
                ufp4.GRID_E2M1_MAX2: 2.0}[grid]
        kw["tensor_scale"] = float(np.float32(4.0 * x.float().abs().max().item() / (gmax * 448.0)))
    run_both(x, ufp4.AXIS_BOTH, **kw)


@pytest.mark.parametrize("rht_block,shape", [(32, (288, 160)), (64, (320, 192)), (128, (384, 256)), (128, (128, 128))])
@pytest.mark.parametrize("grid", [ufp4.GRID_INT4, ufp4.GRID_E1M2, ufp4.GRID_E2M1])
@pytest.mark.parametrize("rounding", [ufp4.ROUND_RTNE, ufp4.ROUND_SR])
@pytest.mark.parametrize("scale_fmt", [ufp4.SCALE_FP32, ufp4.SCALE_POW2, ufp4.SCALE_E4M3_TENSOR])
def test_wide_rht_blocks(rht_block, shape, grid, rounding, scale_fmt):
    """RHT blocks of 32 / 64 / 128 (the block sizes App. B lists beside the selected 16) on multi-tile matrices with
    ragged tile edges: both layouts bit-equal to the oracle."""
    x = inputs.spiky_normal(shape[0], shape[1], seed=rht_block + shape[0])
    kw = dict(rht_block=rht_block, grid=grid, rounding=rounding, scale_fmt=scale_fmt, seed_rht=7, seed_sr=13)
    if scale_fmt == ufp4.SCALE_E4M3_TENSOR:
        gmax = {ufp4.GRID_INT4: 7.0, ufp4.GRID_E1M2: 1.75, ufp4.GRID_E2M1: 6.0}[grid]
        kw["tensor_scale"] = float(np.float32(4.0 * x.float().abs().max().item() / (gmax * 448.0)))
    run_both(x, ufp4.AXIS_BOTH, **kw)


@pytest.mark.parametrize("rht_block", [0, 16, 64])
@pytest.mark.parametrize("grid", [ufp4.GRID_INT4, ufp4.GRID_E1M2, ufp4.GRID_E2M1, ufp4.GRID_E2M1_MAX4])
@pytest.mark.parametrize("rounding", [ufp4.ROUND_RTNE, ufp4.ROUND_SR])
def test_1x32_blocks_with_a_power_of_two_scale(rht_block, grid, rounding):
    """The MXFP4 block layout (1 x 32 blocks, E8M0 scale; Sec. 2.1's footnote): both layouts bit-equal to the oracle on a
    ragged multi-tile matrix, and the two halves of every 32-block share their scale."""
    x = inputs.spiky_normal(320, 192, seed=17)
    row, col = run_both(x, ufp4.AXIS_BOTH, rht_block=rht_block, grid=grid, rounding=rounding,
                        scale_fmt=ufp4.SCALE_E8M0_B32, seed_rht=5, seed_sr=9)
    for q in (row, col):
        assert torch.equal(q.scales[:, 0::2], q.scales[:, 1::2])


def test_1x32_blocks_feed_every_gemm_path_as_power_of_two_scales():
    from helpers import assert_gemm_close
    X = inputs.heavy_tailed_activations(200, 256, seed=81)
    W = inputs.normal_bf16(136, 256, 0.02, seed=82)
    kw = dict(rht_block=16, scale_fmt=ufp4.SCALE_E8M0_B32, seed_rht=3)
    A, _ = ufp4.quantize(X.cuda(), axis=ufp4.AXIS_ROW, **kw)
    B, _ = ufp4.quantize(W.cuda(), axis=ufp4.AXIS_ROW, **kw)
    ref, S = oracle.gemm(oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw))
    assert ufp4.gemm_path_name(A, B) == "tensor"
    for path in (ufp4.PATH_AUTO, ufp4.PATH_TENSOR, ufp4.PATH_SPLIT, ufp4.PATH_PROMOTE, ufp4.PATH_EXACT):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = ufp4.gemm(A, B, path=path, dev_status=status)
        assert int(status.item()) == 0
        assert_gemm_close(out.cpu().numpy(), ref, S, f"path {path}")
    with pytest.raises(ufp4.Ufp4Error):                     # 48 columns: not a multiple of 32
        ufp4.quantize(inputs.normal_bf16(32, 48, 1.0, seed=1).cuda(), axis=ufp4.AXIS_ROW, scale_fmt=ufp4.SCALE_E8M0_B32)


def test_wide_rht_single_axis_and_shape_rules():
    x = inputs.normal_bf16(48, 256, 1.0, seed=3)            # 48 rows: the row variant alone takes any row count
    run_both(x, ufp4.AXIS_ROW, rht_block=128, seed_rht=2)
    x = inputs.normal_bf16(192, 80, 1.0, seed=4)            # 80 columns: the col variant alone only needs rows % 64 == 0
    run_both(x, ufp4.AXIS_COL, rht_block=64, seed_rht=2)
    with pytest.raises(ufp4.Ufp4Error):                     # cols = 80 is not a multiple of 32
        ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=32)
    with pytest.raises(ufp4.Ufp4Error):
        ufp4.quantize(x.cuda(), axis=ufp4.AXIS_BOTH, rht_block=48)


def test_wide_rht_operands_feed_the_gemm():
    """Rotating both operands with the same 64-wide RHT leaves the product unchanged up to quantization: the GEMM of the
    GPU-quantized operands equals the oracle's GEMM of the oracle-quantized ones."""
    from helpers import assert_gemm_close
    X = inputs.heavy_tailed_activations(256, 512, seed=71)
    W = inputs.normal_bf16(192, 512, 0.02, seed=72)
    kw = dict(rht_block=64, scale_fmt=ufp4.SCALE_POW2, seed_rht=3)
    A, _ = ufp4.quantize(X.cuda(), axis=ufp4.AXIS_ROW, **kw)
    B, _ = ufp4.quantize(W.cuda(), axis=ufp4.AXIS_ROW, **kw)
    ref, S = oracle.gemm(oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw))
    out = ufp4.gemm(A, B)
    assert_gemm_close(out.cpu().numpy(), ref, S, "rht 64")
    plain = X.double() @ W.double().T
    assert float((out.cpu().double() - plain).norm() / plain.norm()) < 0.2


@pytest.mark.parametrize("shape", [(16, 16), (128, 128), (16, 2048), (2048, 16), (144, 16), (1040, 1296)])
def test_shapes(shape):
    x = inputs.heavy_tailed_activations(shape[0], shape[1], seed=shape[0] + shape[1])
    run_both(x, ufp4.AXIS_BOTH, rht_block=16, seed_rht=1)
    run_both(x, ufp4.AXIS_BOTH, rht_block=16, rounding=ufp4.ROUND_SR, seed_rht=1, seed_sr=77)


def test_single_axis_calls_and_odd_row_counts():
    x = inputs.normal_bf16(37, 96, 1.0, seed=9)       # 37 rows: row variant only
    run_both(x, ufp4.AXIS_ROW, rht_block=16, seed_rht=2)
    x = inputs.normal_bf16(1, 16, 1.0, seed=10)
    run_both(x, ufp4.AXIS_ROW, rht_block=16, seed_rht=2)
    x = inputs.normal_bf16(160, 208, 1.0, seed=11)
    run_both(x, ufp4.AXIS_COL, rht_block=16, seed_rht=2)
    run_both(x, ufp4.AXIS_ROW, rht_block=0)
    with pytest.raises(ufp4.Ufp4Error):
        ufp4.quantize(inputs.normal_bf16(37, 96, 1.0, seed=9).cuda(), axis=ufp4.AXIS_BOTH)


def test_strided_input_and_preallocated_padded_outputs():
    base = inputs.normal_bf16(128, 512, 1.0, seed=12).cuda()
    x = base[:, 64:64 + 208]                            # row pitch 512, start offset 128 bytes
    row, col = ufp4.quantize(x, axis=ufp4.AXIS_BOTH, rht_block=16, seed_rht=4)
    xc = x.contiguous()
    assert_qtensor_equal(row, oracle_quantize(xc, oracle.AXIS_ROW, rht_block=16, seed_rht=4), "strided row")
    assert_qtensor_equal(col, oracle_quantize(xc, oracle.AXIS_COL, rht_block=16, seed_rht=4), "strided col")
    # caller-chosen pitches: the padding must stay untouched
    out_row = ufp4.QTensor(torch.full((128, 128), 0xEE, dtype=torch.uint8, device="cuda"),
                           torch.full((128, 20), -1.0, dtype=torch.float32, device="cuda"), ufp4.GRID_INT4,
                           ufp4.SCALE_FP32, 208)
    ufp4.quantize(x, axis=ufp4.AXIS_ROW, rht_block=16, seed_rht=4, out_row=out_row)
    assert_qtensor_equal(ufp4.QTensor(out_row.codes, out_row.scales[:, :13], 0, 0, 208),
                         oracle_quantize(xc, oracle.AXIS_ROW, rht_block=16, seed_rht=4), "padded row")
    assert torch.all(out_row.codes[:, 104:] == 0xEE) and torch.all(out_row.scales[:, 13:] == -1.0)


def test_degenerate_values():
    x = torch.zeros(64, 64, dtype=torch.bfloat16)
    run_both(x, ufp4.AXIS_BOTH, rht_block=16, seed_rht=1)
    x[3, 5] = 1e-35                                      # below the 2^-100 threshold: still a zero block
    x[40, 17] = -2.5e-3
    x[41, 17] = 3e30
    x[10, :16] = 1.0                                     # a constant block: the RHT concentrates it in one coordinate
    run_both(x, ufp4.AXIS_BOTH, rht_block=16, seed_rht=1)
    run_both(x, ufp4.AXIS_BOTH, rht_block=0, rounding=ufp4.ROUND_SR, seed_sr=5)
    # every BF16 bit pattern that is finite, in one tensor (65280 finite patterns padded to 256 x 256 with zeros)
    bits = np.arange(65536, dtype=np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]
    allv = np.zeros(65536, dtype=np.uint16)
    allv[: bits.size] = bits
    xa = torch.from_numpy(allv.reshape(256, 256).copy()).view(torch.bfloat16)
    xa = torch.where(xa.float().abs() > 1e30, torch.zeros_like(xa), xa)   # stay inside the documented |x'| <= 2^120
    for grid in GRIDS:
        run_both(xa, ufp4.AXIS_BOTH, rht_block=0, grid=grid)
        run_both(xa, ufp4.AXIS_BOTH, rht_block=16, grid=grid, seed_rht=6)


def test_nonfinite_input_sets_the_status_bit():
    x = inputs.normal_bf16(32, 32, 1.0, seed=13)
    x[7, 9] = float("inf")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ufp4.quantize(x.cuda(), axis=ufp4.AXIS_BOTH, dev_status=status)
    assert int(status.item()) & ufp4.DEV_NONFINITE
    x[7, 9] = float("nan")
    status.zero_()
    ufp4.quantize(x.cuda(), axis=ufp4.AXIS_BOTH, rht_block=0, dev_status=status)
    assert int(status.item()) & ufp4.DEV_NONFINITE
    # the plain kernel (wider RHT blocks, 1 x 32 scale blocks) reports it too; finite inputs leave the word clear
    x = inputs.normal_bf16(128, 128, 1.0, seed=13)
    for kw in (dict(rht_block=64), dict(rht_block=16, scale_fmt=ufp4.SCALE_E8M0_B32), dict(rht_block=0, scale_fmt=ufp4.SCALE_E8M0_B32)):
        status.zero_()
        ufp4.quantize(x.cuda(), axis=ufp4.AXIS_BOTH, dev_status=status, **kw)
        assert int(status.item()) == 0
        for bad in (float("inf"), float("nan")):
            y = x.clone()
            y[100, 37] = bad
            status.zero_()
            ufp4.quantize(y.cuda(), axis=ufp4.AXIS_BOTH, dev_status=status, **kw)
            assert int(status.item()) & ufp4.DEV_NONFINITE, (kw, bad)


def test_batched_weights_stack_along_rows():
    E, N, K = 3, 48, 160
    W = inputs.normal_bf16(E * N, K, 0.02, seed=14)
    row, col = ufp4.quantize_batched(W.cuda().view(E, N, K), axis=ufp4.AXIS_BOTH, rht_block=16, seed_rht=8)
    assert_qtensor_equal(row, oracle_quantize(W, oracle.AXIS_ROW, rht_block=16, seed_rht=8), "stacked row variant")
    for e in range(E):
        ref = oracle_quantize(W[e * N:(e + 1) * N], oracle.AXIS_COL, rht_block=16, seed_rht=8)
        assert_qtensor_equal(col.row_slice(e * K, (e + 1) * K), ref, f"col variant of expert {e}")
    with pytest.raises(ufp4.Ufp4Error):
        ufp4.quantize_batched(W.cuda().view(E, N, K), rounding=ufp4.ROUND_SR)
    # the same with a 64-wide RHT block (the plain kernel): 3 experts of 64 x 192
    E, N, K = 3, 64, 192
    W = inputs.normal_bf16(E * N, K, 0.02, seed=16)
    row, col = ufp4.quantize_batched(W.cuda().view(E, N, K), axis=ufp4.AXIS_BOTH, rht_block=64, seed_rht=8)
    assert_qtensor_equal(row, oracle_quantize(W, oracle.AXIS_ROW, rht_block=64, seed_rht=8), "stacked row variant, rht 64")
    for e in range(E):
        ref = oracle_quantize(W[e * N:(e + 1) * N], oracle.AXIS_COL, rht_block=64, seed_rht=8)
        assert_qtensor_equal(col.row_slice(e * K, (e + 1) * K), ref, f"col variant of expert {e}, rht 64")


def test_repeated_runs_are_bit_identical():
    x = inputs.heavy_tailed_activations(512, 768, seed=15).cuda()
    a = ufp4.quantize(x, axis=ufp4.AXIS_BOTH, rounding=ufp4.ROUND_SR, seed_rht=1, seed_sr=2)
    for _ in range(3):
        b = ufp4.quantize(x, axis=ufp4.AXIS_BOTH, rounding=ufp4.ROUND_SR, seed_rht=1, seed_sr=2)
        for p, q in zip(a, b):
            assert torch.equal(p.codes, q.codes) and torch.equal(p.scales, q.scales)


def test_dense_layer_full_size():
    """Dense-1.5B-class up-projection tensors at full size (X 8192x2048, W 8192x2048, dY 8192x8192)."""
    X, W, dY = inputs.dense_layer(8192, 2048, 8192, seed=1, device="cuda")
    run_both(X.cpu(), ufp4.AXIS_BOTH, rht_block=16, seed_rht=1)
    run_both(W.cpu(), ufp4.AXIS_BOTH, rht_block=16, seed_rht=1, scale_fmt=ufp4.SCALE_POW2)
    run_both(dY.cpu(), ufp4.AXIS_BOTH, rht_block=16, rounding=ufp4.ROUND_SR, seed_rht=1, seed_sr=2)


def test_division_shortcuts_match_ieee_division_exhaustively():
    """The kernel's amax / g and g / amax sequences against the IEEE division: all 2^23 mantissas x 8 exponents x 3 g."""
    assert ufp4.selftest_division() == 0


def test_tensor_diagnostics_agree_with_the_oracle():
    """ufp4_diagnose (alpha of Eq. 3, NMSE of Sec. 3.3 / Eq. 7, level counts of Eq. 6, per-bin bias of Sec. 3.1) on the
    CUDA quantizer's output against the oracle's sums on the same tensor; ragged sizes; reproducible."""
    from paper_2606_20381_b200 import diagnostics
    x = inputs.spiky_normal(520, 1040, seed=3)
    xb = inputs.bf16_bits(x)
    for grid in GRIDS:
        for rht in (0, 16):
            row, _ = ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=rht, grid=grid, seed_rht=1)
            got = diagnostics.tensor_diagnostics(x.cuda(), row, rht, 1)
            ref_q = oracle_quantize(x, oracle.AXIS_ROW, rht_block=rht, grid=grid, seed_rht=1, want_y=True)
            ref = oracle.diagnose(xb, ref_q, rht, 1)
            assert np.array_equal(got["count"].numpy(), ref["count"])
            assert np.allclose(got["sums"].numpy()[:3], ref["sums"][:3], rtol=1e-6)   # FP32 inside a block, FP64 across
            assert np.allclose(got["bias"].numpy(), ref["bias"], atol=2e-5, equal_nan=True)
            assert abs(got["alpha"] - ref["alpha"]) < 1e-6 and abs(got["nmse"] - ref["nmse"]) < 1e-6 * ref["nmse"] + 1e-9
            assert abs(got["b_eff"] - ref["b_eff"]) < 1e-12
            # the older per-element measurement (oracle's y) gives the same per-bin means
            rc, rb = oracle.bin_bias(ref_q.y, ref_q.codes, grid)
            assert np.array_equal(got["count"].numpy(), rc)
            assert np.allclose(got["bias"].numpy(), rb, atol=2e-5, equal_nan=True)
            again = diagnostics.tensor_diagnostics(x.cuda(), row, rht, 1)
            assert torch.equal(again["sums"], got["sums"])
    # RHT blocks wider than the quant block (cols = 1040 is no multiple of them: a 1024-column slice)
    xs = x[:, :1024].contiguous()
    xsb = inputs.bf16_bits(xs)
    for rht in (32, 64, 128):
        row, _ = ufp4.quantize(xs.cuda(), axis=ufp4.AXIS_ROW, rht_block=rht, seed_rht=1)
        got = diagnostics.tensor_diagnostics(xs.cuda(), row, rht, 1)
        ref = oracle.diagnose(xsb, oracle_quantize(xs, oracle.AXIS_ROW, rht_block=rht, seed_rht=1), rht, 1)
        assert np.array_equal(got["count"].numpy(), ref["count"])
        assert np.allclose(got["sums"].numpy()[:3], ref["sums"][:3], rtol=1e-6)
        assert np.allclose(got["bias"].numpy(), ref["bias"], atol=2e-5, equal_nan=True)
    # direction of the effect the paper describes: after RHT the E2M1 levels 2 and 4 shrink, the uniform grid does not
    row, _ = ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=16, grid=ufp4.GRID_E2M1, seed_rht=1)
    _, b = diagnostics.per_bin_bias(x.cuda(), row, 16, 1)
    assert b[4] < -0.05 and b[6] < -0.1
    row, _ = ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=16, grid=ufp4.GRID_INT4, seed_rht=1)
    _, b = diagnostics.per_bin_bias(x.cuda(), row, 16, 1)
    assert abs(b[1:7]).max() < 0.05     # what remains is the decreasing density inside symmetric bins, not geometry
    # Sec. 5.4: restricting E2M1 to magnitudes <= 2 removes the asymmetric bins but gives up bucket utilization
    row, _ = ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=16, grid=ufp4.GRID_E2M1_MAX2, seed_rht=1)
    d2 = diagnostics.tensor_diagnostics(x.cuda(), row, 16, 1)
    assert d2["count"][5:].sum() == 0 and abs(d2["bias"][1:4]).max() < 0.05
    row, _ = ufp4.quantize(x.cuda(), axis=ufp4.AXIS_ROW, rht_block=16, grid=ufp4.GRID_E2M1, seed_rht=1)
    assert d2["b_eff"] < diagnostics.tensor_diagnostics(x.cuda(), row, 16, 1)["b_eff"]


def test_rht_helps_the_uniform_grid_more_than_e2m1_on_outlier_heavy_tensors():
    """Sec. 3.3's observation on synthetic heavy-tailed activations: the RHT raises the effective bucket ratio of both
    grids, and its SQNR change (Eq. 7) is better for the uniform grid than for E2M1."""
    from paper_2606_20381_b200 import diagnostics
    x = inputs.heavy_tailed_activations(2048, 2048, seed=9).cuda()
    d = {}
    for grid in (ufp4.GRID_INT4, ufp4.GRID_E2M1):
        for rht in (0, 16):
            row, _ = ufp4.quantize(x, axis=ufp4.AXIS_ROW, rht_block=rht, grid=grid, seed_rht=1)
            d[(grid, rht)] = diagnostics.tensor_diagnostics(x, row, rht, 1)
    dsqnr = {g: 10 * np.log10(d[(g, 0)]["nmse"] / d[(g, 16)]["nmse"]) for g in (ufp4.GRID_INT4, ufp4.GRID_E2M1)}
    assert d[(ufp4.GRID_INT4, 16)]["b_eff"] > d[(ufp4.GRID_INT4, 0)]["b_eff"]
    assert d[(ufp4.GRID_E2M1, 16)]["b_eff"] > d[(ufp4.GRID_E2M1, 0)]["b_eff"]
    assert dsqnr[ufp4.GRID_INT4] > 0 and dsqnr[ufp4.GRID_INT4] > dsqnr[ufp4.GRID_E2M1]


def test_quantize_multi_equals_separate_calls_and_the_oracle():
    """Independent tensors in one call (dependent launches that overlap each other's tails): every output bit-equal to the
    oracle, whatever the mix of shapes, roundings, grids and kernels (the 16-point tile kernel, the plain kernel of the wider
    RHT blocks and of the 1 x 32 scale blocks)."""
    xs = [inputs.spiky_normal(272, 400, seed=1), inputs.normal_bf16(144, 400, 0.02, seed=2), inputs.normal_bf16(272, 144, 1e-3, seed=3),
          inputs.spiky_normal(256, 192, seed=4), inputs.spiky_normal(96, 160, seed=5), inputs.spiky_normal(1040, 2064, seed=6)]
    kws = [dict(rht_block=16, grid=ufp4.GRID_INT4, rounding=ufp4.ROUND_RTNE, scale_fmt=ufp4.SCALE_POW2, seed_rht=1),
           dict(rht_block=16, grid=ufp4.GRID_INT4, rounding=ufp4.ROUND_RTNE, scale_fmt=ufp4.SCALE_POW2, seed_rht=1),
           dict(rht_block=16, grid=ufp4.GRID_INT4, rounding=ufp4.ROUND_SR, scale_fmt=ufp4.SCALE_POW2, seed_rht=1, seed_sr=2),
           dict(rht_block=64, grid=ufp4.GRID_E1M2, rounding=ufp4.ROUND_RTNE, scale_fmt=ufp4.SCALE_FP32, seed_rht=7),
           dict(rht_block=16, grid=ufp4.GRID_E2M1, rounding=ufp4.ROUND_SR, scale_fmt=ufp4.SCALE_E8M0_B32, seed_rht=3, seed_sr=9),
           dict(rht_block=0, grid=ufp4.GRID_E2M1, rounding=ufp4.ROUND_RTNE, scale_fmt=ufp4.SCALE_FP32, seed_rht=0)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dev = [x.cuda() for x in xs]
    for _ in range(3):                      # repeated, so that a launch of one round follows the last of the round before
        outs = ufp4.quantize_multi([dict(x=d, axis=ufp4.AXIS_BOTH, **kw) for d, kw in zip(dev, kws)], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for x, kw, (row, col) in zip(xs, kws, outs):
        assert_qtensor_equal(row, oracle_quantize(x, oracle.AXIS_ROW, **kw), f"multi row {kw}")
        assert_qtensor_equal(col, oracle_quantize(x, oracle.AXIS_COL, **kw), f"multi col {kw}")
    # a consumer enqueued right behind the call sees every tensor complete: the product of the first two tensors' row
    # variants, taken straight after a fresh multi call into fresh outputs
    outs = ufp4.quantize_multi([dict(x=d, axis=ufp4.AXIS_BOTH, **kw) for d, kw in zip(dev[:3], kws[:3])])
    got = ufp4.gemm(outs[0][0], outs[1][0])
    ref, S = oracle.gemm(oracle_quantize(xs[0], oracle.AXIS_ROW, **kws[0]), oracle_quantize(xs[1], oracle.AXIS_ROW, **kws[1]))
    from helpers import assert_gemm_close
    assert_gemm_close(got.cpu().numpy(), ref, S, "product right behind a multi call")


def test_quantize_multi_checks_every_tensor_before_launching_any():
    good = inputs.normal_bf16(64, 64, 1.0, seed=1).cuda()
    row = ufp4.alloc_qtensor(64, 64, ufp4.GRID_INT4, ufp4.SCALE_FP32, "cuda")
    col = ufp4.alloc_qtensor(64, 64, ufp4.GRID_INT4, ufp4.SCALE_FP32, "cuda")
    row.codes.fill_(0xAB)
    bad_out = ufp4.alloc_qtensor(64, 48, ufp4.GRID_INT4, ufp4.SCALE_FP32, "cuda")        # wrong shape for the second tensor
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.quantize_multi([dict(x=good, out_row=row, out_col=col), dict(x=good, out_row=bad_out, out_col=col)])
    assert e.value.status == -2
    torch.cuda.synchronize()
    assert torch.all(row.codes == 0xAB)                       # the first tensor was not quantized either
    assert ufp4.quantize_multi([]) == []
