"""ufp4_gemm_quantized: the tensor-core product with a quantizing epilogue.  The oracle's version of the same thing is
its FP64 product, rounded to BF16, fed to its quantizer.  The GPU rounds its FP32 tensor-core result to BF16, so a BF16
value can differ by one unit in the last place where the exact product lies within the GEMM bound of a rounding boundary,
and codes of the 16-block it sits in can then differ.  The test therefore checks: (1) the BF16 product within the GEMM
bound; (2) every 16-block whose sixteen BF16 inputs agree with the oracle's is bit-identical in codes and scale - the
vast majority; (3) the few other blocks dequantize to within one grid step of the oracle's."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs
from paper_2606_20381_b200.inputs import bf16_bits

pytestmark = pytest.mark.gpu


def _to_bf16_bits(c64: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(c64.astype(np.float32)).to(torch.bfloat16)
    return bf16_bits(t)


def _check_variant(gpu: ufp4.QTensor, ref: oracle.QTensor, agree: np.ndarray, what: str):
    """agree [R][K/16]: the block's sixteen BF16 inputs were the same on both sides."""
    codes = gpu.packed_codes().cpu().numpy().reshape(ref.rows, -1, 8)
    scales = gpu.scales.cpu().numpy()
    rc = ref.codes.reshape(ref.rows, -1, 8)
    same = np.all(codes == rc, axis=2) & (scales.view(np.uint32) == ref.scales.view(np.uint32))
    assert np.all(same[agree]), f"{what}: {np.count_nonzero(~same & agree)} blocks with identical inputs differ"
    assert agree.mean() > 0.9, f"{what}: only {agree.mean():.3f} of the blocks had identical BF16 inputs"
    # the others: dequantized values within one step of the oracle's (the block's input moved by one BF16 ulp)
    g = oracle.QTensor(gpu.packed_codes().cpu().numpy(), scales, ref.grid, ref.scale_fmt)
    dg, dr = oracle.dequantize(g), oracle.dequantize(ref)
    step = np.repeat(np.maximum(scales, ref.scales).astype(np.float64), 16, axis=1)
    assert np.all(np.abs(dg - dr) <= step * 1.0001 + 1e-300), what
    return float(1.0 - same.mean())


@pytest.mark.parametrize("scale_fmt", [oracle.SCALE_FP32, oracle.SCALE_POW2])
@pytest.mark.parametrize("rht", [16, 0])
@pytest.mark.parametrize("shape", [(256, 256, 256), (384, 528, 1040), (1024, 2048, 512)])
def test_quantizing_epilogue_matches_quantizing_the_oracle_product(shape, rht, scale_fmt):
    M, N, K = shape
    X = inputs.heavy_tailed_activations(M, K, seed=51)
    W = inputs.normal_bf16(N, K, 0.02, seed=52)
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    A, B = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)
    C64, S = oracle.gemm(A, B)
    cb = _to_bf16_bits(C64)
    qkw = dict(rht_block=rht, grid=oracle.GRID_INT4, rounding=oracle.ROUND_RTNE, scale_fmt=scale_fmt, seed_rht=7)
    ref_row, ref_col = oracle.quantize(cb, oracle.AXIS_ROW, **qkw), oracle.quantize(cb, oracle.AXIS_COL, **qkw)

    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_row, out_col, c16 = ufp4.gemm_quantized(to_device(A), to_device(B), rht_block=rht, seed_rht=7, scale_fmt=scale_fmt,
                                                want_c=True, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_gemm_close(c16.float().cpu().numpy(), C64, S, "BF16 product", bf16_out=True)
    gb = bf16_bits(c16.cpu())
    eq = gb == cb
    assert eq.mean() > 0.98
    # a differing BF16 value is a neighbour of the oracle's
    d = np.abs(gb[~eq].astype(np.int64) - cb[~eq].astype(np.int64))
    assert np.all((d == 1) | (d == 0x8000) | (d == 0x8001)), "BF16 values differ by more than one unit in the last place"
    agree_row = eq.reshape(M, N // 16, 16).all(axis=2)
    agree_col = eq.T.reshape(N, M // 16, 16).all(axis=2)
    _check_variant(out_row, ref_row, agree_row, f"row layout {shape} rht {rht} fmt {scale_fmt}")
    _check_variant(out_col, ref_col, agree_col, f"col layout {shape} rht {rht} fmt {scale_fmt}")

    # one layout at a time, without the BF16 copy: the same codes
    only_row, none_col, none_c = ufp4.gemm_quantized(to_device(A), to_device(B), rht_block=rht, seed_rht=7, scale_fmt=scale_fmt,
                                                     want_col=False)
    assert none_col is None and none_c is None
    assert torch.equal(only_row.packed_codes(), out_row.packed_codes()) and torch.equal(only_row.scales, out_row.scales)
    none_row, only_col, _ = ufp4.gemm_quantized(to_device(A), to_device(B), rht_block=rht, seed_rht=7, scale_fmt=scale_fmt,
                                                want_row=False)
    assert none_row is None
    assert torch.equal(only_col.packed_codes(), out_col.packed_codes()) and torch.equal(only_col.scales, out_col.scales)


def test_the_outputs_feed_the_next_product():
    """Layer chain: Y = X W1^T quantized in the epilogue is the A operand of Y W2^T; against the oracle chain."""
    T, K, N, N2 = 256, 512, 384, 128
    X = inputs.heavy_tailed_activations(T, K, seed=61)
    W1 = inputs.normal_bf16(N, K, 0.02, seed=62)
    W2 = inputs.normal_bf16(N2, N, 0.02, seed=63)
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    A, B = oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W1, oracle.AXIS_ROW, **kw)
    B2 = oracle_quantize(W2, oracle.AXIS_ROW, **kw)
    yq, _, _ = ufp4.gemm_quantized(to_device(A), to_device(B), rht_block=16, seed_rht=1, scale_fmt=ufp4.SCALE_POW2, want_col=False)
    got = ufp4.gemm(yq, to_device(B2), path=ufp4.PATH_TENSOR).cpu().numpy()
    C64, _ = oracle.gemm(A, B)
    yref = oracle.quantize(_to_bf16_bits(C64), oracle.AXIS_ROW, **dict(kw, grid=oracle.GRID_INT4))
    want, S = oracle.gemm(yref, B2)
    # a few codes of Y may differ by one level (see the module docstring): compare at the size of one grid step per term
    step = np.repeat(yref.scales.astype(np.float64), 16, axis=1)
    slack = np.abs(step) @ np.abs(oracle.dequantize(B2)).T
    assert np.all(np.abs(got - want) <= 1e-5 * S + 0.02 * slack + 1e-300)


def test_rejects_what_it_cannot_do():
    X = inputs.normal_bf16(64, 64, 1.0, seed=1)
    A = to_device(oracle_quantize(X, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1))
    F = to_device(oracle_quantize(X, oracle.AXIS_ROW, rht_block=16, scale_fmt=oracle.SCALE_FP32, seed_rht=1))
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_quantized(F, F)                       # FP32-scale operands have no tensor-core 8-bit form
    assert e.value.status == -5
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_quantized(A, A, rht_block=64)
    assert e.value.status == -5
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_quantized(A, A, want_row=False, want_col=False)
    assert e.value.status == -1
    bad = ufp4.alloc_qtensor(64, 64, ufp4.GRID_E2M1, ufp4.SCALE_FP32, "cuda")
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_quantized(A, A, out_row=bad, want_col=False)
    assert e.value.status == -5
