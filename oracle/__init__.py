"""UFP4 oracle — TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Thin numpy/ctypes access to oracle/ufp4_oracle.c, the plain CPU statement of the paper's definitions (Sec. 2.1
blockwise quantizer and rounding rules, Sec. 2.2 Hadamard / RHT and the RHT'd GEMMs, Sec. 3.1 per-bin rounding
error, Sec. 4 / Table 1 recipe settings).  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; it shares nothing with the CUDA library and never imports it.

BF16 tensors are passed as numpy uint16 arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from .build import build as _build

GRID_INT4, GRID_E1M2, GRID_E2M1 = 0, 1, 2
GRID_E2M1_MAX4, GRID_E2M1_MAX2 = 3, 4      # E2M1 with the magnitudes above 4 / above 2 unused (Sec. 5.4, max_fpx)
ROUND_RTNE, ROUND_SR = 0, 1
SCALE_FP32, SCALE_POW2, SCALE_E4M3_TENSOR = 0, 1, 2
SCALE_E8M0_B32 = 3      # one power-of-two scale per 32 elements (MXFP4's block layout), stored per 16-element half
AXIS_ROW, AXIS_COL = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        p, i64, u64, i32, f32, f64 = C.c_void_p, C.c_int64, C.c_uint64, C.c_int, C.c_float, C.c_double
        L.orc_level.restype = f64
        L.orc_level.argtypes = [i32, i32]
        L.orc_gmax.restype = f64
        L.orc_gmax.argtypes = [i32]
        L.orc_num_levels.restype = i32
        L.orc_num_levels.argtypes = [i32]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [p, p, p]
        L.orc_rht_sign_mask.restype = C.c_uint32
        L.orc_rht_sign_mask.argtypes = [u64]
        L.orc_sr_bytes.restype = None
        L.orc_sr_bytes.argtypes = [u64, u64, C.c_uint32, p]
        L.orc_hadamard_matrix.restype = None
        L.orc_hadamard_matrix.argtypes = [i32, p]
        L.orc_rht_signs.restype = None
        L.orc_rht_signs.argtypes = [u64, p]
        L.orc_rht_f32.restype = None
        L.orc_rht_f32.argtypes = [p, i32, p]
        L.orc_rht16_f32.restype = None
        L.orc_rht16_f32.argtypes = [p, C.c_uint32]
        L.orc_round_rtne.restype = i32
        L.orc_round_rtne.argtypes = [f64, i32]
        L.orc_round_sr.restype = i32
        L.orc_round_sr.argtypes = [f64, i32, i32]
        L.orc_nibble_value.restype = f64
        L.orc_nibble_value.argtypes = [i32, i32]
        L.orc_e4m3_value.restype = f64
        L.orc_e4m3_value.argtypes = [i32]
        L.orc_e4m3_encode.restype = i32
        L.orc_e4m3_encode.argtypes = [f32]
        L.orc_quantize.restype = i32
        L.orc_quantize.argtypes = [p, i64, i64, i64, i32, i32, i32, i32, i32, u64, u64, f32, p, p, p]
        L.orc_quantize_window.restype = i32
        L.orc_quantize_window.argtypes = [p, i64, i64, i64, i32, i32, i32, i32, i32, u64, u64, f32, p, p, p, i64, i64, i64]
        L.orc_dequantize.restype = None
        L.orc_dequantize.argtypes = [p, p, i64, i32, i32, f32, i64, i64, p]
        L.orc_gemm_f64.restype = None
        L.orc_gemm_f64.argtypes = [p, p, i64, i64, i64, p, p]
        L.orc_gemm_sampled.restype = None
        L.orc_gemm_sampled.argtypes = [p, p, i32, i32, f32, p, p, i32, i32, f32, i64, i64, i64, i64, p, p, p, p]
        L.orc_bin_bias.restype = None
        L.orc_bin_bias.argtypes = [p, p, i64, i32, p, p]
        L.orc_diagnose.restype = None
        L.orc_diagnose.argtypes = [p, i64, i64, i64, p, i64, p, i64, i32, i32, u64, p]
        L.orc_b_eff.restype = f64
        L.orc_b_eff.argtypes = [p]
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class QTensor:
    """A quantized tensor: logical [rows][k], k the reduction dimension (blocks of 16 along it)."""
    codes: np.ndarray          # uint8 [rows][k/2], element 2j in the low nibble of byte j
    scales: np.ndarray         # float32 [rows][k/16] (FP32, POW2) or uint8 [rows][k/16] (E4M3_TENSOR)
    grid: int
    scale_fmt: int
    tensor_scale: float = 1.0
    y: np.ndarray | None = None  # normalised pre-rounding values, if requested

    @property
    def rows(self):
        return self.codes.shape[0]

    @property
    def k(self):
        return self.codes.shape[1] * 2


def levels(grid: int) -> np.ndarray:
    return np.array([lib().orc_level(grid, i) for i in range(8)])


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def rht_sign_mask(seed: int) -> int:
    return int(lib().orc_rht_sign_mask(seed))


def sr_bytes(seed_sr: int, block_index: int, variant: int) -> np.ndarray:
    r = np.zeros(16, dtype=np.uint8)
    lib().orc_sr_bytes(seed_sr, block_index, variant, _ptr(r))
    return r


def hadamard_matrix(n: int) -> np.ndarray:
    H = np.zeros((n, n), dtype=np.float64)
    lib().orc_hadamard_matrix(n, _ptr(H))
    return H


def rht16_f32(v, sign_mask: int) -> np.ndarray:
    a = np.ascontiguousarray(v, dtype=np.float32).copy()
    assert a.shape == (16,)
    lib().orc_rht16_f32(_ptr(a), sign_mask)
    return a


def rht_signs(seed: int) -> np.ndarray:
    """The 128 sign bits of a seed as four 32-bit words (bit i set: eps_i = -1)."""
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_rht_signs(seed, _ptr(out))
    return out


def rht_f32(v, n: int, signs: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(v, dtype=np.float32).copy()
    assert a.shape == (n,) and n in (32, 64, 128)
    s = np.ascontiguousarray(signs, dtype=np.uint32)
    lib().orc_rht_f32(_ptr(a), n, _ptr(s))
    return a


def round_rtne(a: float, grid: int) -> int:
    return int(lib().orc_round_rtne(float(a), grid))


def round_sr(a: float, grid: int, r: int) -> int:
    return int(lib().orc_round_sr(float(a), grid, int(r)))


def nibble_value(grid: int, nibble: int) -> float:
    return float(lib().orc_nibble_value(grid, nibble))


def e4m3_value(byte: int) -> float:
    return float(lib().orc_e4m3_value(byte))


def e4m3_encode(u: float) -> int:
    return int(lib().orc_e4m3_encode(float(u)))


def quantize(x_bf16_bits: np.ndarray, axis: int, rht_block: int = 16, grid: int = GRID_INT4,
             rounding: int = ROUND_RTNE, scale_fmt: int = SCALE_FP32, seed_rht: int = 0, seed_sr: int = 0,
             tensor_scale: float = 1.0, want_y: bool = False, window=None) -> QTensor:
    """window = (out_row0, kb0, full_nkb): x is a part of a larger tensor (see orc_quantize_window); only the SR draws
    depend on it."""
    x = np.ascontiguousarray(x_bf16_bits)
    assert x.dtype == np.uint16 and x.ndim == 2
    rows, cols = x.shape
    R, K = (rows, cols) if axis == AXIS_ROW else (cols, rows)
    assert K % 16 == 0
    codes = np.zeros((R, K // 2), dtype=np.uint8)
    scales = np.zeros((R, K // 16), dtype=np.uint8 if scale_fmt == SCALE_E4M3_TENSOR else np.float32)
    y = np.zeros((R, K), dtype=np.float32) if want_y else None
    out_row0, kb0, full_nkb = window if window is not None else (0, 0, K // 16)
    rc = lib().orc_quantize_window(_ptr(x), rows, cols, cols, axis, rht_block, grid, rounding, scale_fmt, seed_rht, seed_sr,
                                   tensor_scale, _ptr(codes), _ptr(scales), _ptr(y) if want_y else None,
                                   out_row0, kb0, full_nkb)
    if rc != 0:
        raise ValueError("orc_quantize rejected its arguments")
    return QTensor(codes, scales, grid, scale_fmt, float(np.float32(tensor_scale)), y)


def dequantize(q: QTensor, r0: int = 0, r1: int | None = None) -> np.ndarray:
    r1 = q.rows if r1 is None else r1
    out = np.zeros((r1 - r0, q.k), dtype=np.float64)
    lib().orc_dequantize(_ptr(q.codes), _ptr(q.scales), q.k, q.grid, q.scale_fmt, q.tensor_scale, r0, r1, _ptr(out))
    return out


def gemm_f64(A: np.ndarray, B: np.ndarray):
    """C = A Bᵀ and S = |A| |B|ᵀ for FP64 A[M][K], B[N][K] (plain triple loop)."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    Cm = np.zeros((M, N), dtype=np.float64)
    S = np.zeros((M, N), dtype=np.float64)
    lib().orc_gemm_f64(_ptr(A), _ptr(B), M, N, K, _ptr(Cm), _ptr(S))
    return Cm, S


def gemm(qa: QTensor, qb: QTensor):
    """The low-precision GEMM of Sec. 2.2 on dequantized operands, FP64: C[m][n] = sum_k a[m][k] b[n][k]."""
    assert qa.k == qb.k
    return gemm_f64(dequantize(qa), dequantize(qb))


def gemm_sampled(qa: QTensor, qb: QTensor, im, in_, k0: int = 0, k1: int | None = None):
    """C and S at the listed (m, n) pairs, reduction over [k0, k1)."""
    assert qa.k == qb.k
    k1 = qa.k if k1 is None else k1
    im = np.ascontiguousarray(im, dtype=np.int64)
    in_ = np.ascontiguousarray(in_, dtype=np.int64)
    c = np.zeros(im.shape[0], dtype=np.float64)
    s = np.zeros(im.shape[0], dtype=np.float64)
    lib().orc_gemm_sampled(_ptr(qa.codes), _ptr(qa.scales), qa.grid, qa.scale_fmt, qa.tensor_scale,
                           _ptr(qb.codes), _ptr(qb.scales), qb.grid, qb.scale_fmt, qb.tensor_scale,
                           qa.k, k0, k1, im.shape[0], _ptr(im), _ptr(in_), _ptr(c), _ptr(s))
    return c, s


def bin_bias(y: np.ndarray, codes: np.ndarray, grid: int):
    """Per non-negative level: (count, mean of level - |y|) in grid units (Sec. 3.1 restricted to each bin)."""
    y = np.ascontiguousarray(y, dtype=np.float32).reshape(-1)
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    assert codes.size * 2 == y.size
    count = np.zeros(8, dtype=np.int64)
    total = np.zeros(8, dtype=np.float64)
    lib().orc_bin_bias(_ptr(y), _ptr(codes), y.size, grid, _ptr(count), _ptr(total))
    with np.errstate(invalid="ignore", divide="ignore"):
        mean = np.where(count > 0, total / np.maximum(count, 1), np.nan)
    return count, mean


def diagnose(x_u16: np.ndarray, q: QTensor, rht_block: int, seed_rht: int) -> dict:
    """Tensor diagnostics of the row variant q of the BF16 matrix x (Eq. 3, Eq. 6, Eq. 7 ingredients, Sec. 3.1 bias):
    alpha, nmse, b_eff, count[8], bias[8] (mean of level - t per magnitude level, NaN where a level is unused)."""
    x = np.ascontiguousarray(x_u16, dtype=np.uint16)
    rows, cols = x.shape
    assert q.scale_fmt != SCALE_E4M3_TENSOR and q.codes.shape == (rows, cols // 2)
    codes = np.ascontiguousarray(q.codes, dtype=np.uint8)
    scales = np.ascontiguousarray(q.scales, dtype=np.float32)
    out = np.zeros(19, dtype=np.float64)
    lib().orc_diagnose(_ptr(x), rows, cols, cols, _ptr(codes), cols // 2, _ptr(scales), cols // 16, q.grid, rht_block,
                       seed_rht, _ptr(out))
    return diagnostics_from_sums(out)


def diagnostics_from_sums(out: np.ndarray) -> dict:
    """alpha (Eq. 3), NMSE (Sec. 3.3), B_eff (Eq. 6) and the per-level bias from the 19 raw sums of orc_diagnose."""
    count, bias_sum = out[3:11], out[11:19]
    with np.errstate(invalid="ignore", divide="ignore"):
        bias = np.where(count > 0, bias_sum / np.maximum(count, 1), np.nan)
        alpha = out[2] / out[0] if out[0] > 0 else float("nan")
        nmse = out[1] / out[0] if out[0] > 0 else float("nan")
    return {"alpha": float(alpha), "nmse": float(nmse), "b_eff": float(lib().orc_b_eff(_ptr(np.ascontiguousarray(count)))),
            "count": count.astype(np.int64), "bias": bias, "sums": out.copy()}
