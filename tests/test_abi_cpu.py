"""The C-ABI library loads without a GPU, exports every symbol include/ufp4.h declares, and its host-side checks
return the documented status codes without launching anything."""
import ctypes as C
import os
import re

import pytest

import oracle
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import build as ufp4_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ufp4_build.build()
    return ufp4.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ufp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ufp4_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "ufp4_quantize" in names and "ufp4_gemm" in names and "ufp4_gemm_grouped" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ufp4.EXPORTS) == [n for n in names]


def test_version_and_status_strings(lib):
    assert lib.ufp4_version() >= 100
    assert lib.ufp4_status_string(0) == b"ok"
    for code in range(-7, 0):
        assert len(lib.ufp4_status_string(code)) > 3
    assert lib.ufp4_status_string(-99) == b"unknown status"


def test_sign_mask_matches_oracle(lib):
    for seed in (0, 1, 2, 12345, 0xDEADBEEFCAFEF00D):
        assert ufp4.rht_sign_mask(seed) == oracle.rht_sign_mask(seed)


def test_wide_rht_signs_match_oracle(lib):
    for seed in (0, 1, 2, 12345, 0xDEADBEEFCAFEF00D):
        got = ufp4.rht_signs(seed)
        assert got == [int(v) for v in oracle.rht_signs(seed)] and got[0] & 0xFFFF == ufp4.rht_sign_mask(seed)


def test_qtensor_bytes(lib):
    cb, sb = C.c_size_t(), C.c_size_t()
    assert lib.ufp4_qtensor_bytes(100, 48, 0, C.byref(cb), C.byref(sb)) == 0
    assert cb.value == 100 * 32 and sb.value == 100 * 3 * 4          # 24 bytes of codes per row padded to 32
    assert lib.ufp4_qtensor_bytes(100, 48, 2, C.byref(cb), C.byref(sb)) == 0 and sb.value == 100 * 3
    assert lib.ufp4_qtensor_bytes(100, 40, 0, C.byref(cb), C.byref(sb)) == -2
    assert lib.ufp4_qtensor_bytes(100, 48, 7, C.byref(cb), C.byref(sb)) == -4
    assert lib.ufp4_qtensor_bytes(100, 48, 0, None, C.byref(sb)) == -1


def _q(rows, k, codes=0x1000, scales=0x2000, grid=0, fmt=0, ld=None, lds=None):
    return ufp4._QTensorStruct(codes, scales, None, rows, k, ld if ld is not None else (k // 2 + 15) // 16 * 16,
                               lds if lds is not None else k // 16, grid, fmt)


def test_quantize_rejects_bad_arguments_without_launching(lib):
    q = lib.ufp4_quantize
    row, col = _q(32, 64), _q(64, 32)
    x = 0x10000
    ok_args = dict(rows=32, cols=64, ld=64, axis=2, rht=16, grid=0, rnd=0, fmt=0)

    def call(x=x, row=row, col=col, **kw):
        a = dict(ok_args, **kw)
        return q(x, a["rows"], a["cols"], a["ld"], a["axis"], a["rht"], a["grid"], a["rnd"], a["fmt"], 1, 2,
                 C.byref(row) if row is not None else None, C.byref(col) if col is not None else None, None, None)

    assert call(x=None) == -1
    assert call(row=None) == -1
    assert call(col=None) == -1
    assert call(axis=5) == -4 and call(grid=5) == -4 and call(rnd=2) == -4 and call(fmt=9) == -4
    assert call(rht=48) == -5 and call(rht=128) == -2   # unknown block size; reduction dimensions not multiples of 128
    assert call(cols=40, ld=40) == -2                    # cols % 16
    assert call(rows=40) == -2                           # rows % 16 for the col variant
    assert call(x=x + 2) == -3 and call(ld=68) == -3     # 16-byte alignment of x and its rows
    assert call(row=_q(32, 48)) == -2                    # output shape does not match the call
    assert call(row=_q(32, 64, grid=1)) == -2
    assert call(row=_q(32, 64, ld=24)) == -3
    assert call(row=_q(32, 64, fmt=2), col=_q(64, 32, fmt=2), fmt=2) == -1   # E4M3_TENSOR without a tensor scale


def test_gemm_rejects_bad_arguments_without_launching(lib):
    A, B = _q(64, 128), _q(32, 128)
    g = lib.ufp4_gemm
    assert g(None, C.byref(B), 0x4000, 32, 0, 0, 0, None, 0, None, None) == -1
    assert g(C.byref(A), C.byref(B), None, 32, 0, 0, 0, None, 0, None, None) == -1
    assert g(C.byref(A), C.byref(_q(32, 64)), 0x4000, 32, 0, 0, 0, None, 0, None, None) == -2   # K mismatch
    assert g(C.byref(A), C.byref(B), 0x4000, 16, 0, 0, 0, None, 0, None, None) == -2           # ldc < N
    assert g(C.byref(A), C.byref(B), 0x4004, 32, 0, 0, 0, None, 0, None, None) == -3
    assert g(C.byref(A), C.byref(B), 0x4000, 32, 0, 9, 0, None, 0, None, None) == -4
    assert g(C.byref(A), C.byref(B), 0x4000, 32, 0, 0, 9, None, 0, None, None) == -4
    assert g(C.byref(_q(64, 120)), C.byref(_q(32, 120)), 0x4000, 32, 0, 0, 0, None, 0, None, None) == -2
    # the tensor-core path is only defined for power-of-two scales
    assert g(C.byref(A), C.byref(B), 0x4000, 32, 0, 0, 2, None, 0, None, None) == -5   # FP32 scales
    assert lib.ufp4_gemm_workspace_bytes(C.byref(A), C.byref(B), 1) == 0


def test_grouped_gemm_checks_offsets_on_the_host(lib):
    gg = lib.ufp4_gemm_grouped
    A, B = _q(256, 64), _q(2 * 32, 64)
    off = (C.c_int64 * 3)(0, 128, 256)
    bad = (C.c_int64 * 3)(0, 100, 256)
    dec = (C.c_int64 * 3)(0, 256, 128)
    short = (C.c_int64 * 3)(0, 128, 128)
    args = lambda o: (C.byref(A), C.byref(B), 0x4000, 32, 0, 0, 1, 0x8000, C.cast(o, C.c_void_p), 2, 32, None, 0, None, None)
    assert gg(*args(bad)) == -2 and gg(*args(dec)) == -2 and gg(*args(short)) == -2
    assert gg(C.byref(A), C.byref(B), 0x4000, 32, 0, 0, 1, None, C.cast(off, C.c_void_p), 2, 32, None, 0, None, None) == -1
    assert gg(C.byref(A), C.byref(_q(3 * 32, 64)), 0x4000, 32, 0, 0, 1, 0x8000, C.cast(off, C.c_void_p), 2, 32, None, 0,
              None, None) == -2


def test_diagnose_ratios_is_host_arithmetic_and_matches_the_oracle(lib):
    """ufp4_diagnose_ratios turns the 19 sums into alpha, NMSE, B_eff and the per-level bias on the host; the same
    numbers from the oracle's own formulae."""
    import numpy as np
    sums = np.array([200.0, 3.0, 198.0, 10, 20, 30, 40, 0, 60, 70, 80, -2.5, 0.5, 0.25, -0.125, 0.0, 1.0, -1.0, 4.0])
    got = ufp4.diagnose_ratios(sums.tolist())
    want = oracle.diagnostics_from_sums(sums)
    assert got[0] == pytest.approx(want["alpha"], rel=1e-15) and got[1] == pytest.approx(want["nmse"], rel=1e-15)
    assert got[2] == pytest.approx(want["b_eff"], rel=1e-12)
    assert np.isnan(got[3 + 4]) and np.isnan(want["bias"][4])
    keep = [i for i in range(8) if i != 4]
    assert np.allclose(np.array(got[3:])[keep], want["bias"][keep], rtol=1e-15)
    zero = ufp4.diagnose_ratios([0.0] * 19)
    assert np.isnan(zero[0]) and np.isnan(zero[1]) and zero[2] == pytest.approx(1.0 / 8.0)
    assert lib.ufp4_diagnose_ratios(None, None) == -1


def test_path_selection_and_workspace_sizes_are_host_decisions(lib):
    """ufp4_gemm_path_taken and ufp4_gemm_workspace_bytes read the operand descriptions only: which path each scale format
    takes by default, which requests are refused, and that the workspace of a path matches what that path lays out."""
    AUTO, EXACT, TENSOR, PROMOTE, SPLIT, FP16, MX, NVF4 = range(8)
    taken, ws = lib.ufp4_gemm_path_taken, lib.ufp4_gemm_workspace_bytes
    ws.restype = C.c_size_t

    def q(fmt, grid=0, rows=256, k=512):
        t = _q(rows, k, grid=grid, fmt=fmt)
        if fmt == 2:
            t.tensor_scale = 0x3000            # E4M3 x tensor scale: any non-null device address will do for a host decision
        return t
    n = C.c_int(0)
    for fmt, want, launches in ((0, SPLIT, 2), (1, TENSOR, 2), (3, TENSOR, 2), (2, NVF4, 2)):
        a, b = q(fmt), q(fmt, rows=128)
        assert taken(C.byref(a), C.byref(b), AUTO, C.byref(n)) == want and n.value == launches
        assert ws(C.byref(a), C.byref(b), AUTO) >= ws(C.byref(a), C.byref(b), want) > 0
    assert taken(C.byref(q(1)), C.byref(q(1)), EXACT, C.byref(n)) == EXACT and n.value == 1
    # on-request paths and the formats they refuse
    assert taken(C.byref(q(1)), C.byref(q(3)), MX, None) == MX and taken(C.byref(q(0)), C.byref(q(1)), MX, None) == -5
    assert taken(C.byref(q(2)), C.byref(q(2)), FP16, None) == FP16 and taken(C.byref(q(1)), C.byref(q(1)), FP16, None) == -5
    assert taken(C.byref(q(2)), C.byref(q(1)), NVF4, None) == -5 and taken(C.byref(q(0)), C.byref(q(0)), TENSOR, None) == -5
    assert taken(C.byref(q(1)), C.byref(q(1)), 8, None) == -4
    assert taken(C.byref(q(1)), C.byref(q(1, k=256)), AUTO, None) == -2
    # MX: one operand byte per element plus one 512-byte scale unit per (128 rows padded to 256, 128 elements of K)
    a, b = q(1, rows=300, k=512), q(1, rows=128, k=512)
    assert ws(C.byref(a), C.byref(b), MX) == 300 * 512 + 128 * 512 + (4 + 2) * 4 * 512
    # NVF4: two half-byte planes per uniform operand, none for an E2M1 tensor, plus one scale unit per 64 elements of K
    au, be = q(2, grid=0, rows=256, k=512), q(2, grid=2, rows=256, k=512)
    units = 2 * 2 * 4 * 512                     # per operand: 2 stages of K x 2 row tiles x 4 steps
    assert ws(C.byref(au), C.byref(au), NVF4) == 4 * 256 * 256 + 2 * units
    assert ws(C.byref(be), C.byref(be), NVF4) == 2 * units
    assert ws(C.byref(au), C.byref(be), NVF4) == 2 * 256 * 256 + 2 * units


def test_quantize_multi_rejects_bad_argument_sets_without_launching(lib):
    qm = lib.ufp4_quantize_multi
    row, col = _q(32, 64), _q(64, 32)
    ok = ufp4._QuantizeArgs(0x10000, 32, 64, 64, 2, 16, 0, 0, 0, 0, 1, 2, C.pointer(row), C.pointer(col))
    bad_axis = ufp4._QuantizeArgs(0x10000, 32, 64, 64, 5, 16, 0, 0, 0, 0, 1, 2, C.pointer(row), C.pointer(col))
    bad_shape = ufp4._QuantizeArgs(0x10000, 32, 40, 40, 2, 16, 0, 0, 0, 0, 1, 2, C.pointer(row), C.pointer(col))
    assert qm(0, None, None, None) == 0
    assert qm(1, None, None, None) == -1 and qm(-1, None, None, None) == -2
    arr = (ufp4._QuantizeArgs * 2)(ok, bad_axis)
    assert qm(2, arr, None, None) == -4                       # the second set is wrong: reported before anything is launched
    arr = (ufp4._QuantizeArgs * 2)(bad_shape, ok)
    assert qm(2, arr, None, None) == -2
