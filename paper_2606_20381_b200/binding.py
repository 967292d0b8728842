"""ctypes binding of libufp4.so (declared in include/ufp4.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch supplies device
memory and streams.  There is no CPU fallback; if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

GRID_INT4, GRID_E1M2, GRID_E2M1 = 0, 1, 2
GRID_E2M1_MAX4, GRID_E2M1_MAX2 = 3, 4      # range-restricted E2M1 (Sec. 5.4, max_fpx = 4 / 2): quantizer-side only
ROUND_RTNE, ROUND_SR = 0, 1
AXIS_ROW, AXIS_COL, AXIS_BOTH = 0, 1, 2
SCALE_FP32, SCALE_POW2, SCALE_E4M3_TENSOR = 0, 1, 2
SCALE_E8M0_B32 = 3      # one power-of-two scale per 32 elements (MXFP4's block layout), read by the GEMMs like POW2
FWD_Y, BWD_DX, BWD_DW = 0, 1, 2
PATH_AUTO, PATH_EXACT, PATH_TENSOR, PATH_PROMOTE, PATH_SPLIT, PATH_FP16, PATH_MX, PATH_NVF4 = 0, 1, 2, 3, 4, 5, 6, 7
DEV_NONFINITE, DEV_EXP_WINDOW, DEV_WAIT_TIMEOUT = 1, 2, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libufp4.so")

EXPORTS = ["ufp4_version", "ufp4_status_string", "ufp4_rht_sign_mask", "ufp4_rht_signs", "ufp4_qtensor_bytes", "ufp4_quantize",
           "ufp4_quantize_batched", "ufp4_selftest_division", "ufp4_gemm_workspace_bytes", "ufp4_gemm_path_taken", "ufp4_gemm", "ufp4_gemm_grouped",
           "ufp4_gemm_noalloc", "ufp4_gemm_noalloc_max_scratch_bytes", "ufp4_diagnose", "ufp4_diagnose_workspace_bytes",
           "ufp4_diagnose_ratios", "ufp4_debug_wait_injection", "ufp4_gemm_quantized",
           "ufp4_probe_issue_rates", "ufp4_probe_decode_rate", "ufp4_quantize_multi"]


class _QTensorStruct(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("tensor_scale", C.c_void_p),
                ("rows", C.c_int64), ("k", C.c_int64), ("ld_codes_bytes", C.c_int64), ("ld_scales", C.c_int64),
                ("grid", C.c_int32), ("scale_fmt", C.c_int32)]


class _QuantizeArgs(C.Structure):
    _fields_ = [("x", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("axis", C.c_int32), ("rht_block", C.c_int32), ("grid", C.c_int32), ("rounding", C.c_int32),
                ("scale_fmt", C.c_int32), ("reserved", C.c_int32), ("seed_rht", C.c_uint64), ("seed_sr", C.c_uint64),
                ("out_row", C.POINTER(_QTensorStruct)), ("out_col", C.POINTER(_QTensorStruct))]


_lib = None


def lib():
    """Load libufp4.so (once).  Raises if it has not been built: there is no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_20381_b200.build` "
                               "(the UFP4 path has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i64, u64, i32, sz = C.c_void_p, C.c_int64, C.c_uint64, C.c_int, C.c_size_t
        qp = C.POINTER(_QTensorStruct)
        L.ufp4_version.restype = i32
        L.ufp4_version.argtypes = []
        L.ufp4_status_string.restype = C.c_char_p
        L.ufp4_status_string.argtypes = [i32]
        L.ufp4_rht_sign_mask.restype = C.c_uint32
        L.ufp4_rht_sign_mask.argtypes = [u64]
        L.ufp4_rht_signs.restype = None
        L.ufp4_rht_signs.argtypes = [u64, C.POINTER(C.c_uint32)]
        L.ufp4_qtensor_bytes.restype = i32
        L.ufp4_qtensor_bytes.argtypes = [i64, i64, i32, C.POINTER(sz), C.POINTER(sz)]
        L.ufp4_quantize.restype = i32
        L.ufp4_quantize.argtypes = [vp, i64, i64, i64, i32, i32, i32, i32, i32, u64, u64, qp, qp, vp, vp]
        L.ufp4_quantize_batched.restype = i32
        L.ufp4_quantize_batched.argtypes = [vp, i64, i64, i64, i64, i64, i32, i32, i32, i32, i32, u64, u64, qp, qp, vp, vp]
        L.ufp4_selftest_division.restype = i32
        L.ufp4_selftest_division.argtypes = [vp, vp]
        L.ufp4_gemm_workspace_bytes.restype = sz
        L.ufp4_gemm_workspace_bytes.argtypes = [qp, qp, i32]
        L.ufp4_gemm_path_taken.restype = i32
        L.ufp4_gemm_path_taken.argtypes = [qp, qp, i32, C.POINTER(i32)]
        L.ufp4_gemm.restype = i32
        L.ufp4_gemm.argtypes = [qp, qp, vp, i64, i32, i32, i32, vp, sz, vp, vp]
        L.ufp4_gemm_grouped.restype = i32
        L.ufp4_gemm_grouped.argtypes = [qp, qp, vp, i64, i32, i32, i32, vp, vp, i32, i64, vp, sz, vp, vp]
        L.ufp4_gemm_noalloc.restype = i32
        L.ufp4_gemm_noalloc.argtypes = [qp, qp, vp, i64, i32, vp, vp]
        L.ufp4_gemm_noalloc_max_scratch_bytes.restype = sz
        L.ufp4_gemm_noalloc_max_scratch_bytes.argtypes = []
        L.ufp4_diagnose_workspace_bytes.restype = sz
        L.ufp4_diagnose_workspace_bytes.argtypes = [i64, i64]
        L.ufp4_diagnose.restype = i32
        L.ufp4_diagnose.argtypes = [vp, i64, i64, i64, qp, i32, u64, vp, vp, sz, vp]
        L.ufp4_gemm_quantized.restype = i32
        L.ufp4_gemm_quantized.argtypes = [qp, qp, vp, i64, i32, u64, qp, qp, vp, sz, vp, vp]
        L.ufp4_probe_issue_rates.restype = i32
        L.ufp4_probe_issue_rates.argtypes = [vp, sz, C.POINTER(C.c_double), vp]
        L.ufp4_quantize_multi.restype = i32
        L.ufp4_quantize_multi.argtypes = [i32, C.POINTER(_QuantizeArgs), vp, vp]
        L.ufp4_probe_decode_rate.restype = i32
        L.ufp4_probe_decode_rate.argtypes = [vp, sz, C.POINTER(C.c_double), vp]
        L.ufp4_debug_wait_injection.restype = i32
        L.ufp4_debug_wait_injection.argtypes = [C.c_uint32, i32]
        L.ufp4_diagnose_ratios.restype = i32
        L.ufp4_diagnose_ratios.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double)]
        _lib = L
    return _lib


class Ufp4Error(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"libufp4 status {status}: {lib().ufp4_status_string(status).decode()}")


def _check(status: int):
    if status != 0:
        raise Ufp4Error(status)


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


@dataclass
class QTensor:
    """A quantized tensor on the device: logical [rows][k], k the reduction dimension."""
    codes: torch.Tensor                     # uint8 [rows][ld_codes_bytes]
    scales: torch.Tensor                    # float32 or uint8 [rows][k/16]
    grid: int
    scale_fmt: int
    k: int
    tensor_scale: torch.Tensor | None = None   # float32 [1] on the device (E4M3_TENSOR only)

    @property
    def rows(self) -> int:
        return self.codes.shape[0]

    def struct(self) -> _QTensorStruct:
        return _QTensorStruct(self.codes.data_ptr(), self.scales.data_ptr(),
                              self.tensor_scale.data_ptr() if self.tensor_scale is not None else None,
                              self.rows, self.k, self.codes.stride(0), self.scales.stride(0), self.grid, self.scale_fmt)

    def packed_codes(self) -> torch.Tensor:
        """uint8 [rows][k/2] view without row padding."""
        return self.codes[:, : self.k // 2]

    def row_slice(self, r0: int, r1: int) -> "QTensor":
        return QTensor(self.codes[r0:r1], self.scales[r0:r1], self.grid, self.scale_fmt, self.k, self.tensor_scale)


def rht_sign_mask(seed: int) -> int:
    return int(lib().ufp4_rht_sign_mask(seed))


def rht_signs(seed: int) -> list:
    """The 128 sign bits of the wider RHT blocks as four 32-bit words."""
    out = (C.c_uint32 * 4)()
    lib().ufp4_rht_signs(seed, out)
    return [int(v) for v in out]


def alloc_qtensor(rows: int, k: int, grid: int, scale_fmt: int, device, tensor_scale=None) -> QTensor:
    cb, sb = C.c_size_t(), C.c_size_t()
    _check(lib().ufp4_qtensor_bytes(rows, k, scale_fmt, C.byref(cb), C.byref(sb)))
    ld = cb.value // rows
    codes = torch.empty(rows, ld, dtype=torch.uint8, device=device)
    sdt = torch.uint8 if scale_fmt == SCALE_E4M3_TENSOR else torch.float32
    scales = torch.empty(rows, k // 16, dtype=sdt, device=device)
    ts = None
    if scale_fmt == SCALE_E4M3_TENSOR:
        if tensor_scale is None:
            raise ValueError("E4M3_TENSOR needs a tensor_scale")
        ts = tensor_scale if isinstance(tensor_scale, torch.Tensor) else torch.tensor(
            [tensor_scale], dtype=torch.float32, device=device)
    return QTensor(codes, scales, grid, scale_fmt, k, ts)


def quantize(x: torch.Tensor, axis: int = AXIS_BOTH, rht_block: int = 16, grid: int = GRID_INT4,
             rounding: int = ROUND_RTNE, scale_fmt: int = SCALE_FP32, seed_rht: int = 0, seed_sr: int = 0,
             tensor_scale=None, out_row: QTensor | None = None, out_col: QTensor | None = None,
             dev_status: torch.Tensor | None = None, stream=None):
    """ufp4_quantize on a BF16 CUDA matrix [rows][cols]; returns (row variant or None, col variant or None)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    if axis != AXIS_COL and out_row is None:
        out_row = alloc_qtensor(rows, cols, grid, scale_fmt, x.device, tensor_scale)
    if axis != AXIS_ROW and out_col is None:
        out_col = alloc_qtensor(cols, rows, grid, scale_fmt, x.device, tensor_scale)
    sr = out_row.struct() if axis != AXIS_COL else None
    sc = out_col.struct() if axis != AXIS_ROW else None
    _check(lib().ufp4_quantize(x.data_ptr(), rows, cols, x.stride(0), axis, rht_block, grid, rounding, scale_fmt,
                               seed_rht, seed_sr, C.byref(sr) if sr is not None else None,
                               C.byref(sc) if sc is not None else None,
                               dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return (out_row if axis != AXIS_COL else None), (out_col if axis != AXIS_ROW else None)


def quantize_multi(items, dev_status: torch.Tensor | None = None, stream=None):
    """ufp4_quantize_multi: several INDEPENDENT tensors in one call (see include/ufp4.h).  items: dicts with the keyword
    arguments of quantize() (x, axis, rht_block, grid, rounding, scale_fmt, seed_rht, seed_sr, tensor_scale, out_row,
    out_col); outputs not given are allocated.  Returns the list of (row variant or None, col variant or None)."""
    n = len(items)
    arr, keep, outs = (_QuantizeArgs * max(n, 1))(), [], []
    for i, it in enumerate(items):
        x = it["x"]
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
        rows, cols = x.shape
        axis, grid, fmt = it.get("axis", AXIS_BOTH), it.get("grid", GRID_INT4), it.get("scale_fmt", SCALE_FP32)
        out_row, out_col = it.get("out_row"), it.get("out_col")
        if axis != AXIS_COL and out_row is None:
            out_row = alloc_qtensor(rows, cols, grid, fmt, x.device, it.get("tensor_scale"))
        if axis != AXIS_ROW and out_col is None:
            out_col = alloc_qtensor(cols, rows, grid, fmt, x.device, it.get("tensor_scale"))
        sr = out_row.struct() if axis != AXIS_COL else None
        sc = out_col.struct() if axis != AXIS_ROW else None
        keep.append((sr, sc))
        arr[i] = _QuantizeArgs(x.data_ptr(), rows, cols, x.stride(0), axis, it.get("rht_block", 16), grid,
                               it.get("rounding", ROUND_RTNE), fmt, 0, it.get("seed_rht", 0), it.get("seed_sr", 0),
                               C.pointer(sr) if sr is not None else None, C.pointer(sc) if sc is not None else None)
        outs.append(((out_row if axis != AXIS_COL else None), (out_col if axis != AXIS_ROW else None)))
    _check(lib().ufp4_quantize_multi(n, arr, dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return outs


def quantize_batched(x: torch.Tensor, axis: int = AXIS_BOTH, rht_block: int = 16, grid: int = GRID_INT4,
                     rounding: int = ROUND_RTNE, scale_fmt: int = SCALE_FP32, seed_rht: int = 0, seed_sr: int = 0,
                     tensor_scale=None, out_row: QTensor | None = None, out_col: QTensor | None = None,
                     dev_status: torch.Tensor | None = None, stream=None):
    """ufp4_quantize_batched on a BF16 CUDA tensor [batch][rows][cols]; outputs stacked along rows."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 3 and x.stride(2) == 1
    batch, rows, cols = x.shape
    if axis != AXIS_COL and out_row is None:
        out_row = alloc_qtensor(batch * rows, cols, grid, scale_fmt, x.device, tensor_scale)
    if axis != AXIS_ROW and out_col is None:
        out_col = alloc_qtensor(batch * cols, rows, grid, scale_fmt, x.device, tensor_scale)
    sr = out_row.struct() if axis != AXIS_COL else None
    sc = out_col.struct() if axis != AXIS_ROW else None
    _check(lib().ufp4_quantize_batched(x.data_ptr(), batch, x.stride(0), rows, cols, x.stride(1), axis, rht_block, grid,
                                       rounding, scale_fmt, seed_rht, seed_sr,
                                       C.byref(sr) if sr is not None else None,
                                       C.byref(sc) if sc is not None else None,
                                       dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return (out_row if axis != AXIS_COL else None), (out_col if axis != AXIS_ROW else None)


def selftest_division(stream=None) -> int:
    """Number of FP32 inputs for which the quantizer's division shortcuts differ from the IEEE division (expected 0)."""
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().ufp4_selftest_division(n.data_ptr(), _stream_ptr(stream)))
    return int(n.item())


def diagnose(x: torch.Tensor, q_row: QTensor, rht_block: int = 16, seed_rht: int = 0, stream=None) -> torch.Tensor:
    """ufp4_diagnose: the 19 raw sums (device, float64) for the BF16 matrix x and its row variant q_row."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    out = torch.empty(19, dtype=torch.float64, device=x.device)
    ws = torch.empty(lib().ufp4_diagnose_workspace_bytes(rows, cols), dtype=torch.uint8, device=x.device)
    s = q_row.struct()
    _check(lib().ufp4_diagnose(x.data_ptr(), rows, cols, x.stride(0), C.byref(s), rht_block, seed_rht, out.data_ptr(),
                               ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
    return out


def gemm_quantized(A: QTensor, B: QTensor, rht_block: int = 16, seed_rht: int = 0, scale_fmt: int = SCALE_FP32,
                   want_row: bool = True, want_col: bool = True, want_c: bool = False, out_row: QTensor | None = None,
                   out_col: QTensor | None = None, out_c: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                   dev_status: torch.Tensor | None = None, stream=None):
    """ufp4_gemm_quantized: returns (row layout [M][N] or None, col layout [N][M] or None, BF16 C or None)."""
    M, N = A.rows, B.rows
    dev = A.codes.device
    if want_row and out_row is None:
        out_row = alloc_qtensor(M, N, GRID_INT4, scale_fmt, dev)
    if want_col and out_col is None:
        out_col = alloc_qtensor(N, M, GRID_INT4, scale_fmt, dev)
    if want_c and out_c is None:
        out_c = _alloc_out(M, N, True, dev)
    if workspace is None:
        workspace = torch.empty(max(16, gemm_workspace_bytes(A, B, PATH_TENSOR)), dtype=torch.uint8, device=dev)
    sa, sb = A.struct(), B.struct()
    sr = out_row.struct() if out_row is not None else None
    sc = out_col.struct() if out_col is not None else None
    _check(lib().ufp4_gemm_quantized(C.byref(sa), C.byref(sb), out_c.data_ptr() if out_c is not None else None,
                                     out_c.stride(0) if out_c is not None else N, rht_block, seed_rht,
                                     C.byref(sr) if sr is not None else None, C.byref(sc) if sc is not None else None,
                                     workspace.data_ptr(), workspace.numel(),
                                     dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return out_row, out_col, out_c


def probe_issue_rates(stream=None) -> dict:
    """ufp4_probe_issue_rates: cycles per scheduler and group of warp instructions (see include/ufp4.h)."""
    scratch = torch.empty(256 * 4096 + 256, dtype=torch.uint8, device="cuda")
    out = (C.c_double * 8)()
    _check(lib().ufp4_probe_issue_rates(scratch.data_ptr(), scratch.numel(), out, _stream_ptr(stream)))
    names = ["add.f32x2", "add.f32, add.f32", "lop3", "mad.lo", "add.f32x2, lop3", "add.f32x2, mad.lo",
             "add.f32x2, lop3, lop3", "add.f32, add.f32, lop3"]
    return {n: float(v) for n, v in zip(names, out)}


def probe_decode_rate(stream=None) -> dict:
    """ufp4_probe_decode_rate: cycles per 32768-element stage decoded in shared memory by 128 / 256 / 512 / 1024 threads of
    one CTA per SM, and the elements per cycle that makes (see include/ufp4.h)."""
    scratch = torch.empty(256 * 4096 + 256, dtype=torch.uint8, device="cuda")
    out = (C.c_double * 4)()
    _check(lib().ufp4_probe_decode_rate(scratch.data_ptr(), scratch.numel(), out, _stream_ptr(stream)))
    return {f"{t}_threads": {"cycles_per_stage": float(v), "elements_per_cycle": 32768.0 / float(v)}
            for t, v in zip((128, 256, 512, 1024), out)}


def debug_wait_injection(poll_limit: int = 0, skip_loads: bool = False):
    """ufp4_debug_wait_injection: test hook, see include/ufp4.h.  Reset with debug_wait_injection()."""
    _check(lib().ufp4_debug_wait_injection(poll_limit, 1 if skip_loads else 0))


def diagnose_ratios(sums) -> list:
    """ufp4_diagnose_ratios: [alpha, nmse, b_eff, bias of level 0..7] from the 19 sums (any host sequence of floats)."""
    a = (C.c_double * 19)(*[float(v) for v in sums])
    out = (C.c_double * 11)()
    _check(lib().ufp4_diagnose_ratios(a, out))
    return [float(v) for v in out]


def gemm_workspace_bytes(A: QTensor, B: QTensor, path: int = PATH_AUTO) -> int:
    sa, sb = A.struct(), B.struct()
    return int(lib().ufp4_gemm_workspace_bytes(C.byref(sa), C.byref(sb), path))


def gemm_path_taken(A: QTensor, B: QTensor, path: int = PATH_AUTO):
    """(path the library would take, kernels one call launches)."""
    sa, sb, n = A.struct(), B.struct(), C.c_int(0)
    rc = lib().ufp4_gemm_path_taken(C.byref(sa), C.byref(sb), path, C.byref(n))
    if rc < 0:
        raise Ufp4Error(rc)
    return rc, n.value


def gemm_launch_count(A: QTensor, B: QTensor, path: int = PATH_AUTO) -> int:
    return gemm_path_taken(A, B, path)[1]


def gemm_path_name(A: QTensor, B: QTensor, path: int = PATH_AUTO) -> str:
    return {PATH_EXACT: "exact", PATH_TENSOR: "tensor", PATH_PROMOTE: "promote", PATH_SPLIT: "split", PATH_FP16: "fp16", PATH_MX: "mx", PATH_NVF4: "nvf4"}[gemm_path_taken(A, B, path)[0]]


def _alloc_out(rows: int, cols: int, bf16: bool, device) -> torch.Tensor:
    """[rows][cols] output whose rows start on 16-byte boundaries (the row pitch is padded if cols is odd-sized)."""
    per16 = 8 if bf16 else 4
    ld = (cols + per16 - 1) // per16 * per16
    buf = torch.empty(rows, ld, dtype=torch.bfloat16 if bf16 else torch.float32, device=device)
    return buf[:, :cols]


def _workspace(A, B, path, workspace):
    need = gemm_workspace_bytes(A, B, path)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=A.codes.device)
    return workspace


def gemm(A: QTensor, B: QTensor, out: torch.Tensor | None = None, out_bf16: bool = False, layout: int = FWD_Y,
         path: int = PATH_AUTO, workspace: torch.Tensor | None = None, dev_status: torch.Tensor | None = None,
         stream=None) -> torch.Tensor:
    """ufp4_gemm: C[m][n] = sum_k a[m][k] b[n][k] for quantized A [M][K], B [N][K]."""
    if out is None:
        out = _alloc_out(A.rows, B.rows, out_bf16, A.codes.device)
    assert out.is_cuda and out.stride(1) == 1
    workspace = _workspace(A, B, path, workspace)
    sa, sb = A.struct(), B.struct()
    _check(lib().ufp4_gemm(C.byref(sa), C.byref(sb), out.data_ptr(), out.stride(0), int(out.dtype == torch.bfloat16),
                           layout, path, workspace.data_ptr() if workspace is not None else None,
                           workspace.numel() if workspace is not None else 0,
                           dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return out


def gemm_grouped(A: QTensor, B: QTensor, offsets_dev: torch.Tensor, offsets_host: torch.Tensor, group_n: int,
                 layout: int, out: torch.Tensor | None = None, out_bf16: bool = False, path: int = PATH_AUTO,
                 workspace: torch.Tensor | None = None, dev_status: torch.Tensor | None = None,
                 stream=None) -> torch.Tensor:
    """ufp4_gemm_grouped (see include/ufp4.h for the operand layouts of each product)."""
    assert offsets_dev.is_cuda and offsets_dev.dtype == torch.int64 and offsets_dev.is_contiguous()
    assert (not offsets_host.is_cuda) and offsets_host.dtype == torch.int64 and offsets_host.is_contiguous()
    G = offsets_host.numel() - 1
    if out is None:
        if layout == BWD_DW:
            out = _alloc_out(G * A.rows, B.rows, out_bf16, A.codes.device)
        else:
            out = _alloc_out(A.rows, group_n, out_bf16, A.codes.device)
    workspace = _workspace(A, B, path, workspace)
    sa, sb = A.struct(), B.struct()
    _check(lib().ufp4_gemm_grouped(C.byref(sa), C.byref(sb), out.data_ptr(), out.stride(0),
                                   int(out.dtype == torch.bfloat16), layout, path, offsets_dev.data_ptr(),
                                   offsets_host.data_ptr(), G, group_n,
                                   workspace.data_ptr() if workspace is not None else None,
                                   workspace.numel() if workspace is not None else 0,
                                   dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return out


def gemm_noalloc_max_scratch_bytes() -> int:
    return int(lib().ufp4_gemm_noalloc_max_scratch_bytes())


def gemm_noalloc(A: QTensor, B: QTensor, out: torch.Tensor, dev_status: torch.Tensor | None = None, stream=None):
    """ufp4_gemm_noalloc: the tensor-core GEMM with its scratch in the library's fixed device array.

    For callers that may not allocate device memory (all of it already belongs to a pool, or an allocation would stall
    the device at this point): `out` must be preallocated by the caller, and this wrapper allocates nothing either.
    Calls share one scratch array, so keep them on one stream.  Shapes whose scratch exceeds
    gemm_noalloc_max_scratch_bytes() raise Ufp4Error (workspace)."""
    assert out.is_cuda and out.stride(1) == 1
    sa, sb = A.struct(), B.struct()
    _check(lib().ufp4_gemm_noalloc(C.byref(sa), C.byref(sb), out.data_ptr(), out.stride(0),
                                   int(out.dtype == torch.bfloat16),
                                   dev_status.data_ptr() if dev_status is not None else None, _stream_ptr(stream)))
    return out
