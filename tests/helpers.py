"""Shared helpers of the parity tests: moving tensors between the oracle (numpy) and the CUDA binding (torch)."""
import numpy as np
import torch

import oracle
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200.inputs import bf16_bits


def oracle_quantize(x: torch.Tensor, axis, **kw) -> oracle.QTensor:
    """Quantize a BF16 torch tensor (any device) with the CPU oracle."""
    return oracle.quantize(bf16_bits(x), axis, **kw)


def assert_qtensor_equal(gpu: ufp4.QTensor, ref: oracle.QTensor, what=""):
    """Bit-exact comparison of codes and scales."""
    assert gpu.rows == ref.rows and gpu.k == ref.k, what
    codes = gpu.packed_codes().cpu().numpy()
    if not np.array_equal(codes, ref.codes):
        bad = np.argwhere(codes != ref.codes)
        r, c = bad[0]
        raise AssertionError(f"{what}: {len(bad)} code bytes differ, first at row {r} byte {c}: "
                             f"gpu {codes[r, c]:#04x} oracle {ref.codes[r, c]:#04x}")
    scales = gpu.scales.cpu().numpy()
    if scales.dtype == np.float32:
        same = scales.view(np.uint32) == ref.scales.view(np.uint32)
    else:
        same = scales == ref.scales
    if not np.all(same):
        bad = np.argwhere(~same)
        r, c = bad[0]
        raise AssertionError(f"{what}: {len(bad)} scales differ, first at row {r} block {c}: "
                             f"gpu {scales[r, c]!r} oracle {ref.scales[r, c]!r}")


def to_device(q: oracle.QTensor, device="cuda") -> ufp4.QTensor:
    """Upload an oracle-quantized tensor as a binding QTensor (codes rows padded to 16 bytes)."""
    rows, kb2 = q.codes.shape
    ld = (kb2 + 15) // 16 * 16
    codes = torch.zeros(rows, ld, dtype=torch.uint8, device=device)
    codes[:, :kb2] = torch.from_numpy(q.codes).to(device)
    scales = torch.from_numpy(q.scales).to(device)
    ts = None
    if q.scale_fmt == oracle.SCALE_E4M3_TENSOR:
        ts = torch.tensor([q.tensor_scale], dtype=torch.float32, device=device)
    return ufp4.QTensor(codes, scales, q.grid, q.scale_fmt, q.k, ts)


GEMM_RTOL = 1e-5    # |C_gpu - C_oracle| <= GEMM_RTOL * sum_k |a_k b_k| per element


def assert_gemm_close(c_gpu: np.ndarray, c_ref: np.ndarray, s_ref: np.ndarray, what="", bf16_out=False):
    tol = GEMM_RTOL * s_ref + 1e-300
    if bf16_out:
        tol = tol + 2.0 ** -8 * np.abs(c_ref)      # BF16 output rounding (half an ulp is 2^-9 relative)
    err = np.abs(c_gpu.astype(np.float64) - c_ref)
    if not np.all(err <= tol):
        i = np.argmax(err / tol)
        raise AssertionError(f"{what}: worst error/tolerance {np.max(err / tol):.3g} "
                             f"(gpu {c_gpu.reshape(-1)[i]!r} oracle {c_ref.reshape(-1)[i]!r} S {s_ref.reshape(-1)[i]!r})")
    return float(np.max(err / tol))
