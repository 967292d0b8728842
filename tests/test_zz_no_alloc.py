"""ufp4_gemm_noalloc: the GEMM for callers that cannot allocate device memory (everything already belongs to a pool,
or a cudaMalloc at that point would stall the device).  Its scratch is a fixed array inside the library, so the test
checks, through the C ABI, that it gives what ufp4_gemm's tensor-core path gives and what the CPU oracle computes - on
two calls in a row, the second with smaller operands so that stale scratch contents from the first call would show -
and that shapes beyond the array's size are refused with a clear error.  Collected last on purpose (file name), and it
must pass on its own too.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs

pytestmark = pytest.mark.gpu


def _operands(M, N, K, seed):
    X = inputs.heavy_tailed_activations(M, K, seed=seed)
    W = inputs.normal_bf16(N, K, 0.02, seed=seed + 1)
    kw = dict(rht_block=16, scale_fmt=oracle.SCALE_POW2, seed_rht=1)
    return oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)


def test_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    assert ufp4.gemm_noalloc_max_scratch_bytes() == 16 << 20
    for (M, N, K, seed) in ((640, 520, 1024, 41), (200, 136, 272, 43)):
        A, B = _operands(M, N, K, seed)
        C_ref, S = oracle.gemm(A, B)
        dA, dB = to_device(A), to_device(B)
        assert ufp4.gemm_workspace_bytes(dA, dB, ufp4.PATH_TENSOR) <= ufp4.gemm_noalloc_max_scratch_bytes()
        want = ufp4.gemm(dA, dB, path=ufp4.PATH_TENSOR)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        got = torch.full_like(want, float("nan"))
        ufp4.gemm_noalloc(dA, dB, got, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # against the oracle's product (the parity bar), and against the entry point that takes a caller's workspace
        assert_gemm_close(got.cpu().numpy(), C_ref, S, f"noalloc vs oracle {M}x{N}x{K}")
        assert_gemm_close(want.cpu().numpy(), C_ref, S, f"workspace entry point vs oracle {M}x{N}x{K}")
        assert_gemm_close(got.cpu().numpy(), want.double().cpu().numpy(), S, f"noalloc vs workspace entry point {M}x{N}x{K}")
        # BF16 output through the same entry point
        got16 = torch.empty(M, (N + 7) // 8 * 8, dtype=torch.bfloat16, device="cuda")[:, :N]
        ufp4.gemm_noalloc(dA, dB, got16)
        assert_gemm_close(got16.float().cpu().numpy(), C_ref, S, "noalloc bf16 vs oracle", bf16_out=True)


def test_refuses_shapes_beyond_its_scratch_and_unsupported_scales():
    # 4096 + 4096 rows at K = 4096 need 32 MiB of decoded operands: more than the fixed array holds
    rows, K = 4096, 4096
    codes = torch.zeros(rows, K // 2, dtype=torch.uint8, device="cuda")
    scales = torch.ones(rows, K // 16, dtype=torch.float32, device="cuda")
    big = ufp4.QTensor(codes, scales, ufp4.GRID_INT4, ufp4.SCALE_POW2, K)
    out = torch.empty(rows, rows, dtype=torch.float32, device="cuda")
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_noalloc(big, big, out)
    assert e.value.status == -7 and "workspace" in str(e.value)
    small = ufp4.QTensor(codes[:128, :64], scales[:128, :8], ufp4.GRID_INT4, ufp4.SCALE_FP32, 128)
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_noalloc(small, small, out[:128, :128])
    assert e.value.status == -5


def test_the_limit_is_where_the_header_says():
    """The largest shape the fixed array still holds is accepted (and computes: all-zero codes give an all-zero C), the
    next one up is refused on the host without a launch."""
    K = 4096
    limit = ufp4.gemm_noalloc_max_scratch_bytes()

    def operand(rows):
        return ufp4.QTensor(torch.zeros(rows, K // 2, dtype=torch.uint8, device="cuda"),
                            torch.ones(rows, K // 16, dtype=torch.float32, device="cuda"), ufp4.GRID_INT4, ufp4.SCALE_POW2, K)
    a, fits, too_big = operand(2048), operand(2040), operand(2048)
    assert ufp4.gemm_workspace_bytes(a, fits, ufp4.PATH_TENSOR) <= limit < ufp4.gemm_workspace_bytes(a, too_big, ufp4.PATH_TENSOR)
    out = torch.full((2048, 2040), float("nan"), dtype=torch.float32, device="cuda")
    ufp4.gemm_noalloc(a, fits, out)
    torch.cuda.synchronize()
    assert torch.count_nonzero(out).item() == 0
    with pytest.raises(ufp4.Ufp4Error) as e:
        ufp4.gemm_noalloc(a, too_big, torch.empty(2048, 2048, dtype=torch.float32, device="cuda"))
    assert e.value.status == -7
