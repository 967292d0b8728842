"""The give-up path of the tensor-core kernels' bounded waits, exercised without faulting or hanging anything: with the
test hook ufp4_debug_wait_injection the producer issues no loads, so the first wait of the MMA-issuing thread runs out
after a short poll limit with no copy and no MMA in flight.  The kernel must return by itself, report
UFP4_DEV_WAIT_TIMEOUT, release tensor memory, and leave the stream usable: the very next normal call is bit-correct."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_gemm_close, oracle_quantize, to_device
from paper_2606_20381_b200 import binding as ufp4
from paper_2606_20381_b200 import inputs

pytestmark = pytest.mark.gpu


def _operands(M, N, K, scale_fmt):
    X = inputs.heavy_tailed_activations(M, K, seed=5)
    W = inputs.normal_bf16(N, K, 0.02, seed=6)
    kw = dict(rht_block=16, scale_fmt=scale_fmt, seed_rht=1)
    if scale_fmt == oracle.SCALE_E4M3_TENSOR:
        return (oracle_quantize(X, oracle.AXIS_ROW, tensor_scale=float(np.float32(4 * X.float().abs().max() / (7 * 448))), **kw),
                oracle_quantize(W, oracle.AXIS_ROW, tensor_scale=float(np.float32(4 * W.float().abs().max() / (7 * 448))), **kw))
    return oracle_quantize(X, oracle.AXIS_ROW, **kw), oracle_quantize(W, oracle.AXIS_ROW, **kw)


@pytest.mark.parametrize("path,scale_fmt", [(ufp4.PATH_TENSOR, oracle.SCALE_POW2), (ufp4.PATH_SPLIT, oracle.SCALE_FP32),
                                            (ufp4.PATH_PROMOTE, oracle.SCALE_FP32),
                                            (ufp4.PATH_FP16, oracle.SCALE_E4M3_TENSOR), (ufp4.PATH_MX, oracle.SCALE_E8M0_B32),
                                            (ufp4.PATH_NVF4, oracle.SCALE_E4M3_TENSOR)])
@pytest.mark.parametrize("shape", [(384, 512, 256), (4096, 4096, 256)])     # a few tiles; more tiles than CTA pairs
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(path, scale_fmt, shape):
    M, N, K = shape
    A, B = _operands(M, N, K, scale_fmt)
    dA, dB = to_device(A), to_device(B)
    ws = torch.empty(ufp4.gemm_workspace_bytes(dA, dB, path), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    good = ufp4.gemm(dA, dB, path=path, workspace=ws, dev_status=status).clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    try:
        ufp4.debug_wait_injection(poll_limit=1 << 12, skip_loads=True)
        out = torch.zeros_like(good)
        ufp4.gemm(dA, dB, out=out, path=path, workspace=ws, dev_status=status)
        torch.cuda.synchronize()                      # the kernel came back by itself
    finally:
        ufp4.debug_wait_injection()
    assert int(status.item()) & ufp4.DEV_WAIT_TIMEOUT
    # the same stream, the same workspace, straight afterwards: a normal call, bit-identical to the first
    status.zero_()
    again = ufp4.gemm(dA, dB, path=path, workspace=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(again, good)
    if M <= 512:
        ref, S = oracle.gemm(A, B)
        assert_gemm_close(again.cpu().numpy(), ref, S, "the call after the timed-out one")


def test_the_hook_rejects_bad_arguments():
    assert ufp4.lib().ufp4_debug_wait_injection(0, 2) == -4
    ufp4.debug_wait_injection()
