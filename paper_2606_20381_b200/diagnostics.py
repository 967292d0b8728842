"""Measurement helpers around ufp4_diagnose (not part of the hot path): the Shrinkage-Bias diagnostic of Sec. 3.1, the
operand projection alpha of Eq. 3, the NMSE behind Eq. 7 and the effective bucket ratio of Eq. 6, for a tensor
quantized by libufp4.  Both the sums (a kernel) and the ratios (ufp4_diagnose_ratios) come from the library; this
module only names the entries of what it returns."""
from __future__ import annotations

import torch

from . import binding as ufp4


def tensor_diagnostics(x: torch.Tensor, q_row: ufp4.QTensor, rht_block: int, seed_rht: int) -> dict:
    """alpha, nmse, b_eff, count[8] and bias[8] (NaN where a level is unused) of the row variant q_row of x."""
    sums = ufp4.diagnose(x, q_row, rht_block, seed_rht).cpu()
    r = ufp4.diagnose_ratios(sums.tolist())
    return {"alpha": r[0], "nmse": r[1], "b_eff": r[2], "count": sums[3:11].to(torch.int64),
            "bias": torch.tensor(r[3:11], dtype=torch.float64), "sums": sums}


def per_bin_bias(x: torch.Tensor, q_row: ufp4.QTensor, rht_block: int, seed_rht: int):
    """(count[8], mean of level - t per level) for the row variant q_row of the BF16 matrix x."""
    d = tensor_diagnostics(x, q_row, rht_block, seed_rht)
    return d["count"], d["bias"]
