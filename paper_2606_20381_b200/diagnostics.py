"""Measurement helpers around ufp4_diagnose (not part of the hot path): the Shrinkage-Bias diagnostic of Sec. 3.1,
b_G = E[rho_G(t) - t] restricted to the bin of each level, the operand projection alpha of Eq. 3, the NMSE behind
Eq. 7 and the effective bucket ratio of Eq. 6, for a tensor quantized by libufp4.  The sums come from the library's
kernel; this module only turns them into ratios."""
from __future__ import annotations

import math

import torch

from . import binding as ufp4


def tensor_diagnostics(x: torch.Tensor, q_row: ufp4.QTensor, rht_block: int, seed_rht: int) -> dict:
    """alpha (Eq. 3), nmse (Sec. 3.3), b_eff (Eq. 6: natural log, eps = 1e-12, K = 8 magnitude buckets incl. zero),
    count[8] and bias[8] (mean of level - t per magnitude level, NaN where a level is unused) of the row variant."""
    sums = ufp4.diagnose(x, q_row, rht_block, seed_rht).cpu()
    count, bias_sum = sums[3:11], sums[11:19]
    n = float(count.sum())
    ent = -sum((float(c) / n) * math.log(float(c) / n + 1e-12) for c in count) if n > 0 else 0.0
    sxx = float(sums[0])
    return {"alpha": float(sums[2]) / sxx if sxx > 0 else float("nan"),
            "nmse": float(sums[1]) / sxx if sxx > 0 else float("nan"),
            "b_eff": math.exp(ent) / 8.0,
            "count": count.to(torch.int64),
            "bias": torch.where(count > 0, bias_sum / count.clamp_min(1), torch.full_like(bias_sum, float("nan"))),
            "sums": sums}


def per_bin_bias(x: torch.Tensor, q_row: ufp4.QTensor, rht_block: int, seed_rht: int):
    """(count[8], mean of level - t per level) for the row variant q_row of the BF16 matrix x, t = |x'| / s in grid
    units, x' the rotated input."""
    d = tensor_diagnostics(x, q_row, rht_block, seed_rht)
    return d["count"], d["bias"]
