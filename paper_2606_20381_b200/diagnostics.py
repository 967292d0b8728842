"""Measurement helpers (plain torch ops on the GPU, not part of the hot path): the Shrinkage-Bias diagnostic of
Sec. 3.1, b_G = E[rho_G(t) - t] restricted to the bin of each level, evaluated on a tensor quantized by libufp4."""
from __future__ import annotations

import torch

from . import binding as ufp4

_LEVELS = {ufp4.GRID_INT4: [0, 1, 2, 3, 4, 5, 6, 7], ufp4.GRID_E1M2: [0, .25, .5, .75, 1, 1.25, 1.5, 1.75],
           ufp4.GRID_E2M1: [0, .5, 1, 1.5, 2, 3, 4, 6]}


def hadamard16(device) -> torch.Tensor:
    h = torch.ones(1, 1, dtype=torch.float64, device=device)
    for _ in range(4):
        h = torch.cat([torch.cat([h, h], 1), torch.cat([h, -h], 1)], 0)
    return h / 4.0


def unpack_levels(q: ufp4.QTensor) -> torch.Tensor:
    """Magnitude level index (0..7) of every element of a quantized tensor, [rows][k]."""
    c = q.packed_codes()
    nib = torch.stack([c & 0xF, c >> 4], -1).reshape(c.shape[0], -1).to(torch.int16)
    if q.grid == ufp4.GRID_INT4:
        return torch.where(nib >= 8, 16 - nib, nib)
    return nib & 7


def per_bin_bias(x: torch.Tensor, q_row: ufp4.QTensor, rht_block: int, seed_rht: int):
    """(count[8], mean of level - t per level) for the row variant q_row of the BF16 matrix x, t = |x'| / s in grid
    units, x' the rotated input (FP64 matrix product with H'_16; a measurement, not a bit-exact replay)."""
    rows, cols = x.shape
    xb = x.double().reshape(rows, cols // 16, 16)
    if rht_block == 16:
        mask = ufp4.rht_sign_mask(seed_rht)
        eps = torch.tensor([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)], dtype=torch.float64, device=x.device)
        xb = (xb * eps) @ hadamard16(x.device)
    s = q_row.scales.double().unsqueeze(-1)
    t = torch.where(s > 0, xb.abs() / s.clamp_min(1e-300), torch.zeros_like(xb)).reshape(rows, cols)
    idx = unpack_levels(q_row).long()
    lv = torch.tensor(_LEVELS[q_row.grid], dtype=torch.float64, device=x.device)
    err = lv[idx] - t
    count = torch.bincount(idx.reshape(-1), minlength=8)
    total = torch.zeros(8, dtype=torch.float64, device=x.device).index_add_(0, idx.reshape(-1), err.reshape(-1))
    return count.cpu(), (total / count.clamp_min(1)).cpu()
