"""Ablation only, not part of the library's path: Eq. 7 evaluated the way the paper ran it -- a numerical
framework's cumulative-sum and LogCumSumExp kernels plus elementwise kernels, every one of them a full
pass over HBM.  `bench.py --ablation unfused` times it beside the fused kernels and a GPU test checks it
against the float64 oracle, so that the comparison is between two correct evaluations."""
from __future__ import annotations

import torch

FRAMEWORK_KERNELS_PER_CALL = 5
# least traffic of the recipe in 4-byte elements: cumsum r+w, subtract r+r+w, cat r+w, LCSE r+w, slice+add r+r+w
MIN_BYTES_PER_ELEMENT = (2 + 3 + 2 + 2 + 3) * 4


def scan_log_unfused(log_a: torch.Tensor, log_b: torch.Tensor, log_x0: torch.Tensor) -> torch.Tensor:
    """log x of Eq. 7 from framework scans: a* = cumsum(log a) (Eq. 2), log x = a* + tail(LCSE(cat(log x0,
    log b - a*))) (Eq. 7-8); [rows, n] float32 tensors, log_x0 [rows].  Eq. 3 would add one exp."""
    a_star = torch.cumsum(log_a, dim=1)
    z = torch.cat([log_x0[:, None], log_b - a_star], dim=1)
    return a_star + torch.logcumsumexp(z, dim=1)[:, 1:]
