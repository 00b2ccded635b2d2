"""Bytes a linear layer keeps for its backward pass, with and without VeLoRA.

The paper's accounting (Appendix, memory estimates; Table 5(b)) counts the saved
input of each layer: N*D elements without compression, N*M scalars with it,
M = ceil(D / Dsub) sub-tokens per token, plus the Dsub-long vector v.
"""
from __future__ import annotations

from typing import Optional


def saved_activation_bytes(N: int, D: int, Dsub: Optional[int], x_bytes: int = 2, z_bytes: int = 4) -> int:
    """Bytes saved for backward: ``Dsub=None`` means the uncompressed input."""
    if Dsub is None:
        return N * D * x_bytes
    M = -(-D // Dsub)
    return N * M * z_bytes + Dsub * 4
