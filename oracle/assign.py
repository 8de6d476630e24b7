"""Window ownership across window-parallel ranks, written out from the definitions (test infrastructure, not
the product; the same import rule as the rest of this package applies).

Section V-A, Eq. 3: the fixed assignment pads the input field so that an m x n rank mesh holds equal numbers of
complete windows.  Section V-A, Eq. 4: the ragged assignment gives rank r the contiguous row-major window range
[floor(r M / R), floor((r + 1) M / R)).  Python integers: exact at any size.
"""
from __future__ import annotations


def fixed_assignment_padding(H: int, W: int, p: int, alpha: int, w: int, m: int = 1, n: int = 1):
    """(H_hat, W_hat) of Eq. 3."""
    uh, uw = p * alpha * w * m, p * alpha * w * n
    return -(-H // uh) * uh, -(-W // uw) * uw


def padding_overhead(H: int, W: int, H_hat: int, W_hat: int) -> float:
    """Extra grid points relative to the unpadded field (the figure Section VII-E quotes in per cent)."""
    return H_hat * W_hat / (H * W) - 1.0


def ragged_window_range(M: int, ranks: int, r: int):
    """[L_r, R_r) of Eq. 4."""
    return (r * M) // ranks, ((r + 1) * M) // ranks


def ragged_owner(M: int, ranks: int, j: int) -> int:
    """The rank that owns window j under Eq. 4, from the inequalities L_r <= j < R_r solved for r."""
    return -(-((j + 1) * ranks) // M) - 1
