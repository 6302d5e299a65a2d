"""Roofline speed-up model for software-decoded weight formats.  TEST
INFRASTRUCTURE / REPORTING ONLY (never imported by the library).

Plain restatement of the paper's Appendix "Theoretical model of
software-decoded formats" and of Eq. "theoretical speedup" (Section 3.3):
a kernel computing ``Y^T = W X^T`` with ``X, Y`` of shape ``m x h`` and ``W`` of
``h x h`` at ``P_w`` bits per parameter takes

    t_compute  = 2 m h^2 / R_compute
    t_transfer = P_w h^2 / (8 R_transfer)
    t          = max(t_compute, t_transfer)

and switching from ``P_w1`` to ``P_w2`` at the same compute rate gives

    speedup = max(1, P_w1 nu / (16 m)) / max(1, P_w2 nu / (16 m)),  nu = R_compute / R_transfer.

Also the average bit-width of a block format, ``P_w = n + m_scale / B``
(Eq. "fractional bit width", Section 2.1) and of the n-bit integer format,
``log2(2^n - 1) + 16/64`` (Section 2.2).

Pinned by the numbers the paper prints for the L40S (362 TFLOP/s, 864 GB/s):
peak speed-ups 3.8x / 12.8x, memory-bound up to m = 111 (4.25 bit) and m = 32
(1.25 bit), no speed-up beyond m = 418; and by the printed P_w table.
"""
from __future__ import annotations

import math


def block_bit_width(n_bits: float, scale_bits: float = 16.0, block: int = 64) -> float:
    return n_bits + scale_bits / block


def integer_format_bit_width(n: int, scale_bits: float = 16.0, block: int = 64) -> float:
    levels = 2 if n == 1 else (1 << n) - 1
    return math.log2(levels) + scale_bits / block


def per_row_codebook_bit_width(bits: int, K: int) -> float:
    """Format built here: b index bits + one 2^b-entry bf16 codebook per row of K weights."""
    return bits + 16.0 * (1 << bits) / K


def kernel_time(m: int, h: int, p_w: float, r_compute: float, r_transfer: float) -> float:
    t_compute = 2.0 * m * h * h / r_compute
    t_transfer = p_w * h * h / (8.0 * r_transfer)
    return max(t_compute, t_transfer)


def speedup(p_w1: float, p_w2: float, m: float, nu: float) -> float:
    return max(1.0, p_w1 * nu / (16.0 * m)) / max(1.0, p_w2 * nu / (16.0 * m))


def memory_bound_batch_limit(p_w: float, nu: float) -> float:
    """Largest m for which a P_w-bit kernel is still transfer-bound: P_w nu / 16."""
    return p_w * nu / 16.0
