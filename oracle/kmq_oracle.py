"""CPU oracle for the k-means-quantised linear layer.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA library is checked
against.  It shares no code with the CUDA path and must never be imported by
the library or its Python binding: only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

What it defines (NumPy, float64 arithmetic):

* ``pack_canonical`` / ``unpack_canonical`` -- the interchange bit layout.
  The paper packs quantised elements along the input dimension (Appendix
  "Benchmarking", "Kernel implementations": ``Wq`` is ``output_size x
  (input_size // elements_per_byte)``) and leaves the order inside a storage
  unit open.  Reading used here: 32-bit words, fields LSB first, i.e. bits
  ``[i*b, (i+1)*b)`` of word ``j`` of row ``n`` hold ``idx[n, j*(32/b) + i]``.
* ``dequant_bits`` -- the lookup ``W^[n, k] = C_n[idx[n, k]]`` (the listing's
  table gather ``lut[Wq]`` with the table indexed per output row and no block
  scale).  A stored centroid is copied, never rounded, so the result is a
  bf16 bit pattern and comparisons are exact.
* ``linear_f64`` -- ``y[m, n] = sum_k x[m, k] * W^[n, k]`` (the listing's
  ``x @ W.T``; Appendix "Theoretical model": ``Y^T = W X^T``), every bf16
  operand widened exactly to float64 and the sum taken in float64 by
  ``numpy.matmul``.  It also returns ``sum_k |x[m, k] * W^[n, k]|``, the
  quantity the acceptance bound is relative to.
* ``tolerance`` / ``check_linear`` -- the acceptance rule
  ``|y - y_ref| <= 2^-7 * sum_k |x_k * w_k| + 1e-6``.

Pins (see the CPU tests): brute force in pure Python on tiny shapes; a 1-bit
codebook {-a, +a} reduces to a * sign-matmul; a uniform-grid codebook
reduces to integer quantisation; pack/unpack round trip on random and
adversarial patterns; the shared-codebook special case equals a byte-table
restatement of the paper's listing; exactly-summed (``math.fsum``) dot
products.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "bf16_bits_to_f64", "pack_canonical", "unpack_canonical", "dequant_bits",
    "linear_f64", "tolerance", "check_linear", "words_per_row",
]

REL_TOL = 2.0 ** -7
ABS_TOL = 1e-6


def _check_bits(bits: int) -> int:
    if bits not in (1, 2, 4):
        raise ValueError("bits must be 1, 2 or 4")
    return 32 // bits


def words_per_row(K: int, bits: int) -> int:
    per = _check_bits(bits)
    if K <= 0 or K % per:
        raise ValueError("K must be a positive multiple of 32/bits")
    return K // per


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    u = np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def pack_canonical(idx: np.ndarray, bits: int) -> np.ndarray:
    """``idx`` uint8 ``[N, K]`` -> uint32 ``[N, K*bits/32]``, fields LSB first.

    Only the low ``bits`` bits of each index are stored.
    """
    per = _check_bits(bits)
    idx = np.asarray(idx, dtype=np.uint8)
    N, K = idx.shape
    wpr = words_per_row(K, bits)
    fields = (idx.reshape(N, wpr, per).astype(np.uint32)) & np.uint32((1 << bits) - 1)
    words = np.zeros((N, wpr), dtype=np.uint32)
    for i in range(per):
        words |= fields[:, :, i] << np.uint32(i * bits)
    return words


def unpack_canonical(packed: np.ndarray, K: int, bits: int) -> np.ndarray:
    """uint32 ``[N, K*bits/32]`` -> uint8 ``[N, K]``."""
    per = _check_bits(bits)
    packed = np.asarray(packed, dtype=np.uint32)
    N, wpr = packed.shape
    if wpr != words_per_row(K, bits):
        raise ValueError("packed width does not match K and bits")
    mask = np.uint32((1 << bits) - 1)
    out = np.empty((N, wpr, per), dtype=np.uint8)
    for i in range(per):
        out[:, :, i] = ((packed >> np.uint32(i * bits)) & mask).astype(np.uint8)
    return out.reshape(N, K)


def dequant_bits(packed: np.ndarray, codebooks: np.ndarray, K: int, bits: int) -> np.ndarray:
    """bf16 bit patterns ``[N, K]`` of ``W^[n, k] = C[n, idx[n, k]]``."""
    idx = unpack_canonical(packed, K, bits)
    codebooks = np.asarray(codebooks, dtype=np.uint16)
    if codebooks.shape != (idx.shape[0], 1 << bits):
        raise ValueError("codebooks must be [N, 2^bits]")
    return np.take_along_axis(codebooks, idx.astype(np.int64), axis=1)


def linear_f64(packed: np.ndarray, codebooks: np.ndarray, x: np.ndarray, K: int,
               bits: int, chunk_rows: int = 1024):
    """Reference output and bound base, both float64 ``[M, N]``.

    ``y_ref[m, n] = sum_k x[m, k] * W^[n, k]`` and
    ``abs_sum[m, n] = sum_k |x[m, k] * W^[n, k]|``.  Rows are processed in
    chunks only to bound the size of the float64 copy of ``W^``.
    """
    packed = np.asarray(packed, dtype=np.uint32)
    N = packed.shape[0]
    xf = bf16_bits_to_f64(x)
    if xf.ndim != 2 or xf.shape[1] != K:
        raise ValueError("x must be [M, K]")
    M = xf.shape[0]
    xa = np.abs(xf)
    y = np.empty((M, N), dtype=np.float64)
    s = np.empty((M, N), dtype=np.float64)
    for r0 in range(0, N, chunk_rows):
        r1 = min(N, r0 + chunk_rows)
        w = bf16_bits_to_f64(dequant_bits(packed[r0:r1], codebooks[r0:r1], K, bits))
        y[:, r0:r1] = xf @ w.T
        s[:, r0:r1] = xa @ np.abs(w).T
    return y, s


def tolerance(abs_sum: np.ndarray) -> np.ndarray:
    """Elementwise acceptance bound ``2^-7 * abs_sum + 1e-6``."""
    return REL_TOL * np.asarray(abs_sum, dtype=np.float64) + ABS_TOL


def check_linear(y_bits: np.ndarray, y_ref: np.ndarray, abs_sum: np.ndarray) -> float:
    """Largest ``|y - y_ref| / tolerance`` over all outputs (pass iff <= 1).

    ``y_bits`` are the bf16 bit patterns produced by the implementation under
    test; they are widened exactly before the comparison.
    """
    y = bf16_bits_to_f64(y_bits)
    if y.shape != y_ref.shape:
        raise ValueError("shape mismatch")
    if not np.all(np.isfinite(y)):
        return float("inf")
    return float(np.max(np.abs(y - y_ref) / tolerance(abs_sum))) if y.size else 0.0
