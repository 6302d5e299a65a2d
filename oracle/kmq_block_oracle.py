"""CPU oracle for the paper's own k-means block format.  TEST INFRASTRUCTURE ONLY.

The slow, plain definition that the CUDA entry points ``kmq_block_*`` are checked against.  It shares no code with
the CUDA path and must never be imported by the library or its binding: only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

The format (paper, Section 2.1 "Block formats" and Eq. "fractional bit width"; Section 2.2 "Nonlinear k-means
quantization"; Appendix "Benchmarking", "Kernel implementations"):

* one codebook of ``2^b`` centroids in ``[-1, 1]`` per weight tensor, ``b`` in {1, 2, 4, 8};
* the weights of an output row are cut into blocks of ``B = 64`` consecutive inputs, one 16-bit (bf16) scale per
  block: ``W^[n, k] = scale[n, k // B] * c[idx[n, k]]``, ``P_w = b + 16 / B = b + 0.25`` bits per weight;
* the indices are packed along the input dimension into bytes, ``8 / b`` per byte (``Wq`` is ``output_size x
  (input_size // elements_per_byte)`` bytes).  The order inside a byte is left open by the paper; the reading here is
  LSB first: bits ``[i*b, (i+1)*b)`` of byte ``j`` of row ``n`` hold ``idx[n, j*(8/b) + i]``.

Functions (NumPy, float64 arithmetic):

* ``pack_bytes`` / ``unpack_bytes`` -- that byte layout.
* ``lut8`` -- the paper's 256-entry table: byte value -> its ``8 / b`` decoded centroids.
* ``dequant_unscaled`` -- the listing's gather ``lut8[Wq]`` flattened: the centroid of every weight (bf16 bits).
* ``block_linear_f64`` -- the layer in both orders the paper gives.  ``order="direct"`` scales every weight and
  then contracts (the first listing: ``W = Wu * Wscale; x @ W.T``); ``order="deferred"`` contracts every block with
  the unscaled centroids and scales the per-block sums (the second listing: ``z = einsum(x, Wu)`` per block, ``y =
  einsum(z, Wscale)``).  Every bf16 operand is widened exactly to float64 and nothing is rounded in between, so the
  two orders agree to float64 rounding; reading taken where the listings, run in bf16 as printed, would round ``W``
  (or ``z``) to bf16: that rounding is an artefact of the compute type, not part of the format, and it stays inside
  the acceptance bound either way.  Also returns ``sum_k |x_k * W^[n, k]|``.
* ``dequant_scaled_bits`` -- ``bf16(scale * centroid)``, round to nearest even of the exact product: what a
  separate dequantise step ahead of a standard GEMM stores.
* ``block_bits_per_weight`` -- ``b + 16 / B``.

Pins (tests/test_block_oracle_pins.py): pure-Python brute force on tiny shapes; all scales 1 and the rows' shared
codebook reduce to the per-row oracle ``kmq_oracle.linear_f64``; direct and deferred agree to 1e-12 relative; a
literal restatement of the first listing with a 256-entry table; ``P_w = b + 0.25`` reproduces the bytes behind the
effective bandwidths of the paper's micro-benchmark table; planted mistakes (MSB-first bytes, scale of the wrong
block, transposed scale index) fail.
"""
from __future__ import annotations

import numpy as np

__all__ = ["BLOCK", "pack_bytes", "unpack_bytes", "lut8", "dequant_unscaled", "block_linear_f64",
           "dequant_scaled_bits", "block_bits_per_weight", "f64_to_bf16_bits"]

BLOCK = 64   # the paper's block size B


def _check(bits: int) -> int:
    if bits not in (1, 2, 4, 8):
        raise ValueError("bits must be 1, 2, 4 or 8")
    return 8 // bits


def _bf16_to_f64(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16, ties to even.  The values rounded here are products of two bf16 numbers (16
    significant bits at most), hence exact in float32; the float32 bit pattern is then rounded to its upper 16 bits
    by the integer rule (add half of the dropped range, and the kept bit's parity on a tie)."""
    f = np.asarray(v, dtype=np.float64).astype(np.float32)
    if not np.array_equal(f.astype(np.float64), np.asarray(v, dtype=np.float64)):
        raise ValueError("value not exactly representable in float32")
    u = f.view(np.uint32).astype(np.uint64)
    return ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)).astype(np.uint16)


def pack_bytes(idx: np.ndarray, bits: int) -> np.ndarray:
    """idx uint8 [N, K] -> bytes uint8 [N, K*bits/8], fields LSB first; values are reduced to their low `bits` bits."""
    per = _check(bits)
    idx = np.asarray(idx, dtype=np.uint8)
    N, K = idx.shape
    if K % per:
        raise ValueError("K must be a multiple of 8/bits")
    f = (idx.reshape(N, K // per, per).astype(np.uint16) & ((1 << bits) - 1))
    shifts = (np.arange(per) * bits).astype(np.uint16)
    return (f << shifts).sum(axis=2).astype(np.uint8)


def unpack_bytes(wq: np.ndarray, K: int, bits: int) -> np.ndarray:
    per = _check(bits)
    wq = np.asarray(wq, dtype=np.uint8)
    shifts = (np.arange(per) * bits).astype(np.uint8)
    f = (wq[:, :, None] >> shifts) & np.uint8((1 << bits) - 1)
    return f.reshape(wq.shape[0], -1)[:, :K]


def lut8(codebook: np.ndarray, bits: int) -> np.ndarray:
    """The 256-entry table of the paper's listing: byte value -> the 8/bits centroids it encodes (bf16 bits)."""
    per = _check(bits)
    cb = np.asarray(codebook, dtype=np.uint16).reshape(-1)
    if cb.size != 1 << bits:
        raise ValueError("codebook must have 2^bits entries")
    byte = np.arange(256, dtype=np.uint16)[:, None]
    return cb[(byte >> (np.arange(per, dtype=np.uint16) * bits)) & ((1 << bits) - 1)]


def dequant_unscaled(wq: np.ndarray, codebook: np.ndarray, K: int, bits: int) -> np.ndarray:
    """Centroid of every weight, bf16 bits [N, K]: the listing's ``lut8[Wq].flatten(start_dim=1)``."""
    return lut8(codebook, bits)[np.asarray(wq, dtype=np.uint8)].reshape(wq.shape[0], -1)[:, :K]


def block_linear_f64(wq, scales, codebook, x, K: int, bits: int, order: str = "direct"):
    """y[m, n] = sum_k x[m, k] * scale[n, k // 64] * c[idx[n, k]] in float64, and sum_k |x * W^|.

    wq uint8 [N, K*bits/8]; scales bf16 bits [N, K/64]; codebook bf16 bits [2^bits]; x bf16 bits [M, K]."""
    if K % BLOCK:
        raise ValueError("K must be a multiple of the block size 64")
    N = wq.shape[0]
    G = K // BLOCK
    wu = _bf16_to_f64(dequant_unscaled(wq, codebook, K, bits)).reshape(N, G, BLOCK)
    s = _bf16_to_f64(scales).reshape(N, G)
    xf = _bf16_to_f64(x).reshape(-1, G, BLOCK)
    if order == "direct":
        w = (wu * s[:, :, None]).reshape(N, K)
        y = xf.reshape(-1, K) @ w.T
    elif order == "deferred":
        z = np.einsum("mGg,hGg->mhG", xf, wu)
        y = np.einsum("mhG,hG->mh", z, s)
    else:
        raise ValueError("order must be 'direct' or 'deferred'")
    abs_sum = np.abs(xf.reshape(-1, K)) @ np.abs(wu * s[:, :, None]).reshape(N, K).T
    return y, abs_sum


def dequant_scaled_bits(wq, scales, codebook, K: int, bits: int) -> np.ndarray:
    """bf16(scale * centroid) for every weight, [N, K] bf16 bits: the exact product rounded to nearest even."""
    N = wq.shape[0]
    wu = _bf16_to_f64(dequant_unscaled(wq, codebook, K, bits)).reshape(N, K // BLOCK, BLOCK)
    w = wu * _bf16_to_f64(scales).reshape(N, K // BLOCK)[:, :, None]     # exact in float64: 8 x 8 significant bits
    return f64_to_bf16_bits(w.reshape(N, K)).reshape(N, K)


def block_bits_per_weight(bits: int, scale_bits: int = 16, block: int = BLOCK) -> float:
    """P_w = n + m / B (Eq. "fractional bit width")."""
    return bits + scale_bits / block
