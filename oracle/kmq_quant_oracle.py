"""CPU oracle for the quantiser side: centroid fit, nearest-centroid assignment, block scales.
TEST INFRASTRUCTURE ONLY.

The slow, plain definition that the CUDA entry points ``kmq_kmeans_rows``, ``kmq_assign_pack``, ``kmq_block_scales``,
``kmq_block_sample`` and ``kmq_block_assign`` are checked against.  It shares no code with the CUDA path (nor with the
seeded input generators) and must never be imported by the library or its binding.

What the paper fixes (Section 2.1, "Rounding to nearest centroids", Eq. "centroid quantizer"; "Block formats";
Section 2.2, "Uniform integer quantization" for the two scale functions, "Nonlinear k-means quantization"):

* the quantiser is ``f_c(x) = argmin_{c_i} |x - c_i|``;
* the centroids come from 1-D k-means clustering (Lloyd) of the (normalised) weights;
* a block format stores one scale ``lambda(w_J)`` per block of ``B = 64`` weights in 16 bits, ``lambda`` being the
  block's absmax or absmean, and the k-means centroids of the normalised weights lie in [-1, 1].

What it leaves open, and the reading taken here (the same on both sides of every parity test):

* start of the iteration: the ``2^b`` linearly interpolated quantiles of the values at ``(i + 1/2) / 2^b``; a fixed
  number of iterations (20 unless told otherwise); an empty cluster keeps its centroid;
* a value exactly half-way between two centroids goes to the lower one, and equal centroids are represented by the
  lowest index among them.  In one dimension with sorted centroids the argmin is then the number of midpoints
  ``(c_i + c_{i+1}) / 2`` strictly below the value.  Inside the iteration the midpoint is the float64 value of that
  expression.  For stored (bf16) centroids the comparison is exact whatever their magnitudes: with ``s + e = c_i +
  c_{i+1}`` exactly (``s`` the float64 sum, ``e`` its rounding error), ``x`` lies above the midpoint iff ``2x > s``, or
  ``2x = s`` and ``e < 0`` (if ``2x`` differs from ``s`` it differs by more than ``|e|``, both being multiples of the
  last place of ``s`` or far apart);
* arithmetic: float64 sums and means; the stored centroid is the float64 mean rounded to float32 and then to bf16,
  both to nearest even; a centroid that is zero is stored as +0 (the sign of a zero mean depends on the order of
  the additions and carries no information);
* absmean sums the 64 magnitudes in float64 in index order (the order is part of the reading so that the stored bf16
  scale is reproducible bit for bit); a block of zeros gets scale 1; normalised weight = ``w / scale``, the
  float64 quotient with the stored scale, not clipped: with absmax it lies in [-1, 1] up to the bf16 rounding of the
  scale (at most 1 + 2^-8 in magnitude), with absmean it does not, and the paper fits k-means under both;
* the per-tensor fit of the block format runs on an evenly strided sample of the normalised weights, rounded to
  float32: flat indices ``0, s, 2s, ...`` with ``s = max(1, N*K // samples)``, the first ``samples`` of them.

Functions: ``quantile_start``, ``lloyd_1d``, ``lloyd_rows``, ``centroids_to_bf16``, ``nearest_centroid``,
``block_scales``, ``normalise``, ``strided_sample``, ``block_assign``.

Pins (tests/test_quant_oracle_pins.py): exact rational brute force of the argmin on tiny and on badly scaled inputs;
scikit-learn's Lloyd iteration from the same start; NumPy's quantile routine; the fixed-point and monotone-error
properties of Lloyd's method; closed forms (two separated clusters, a uniform grid, the 1-bit optimum of a Gaussian);
planted mistakes.
"""
from __future__ import annotations

import numpy as np

__all__ = ["BLOCK", "ABSMAX", "ABSMEAN", "quantile_start", "lloyd_1d", "lloyd_rows", "centroids_to_bf16",
           "nearest_centroid", "block_scales", "normalise", "strided_sample", "block_assign", "f32_to_bf16_rne"]

BLOCK = 64
ABSMAX, ABSMEAN = 0, 1


def _bf16_to_f64(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f32_to_bf16_rne(f: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern, round to nearest, ties to even (finite inputs)."""
    u = np.ascontiguousarray(f, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)).astype(np.uint16)


def quantile_start(values: np.ndarray, Q: int) -> np.ndarray:
    """The Q start centroids of one set of values: order statistics interpolated linearly at (i + 1/2) / Q."""
    v = np.sort(np.asarray(values, dtype=np.float64))
    K = v.size
    out = np.empty(Q, dtype=np.float64)
    for i in range(Q):
        pos = (i + 0.5) / Q * (K - 1)
        lo = int(np.floor(pos))
        hi = min(lo + 1, K - 1)
        t = pos - lo
        out[i] = v[lo] * (1.0 - t) + v[hi] * t
    return out


def _assign_sorted(values: np.ndarray, c: np.ndarray) -> np.ndarray:
    """Index of the nearest centroid, c non-decreasing: the number of midpoints strictly below the value."""
    mids = 0.5 * (c[:-1] + c[1:])
    idx = np.zeros(values.shape, dtype=np.int64)
    for m in mids:
        idx += values > m
    return idx


def _assign_exact(values: np.ndarray, cb: np.ndarray) -> np.ndarray:
    """Number of exact midpoints of neighbouring stored centroids strictly below each value (float64 inputs)."""
    idx = np.zeros(values.shape, dtype=np.int64)
    two = 2.0 * values
    for a, b in zip(cb[:-1], cb[1:]):
        s = a + b
        bb = s - a
        e = (a - (s - bb)) + (b - bb)            # s + e = a + b exactly
        idx += (two > s) | ((two == s) & (e < 0))
    return idx


def lloyd_1d(values: np.ndarray, bits: int, iters: int = 20, start: np.ndarray | None = None) -> np.ndarray:
    """Lloyd's method on one set of values: `iters` times (assign every value to its nearest centroid, move every
    centroid to the mean of its values).  float64 [2^bits], non-decreasing."""
    v = np.asarray(values, dtype=np.float64).reshape(-1)
    Q = 1 << bits
    c = quantile_start(v, Q) if start is None else np.array(start, dtype=np.float64)
    for _ in range(iters):
        idx = _assign_sorted(v, c)
        for j in range(Q):
            members = v[idx == j]
            if members.size:
                c[j] = members.sum() / members.size
    return c


def lloyd_rows(W: np.ndarray, bits: int, iters: int = 20) -> np.ndarray:
    """One fit per row of W: float64 [N, 2^bits]."""
    W = np.asarray(W)
    return np.stack([lloyd_1d(W[n], bits, iters) for n in range(W.shape[0])])


def centroids_to_bf16(c: np.ndarray) -> np.ndarray:
    """Stored form of fitted centroids: float64 -> float32 -> bf16, each step to nearest even; zero as +0."""
    bits = f32_to_bf16_rne(np.asarray(c, dtype=np.float64).astype(np.float32))
    return np.where((bits & np.uint16(0x7FFF)) == 0, np.uint16(0), bits).astype(np.uint16)


def _first_of_equal(cb: np.ndarray) -> np.ndarray:
    first = np.arange(cb.size)
    for i in range(1, cb.size):
        if cb[i] == cb[i - 1]:
            first[i] = first[i - 1]
    return first


def nearest_centroid(W: np.ndarray, codebooks_bf16: np.ndarray) -> np.ndarray:
    """Eq. "centroid quantizer" per row: uint8 [N, K], index of the stored centroid nearest to each weight.
    codebooks_bf16 uint16 [N, Q], each row non-decreasing.  The comparison with the midpoints is exact.  NaN weights
    get index 0."""
    W = np.asarray(W, dtype=np.float32)
    cb = _bf16_to_f64(codebooks_bf16)
    if np.any(cb[:, 1:] < cb[:, :-1]):
        raise ValueError("codebook rows must be non-decreasing")
    out = np.empty(W.shape, dtype=np.uint8)
    for n in range(W.shape[0]):
        idx = _assign_exact(W[n].astype(np.float64), cb[n])
        out[n] = _first_of_equal(cb[n])[idx]
    return out


def block_scales(W: np.ndarray, mode: int = ABSMAX) -> np.ndarray:
    """bf16 scale per block of 64 consecutive inputs of a row: uint16 [N, K/64]."""
    W = np.asarray(W, dtype=np.float32)
    N, K = W.shape
    if K % BLOCK:
        raise ValueError("K must be a multiple of 64")
    a = np.abs(W.astype(np.float64)).reshape(N, K // BLOCK, BLOCK)
    if mode == ABSMAX:
        lam = a.max(axis=2)
    elif mode == ABSMEAN:
        acc = np.zeros((N, K // BLOCK), dtype=np.float64)
        for j in range(BLOCK):                       # index order: part of the reading
            acc = acc + a[:, :, j]
        lam = acc / BLOCK
    else:
        raise ValueError("mode must be ABSMAX or ABSMEAN")
    bits = f32_to_bf16_rne(lam.astype(np.float32))
    # a scale that is zero (an all-zero block, or an absmean that rounds to zero) is stored as 1
    return np.where(_bf16_to_f64(bits) > 0, bits, np.uint16(0x3F80)).astype(np.uint16)


def normalise(W: np.ndarray, scales_bf16: np.ndarray) -> np.ndarray:
    """w / stored scale in float64: [N, K]."""
    W = np.asarray(W, dtype=np.float32)
    N, K = W.shape
    s = _bf16_to_f64(scales_bf16).reshape(N, K // BLOCK, 1)
    return (W.astype(np.float64).reshape(N, K // BLOCK, BLOCK) / s).reshape(N, K)


def strided_sample(W: np.ndarray, scales_bf16: np.ndarray, samples: int) -> np.ndarray:
    """float32 [min(samples, ...)]: the normalised weights at flat indices 0, s, 2s, ... with s = max(1, N*K //
    samples), the first `samples` of them, rounded to float32."""
    flat = normalise(W, scales_bf16).reshape(-1)
    s = max(1, flat.size // samples)
    return flat[::s][:samples].astype(np.float32)


def block_assign(W: np.ndarray, scales_bf16: np.ndarray, codebook_bf16: np.ndarray) -> np.ndarray:
    """uint8 [N, K]: index of the shared stored centroid nearest to the normalised weight."""
    cb = _bf16_to_f64(np.asarray(codebook_bf16, dtype=np.uint16).reshape(-1))
    if np.any(cb[1:] < cb[:-1]):
        raise ValueError("codebook must be non-decreasing")
    norm = normalise(W, scales_bf16)
    idx = _assign_exact(norm, cb)
    return _first_of_equal(cb)[idx].astype(np.uint8)
