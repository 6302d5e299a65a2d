"""Seeded synthetic inputs for the k-means-quantized linear layer.

This module only *prepares inputs*: it draws weights and activations, fits the
per-row codebooks and assigns every weight to its nearest centroid.  It holds
none of the arithmetic of the inference path (no bit-packing, no table-lookup
dequantisation, no matrix product), so it can feed both the CUDA library and
the CPU oracle without coupling them.

What is generated, and where each choice comes from:

* Weights ``W`` (fp32, ``[N, K]``): the trained checkpoints the paper measures
  are not available, so the layer shapes and value distributions of the
  benchmark configurations stand in for them: Normal(0, std 0.02),
  Student-t(nu=5) rescaled to std 0.02, Laplace(0, scale 0.014).
* Codebooks: the paper obtains centroids "algorithmically by 1-D k-means"
  (Section 2.1, "Rounding to nearest centroids"; Section 2.2, "Nonlinear
  k-means quantization").  Here the fit is per output row, 2^b centroids,
  Lloyd's algorithm started at the row quantiles (i + 0.5) / 2^b and run for
  exactly 20 iterations in float64.  A weight that sits exactly on a boundary
  goes to the lower cluster, an empty cluster keeps its centroid.
* Indices: the nearest-centroid quantiser f_c(x) = argmin_i |x - c_i|
  (Eq. "centroid quantizer", Section 2.1), evaluated against the *stored*
  bf16 centroids, ties and duplicates resolved to the lowest index.
* Activations ``x`` (bf16 bit patterns, ``[M, K]``): Normal(0, 1) rounded to
  bf16 with round-to-nearest-even.

All tensors leave this module as NumPy arrays; bf16 values are carried as
``uint16`` bit patterns.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "f32_to_bf16_bits", "bf16_bits_to_f32", "rng_for", "draw_weights",
    "draw_activations", "lloyd_rows", "assign_rows", "make_layer",
    "CONFIG_LAYERS",
]

TENSOR_W = 0
TENSOR_X = 1


# --------------------------------------------------------------------------
# bf16 <-> fp32 on bit patterns
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round finite fp32 values to bf16 (round-to-nearest-even), as uint16."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 exactly."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


# --------------------------------------------------------------------------
# random draws
# --------------------------------------------------------------------------
def rng_for(config_id: int, tensor_id: int, seed: int = 0) -> np.random.Generator:
    """One independent PCG64 stream per (seed, configuration, tensor)."""
    ss = np.random.SeedSequence([int(seed), int(config_id), int(tensor_id)])
    return np.random.Generator(np.random.PCG64(ss))


def draw_weights(dist: str, N: int, K: int, rng: np.random.Generator) -> np.ndarray:
    """fp32 ``[N, K]`` weights with standard deviation close to 0.02.

    ``normal``   : N(0, 0.02^2)
    ``student_t``: t(nu=5) * 0.02 / sqrt(5/3)   (variance of t_nu is nu/(nu-2))
    ``laplace``  : Laplace(0, scale=0.014)      (std = 0.014*sqrt(2) ~ 0.0198)
    """
    if dist == "normal":
        w = rng.standard_normal((N, K)) * 0.02
    elif dist == "student_t":
        w = rng.standard_t(5.0, size=(N, K)) * (0.02 / np.sqrt(5.0 / 3.0))
    elif dist == "laplace":
        w = rng.laplace(0.0, 0.014, size=(N, K))
    else:
        raise ValueError(f"unknown weight distribution {dist!r}")
    return w.astype(np.float32)


def draw_activations(M: int, K: int, rng: np.random.Generator) -> np.ndarray:
    """bf16 bit patterns ``[M, K]`` of N(0, 1) draws."""
    return f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))


# --------------------------------------------------------------------------
# per-row 1-D k-means (Lloyd) and nearest-centroid assignment
# --------------------------------------------------------------------------
def lloyd_rows(W: np.ndarray, bits: int, iters: int = 20) -> np.ndarray:
    """Per-row 1-D Lloyd k-means with 2^bits centroids; float64 ``[N, 2^bits]``.

    Each row is sorted once; one iteration then needs only the positions of
    the 2^bits - 1 cluster boundaries in the sorted row (binary search) and
    differences of the row's prefix sums.  The centroids stay sorted.
    """
    W = np.asarray(W)
    N, K = W.shape
    Q = 1 << bits
    Ws = np.sort(W.astype(np.float64), axis=1)
    csum = np.zeros((N, K + 1), dtype=np.float64)
    np.cumsum(Ws, axis=1, out=csum[:, 1:])

    # start: linear-interpolated row quantiles at (i + 0.5) / Q
    pos = (np.arange(Q, dtype=np.float64) + 0.5) / Q * (K - 1)
    lo = np.floor(pos).astype(np.int64)
    hi = np.minimum(lo + 1, K - 1)
    frac = pos - lo
    c = Ws[:, lo] * (1.0 - frac) + Ws[:, hi] * frac

    rows = np.arange(N)[:, None]
    edges = np.empty((N, Q + 1), dtype=np.int64)
    edges[:, 0] = 0
    edges[:, Q] = K
    for _ in range(iters):
        mids = 0.5 * (c[:, :-1] + c[:, 1:])
        for n in range(N):
            # members of cluster i are the sorted positions [edges[i], edges[i+1]):
            # a weight equal to a midpoint stays in the lower cluster.
            edges[n, 1:Q] = np.searchsorted(Ws[n], mids[n], side="right")
        cnt = edges[:, 1:] - edges[:, :-1]
        tot = csum[rows, edges[:, 1:]] - csum[rows, edges[:, :-1]]
        mean = tot / np.maximum(cnt, 1)
        c = np.where(cnt > 0, mean, c)
    return c


def assign_rows(W: np.ndarray, codebooks_bf16: np.ndarray, chunk_rows: int = 512) -> np.ndarray:
    """uint8 ``[N, K]``: index of the stored centroid nearest to each weight.

    ``codebooks_bf16`` is ``[N, Q]`` uint16 (bf16 bits), non-decreasing along
    each row.  Distances are compared in float64 (sums of two bf16 values are
    exact there).  Ties and duplicated centroids resolve to the lowest index.
    """
    W = np.asarray(W)
    N, K = W.shape
    cb = bf16_bits_to_f32(codebooks_bf16).astype(np.float64)
    Q = cb.shape[1]
    if np.any(cb[:, 1:] < cb[:, :-1]):
        raise ValueError("codebook rows must be sorted ascending")
    mids = 0.5 * (cb[:, :-1] + cb[:, 1:])
    # lowest index holding the same centroid value
    first = np.zeros((N, Q), dtype=np.uint8)
    for i in range(1, Q):
        same = cb[:, i] == cb[:, i - 1]
        first[:, i] = np.where(same, first[:, i - 1], i)
    idx = np.empty((N, K), dtype=np.uint8)
    for r0 in range(0, N, chunk_rows):
        r1 = min(N, r0 + chunk_rows)
        w = W[r0:r1].astype(np.float64)
        acc = np.zeros((r1 - r0, K), dtype=np.uint8)
        for j in range(Q - 1):
            acc += w > mids[r0:r1, j:j + 1]
        idx[r0:r1] = np.take_along_axis(first[r0:r1], acc.astype(np.int64), axis=1)
    return idx


# --------------------------------------------------------------------------
# whole layers
# --------------------------------------------------------------------------
def make_layer(N: int, K: int, bits: int, M: int, dist: str = "normal",
               config_id: int = 1, seed: int = 0, keep_weights: bool = False) -> dict:
    """One synthetic layer: ``idx`` uint8 [N,K], ``codebooks`` bf16 bits
    [N, 2^bits], ``x`` bf16 bits [M,K] (and ``W`` fp32 when asked for)."""
    W = draw_weights(dist, N, K, rng_for(config_id, TENSOR_W, seed))
    cb = f32_to_bf16_bits(lloyd_rows(W, bits).astype(np.float32))
    idx = assign_rows(W, cb)
    x = draw_activations(M, K, rng_for(config_id, TENSOR_X, seed))
    out = {"N": N, "K": K, "bits": bits, "M": M, "idx": idx, "codebooks": cb, "x": x}
    if keep_weights:
        out["W"] = W
    return out


# (name, N, K, distribution) for the benchmark configurations; bits and batch
# sizes are chosen by the caller.
def make_block_layer(N: int, K: int, bits: int, M: int, dist: str = "normal", config_id: int = 0,
                     fit_samples: int = 1 << 20) -> dict:
    """Synthetic layer in the paper's k-means block format (Section 2.2): one bf16 scale per block of 64 inputs of a
    row (absmax of the block; a block of zeros gets scale 1), the weights divided by their stored scale lie in
    [-1, 1], one codebook of 2^bits centroids per tensor from 1-D Lloyd (same rules as lloyd_rows: quantile start,
    20 iterations) on an evenly strided sample of at most `fit_samples` normalised weights, indices = nearest stored
    centroid (ties and duplicates to the lowest index).  Input generation only: nothing here is on the timed path.
    Returns idx uint8 [N, K], scales bf16 bits [N, K/64], codebook bf16 bits [2^bits], x bf16 bits [M, K], W fp32."""
    if K % 64:
        raise ValueError("K must be a multiple of 64")
    W = draw_weights(dist, N, K, rng_for(config_id, TENSOR_W))
    blocks = W.reshape(N, K // 64, 64).astype(np.float64)
    absmax = np.abs(blocks).max(axis=2)
    scales = f32_to_bf16_bits(np.where(absmax > 0, absmax, 1.0).astype(np.float32))
    s64 = bf16_bits_to_f32(scales).astype(np.float64)
    # bf16 rounding may bring the stored scale just below the block's absmax: clip the ratio into [-1, 1]
    norm = np.clip(blocks / s64[:, :, None], -1.0, 1.0).reshape(N, K)
    flat = norm.reshape(1, -1)
    stride = max(1, flat.shape[1] // fit_samples)
    cent = lloyd_rows(flat[:, ::stride], bits)                     # [1, 2^bits], sorted
    codebook = f32_to_bf16_bits(cent.astype(np.float32))[0]
    cb = bf16_bits_to_f32(codebook).astype(np.float64)
    mids = 0.5 * (cb[:-1] + cb[1:])
    first = np.arange(cb.size)
    for i in range(1, cb.size):
        if cb[i] == cb[i - 1]:
            first[i] = first[i - 1]
    idx = first[np.searchsorted(mids, norm, side="left")].astype(np.uint8)   # a weight on a midpoint stays below
    x = draw_activations(M, K, rng_for(config_id, TENSOR_X))
    return {"idx": idx, "scales": scales, "codebook": codebook, "x": x, "W": W}


CONFIG_LAYERS = {
    1: [("tiny", 256, 256, "normal")],
    2: [("square4096", 4096, 4096, "normal")],
    3: [("qkv", 9216, 3072, "student_t"), ("o", 3072, 3072, "student_t"),
        ("gate_up", 16384, 3072, "student_t"), ("down", 3072, 8192, "student_t")],
    4: [("square8192", 8192, 8192, "normal")],
    5: [("down_large", 8192, 28672, "laplace")],
}
