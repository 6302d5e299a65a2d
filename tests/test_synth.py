"""Input generators: bf16 rounding, the per-row Lloyd fit and the assignment."""
import math

import numpy as np
import pytest
import torch

from paper_2602_15563_b200 import synth


def test_bf16_rounding_matches_torch_and_round_trips():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 0.02,
                        rng.standard_normal(5000).astype(np.float32) * 100,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -3.0e38, 1e-40],
                                 np.float32)])
    bits = synth.f32_to_bf16_bits(a)
    t = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, t)
    # ties go to even: 1 + 2^-8 -> 1.0 ; 1 + 3*2^-8 -> 1 + 2^-6
    assert bits[-5] == 0x3F80 and bits[-4] == 0x3F82
    back = synth.bf16_bits_to_f32(bits)
    assert np.array_equal(synth.f32_to_bf16_bits(back), bits)


def naive_lloyd(row, bits, iters):
    Q = 1 << bits
    row = np.asarray(row, np.float64)
    c = np.quantile(row, (np.arange(Q) + 0.5) / Q)
    sse = []
    for _ in range(iters):
        mids = 0.5 * (c[:-1] + c[1:])
        lab = np.array([sum(1 for m in mids if w > m) for w in row])
        sse.append(float(((row - c[lab]) ** 2).sum()))
        for i in range(Q):
            if np.any(lab == i):
                c[i] = row[lab == i].mean()
    return c, sse


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_lloyd_matches_naive_and_objective_never_rises(bits):
    rng = np.random.default_rng(bits)
    W = (rng.standard_normal((4, 512)) * 0.02).astype(np.float32)
    c = synth.lloyd_rows(W, bits, iters=20)
    assert c.shape == (4, 1 << bits) and np.all(np.diff(c, axis=1) > 0)
    for n in range(4):
        ref, sse = naive_lloyd(W[n], bits, 20)
        np.testing.assert_allclose(c[n], ref, rtol=1e-9, atol=1e-12)
        assert all(b <= a + 1e-15 for a, b in zip(sse, sse[1:]))


def test_one_bit_centroids_approach_mean_abs():
    W = synth.draw_weights("normal", 4, 1 << 16, synth.rng_for(99, 0))
    c = synth.lloyd_rows(W, 1)
    target = 0.02 * math.sqrt(2 / math.pi)
    np.testing.assert_allclose(c[:, 1], target, rtol=0.03)
    np.testing.assert_allclose(c[:, 0], -target, rtol=0.03)


@pytest.mark.parametrize("bits", (2, 4))
def test_kmeans_error_not_worse_than_uniform_grid(bits):
    """The premise of the format (Section 2.1, 'Rounding to nearest centroids'):
    fitted centroids give a reconstruction error no larger than a uniform grid."""
    W = synth.draw_weights("laplace", 8, 4096, synth.rng_for(98, 0))
    cb = synth.f32_to_bf16_bits(synth.lloyd_rows(W, bits).astype(np.float32))
    idx = synth.assign_rows(W, cb)
    rec = np.take_along_axis(synth.bf16_bits_to_f32(cb), idx.astype(np.int64), axis=1)
    mse_km = ((W - rec) ** 2).mean(axis=1)
    Q = 1 << bits
    amax = np.abs(W).max(axis=1, keepdims=True)
    step = 2 * amax / (Q - 1)
    uni = np.round((W + amax) / step) * step - amax
    mse_uni = ((W - uni) ** 2).mean(axis=1)
    assert np.all(mse_km < mse_uni)


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_assignment_is_first_argmin_against_stored_centroids(bits):
    rng = np.random.default_rng(5 + bits)
    N, K, Q = 6, 300, 1 << bits
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    cb = synth.f32_to_bf16_bits(synth.lloyd_rows(W, bits).astype(np.float32))
    if Q >= 4:                       # force duplicated centroids in one row
        cb[0, 1] = cb[0, 0]
        cb[1, Q - 1] = cb[1, Q - 2]
    cf = synth.bf16_bits_to_f32(cb).astype(np.float64)
    # plant exact ties: a weight on the midpoint of two neighbouring centroids
    mid = (0.5 * (cf[2, 0] + cf[2, 1]))
    if np.float32(mid) == mid:
        W[2, 0] = np.float32(mid)
    idx = synth.assign_rows(W, cb, chunk_rows=4)
    brute = np.abs(W.astype(np.float64)[:, :, None] - cf[:, None, :]).argmin(axis=2)
    assert np.array_equal(idx, brute.astype(np.uint8))


def test_distributions_and_determinism():
    for dist in ("normal", "student_t", "laplace"):
        W = synth.draw_weights(dist, 64, 4096, synth.rng_for(3, 0))
        assert W.dtype == np.float32 and abs(W.std() - 0.02) < 0.002 and abs(W.mean()) < 1e-3
    a = synth.make_layer(32, 64, 2, 3, "student_t", config_id=3)
    b = synth.make_layer(32, 64, 2, 3, "student_t", config_id=3)
    for k in ("idx", "codebooks", "x"):
        assert np.array_equal(a[k], b[k])
    assert a["idx"].max() < 4 and a["x"].shape == (3, 64) and a["codebooks"].shape == (32, 4)
    c = synth.make_layer(32, 64, 2, 3, "student_t", config_id=4)
    assert not np.array_equal(a["x"], c["x"])


@pytest.mark.parametrize("bits", (1, 2, 4, 8))
def test_block_layer_generator(bits):
    """make_block_layer: scales are the stored absmax of each block, the codebook is sorted and inside [-1, 1], and
    every index is the nearest stored centroid of the normalised weight (brute force, lowest index on ties)."""
    L = synth.make_block_layer(24, 256, bits, 1, "normal", config_id=3)
    W = L["W"].astype(np.float64).reshape(24, 4, 64)
    s = synth.bf16_bits_to_f32(L["scales"]).astype(np.float64)
    assert np.array_equal(L["scales"], synth.f32_to_bf16_bits(np.abs(L["W"]).reshape(24, 4, 64).max(axis=2)))
    cb = synth.bf16_bits_to_f32(L["codebook"]).astype(np.float64)
    assert cb.size == 1 << bits and np.all(np.diff(cb) >= 0) and cb.min() >= -1.0 and cb.max() <= 1.0
    norm = np.clip(W / s[:, :, None], -1.0, 1.0).reshape(24, 256)
    brute = np.abs(norm[:, :, None] - cb[None, None, :]).argmin(axis=2)        # argmin takes the first minimum
    assert np.array_equal(L["idx"], brute)
    assert L["idx"].max() < (1 << bits)
