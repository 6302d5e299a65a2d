"""Pins of the quantiser oracle (oracle/kmq_quant_oracle.py) against things other than itself: exact rational brute
force, scikit-learn's Lloyd iteration, NumPy's quantiles, the defining properties of Lloyd's method, closed forms, and
planted mistakes that each of them must catch."""
from fractions import Fraction
import struct

import numpy as np
import pytest

from oracle import kmq_quant_oracle as q


def bf16_bits(values):
    """Exactly representable values -> bf16 bit patterns (asserted)."""
    f = np.asarray(values, dtype=np.float32)
    u = f.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "test value is not a bf16 number"
    return (u >> 16).astype(np.uint16)


def frac_of_f32(v) -> Fraction:
    return Fraction(struct.unpack("<f", struct.pack("<f", float(v)))[0])


def brute_argmin(w, cb_values):
    """argmin_j |w - c_j| in exact rational arithmetic, first minimum."""
    fw = frac_of_f32(w)
    best, arg = None, 0
    for j, c in enumerate(cb_values):
        d = abs(fw - Fraction(float(c)))
        if best is None or d < best:
            best, arg = d, j
    return arg


# ---------------------------------------------------------------- nearest centroid (Eq. "centroid quantizer")
@pytest.mark.parametrize("bits", (1, 2, 4))
def test_nearest_centroid_equals_exact_rational_argmin(bits):
    rng = np.random.default_rng(bits)
    Q = 1 << bits
    N, K = 6, 40
    cbv = np.sort((rng.integers(-120, 120, size=(N, Q)) / 64.0).astype(np.float32), axis=1)   # bf16-exact, with ties
    cbv[1, :] = cbv[1, 0]                                   # all centroids equal
    if Q > 2:
        cbv[2, 1] = cbv[2, 2]                               # a duplicated pair
    W = (rng.integers(-130, 130, size=(N, K)) / 128.0).astype(np.float32)   # many values exactly on midpoints
    W[3, :Q] = cbv[3]                                       # values equal to centroids
    got = q.nearest_centroid(W, bf16_bits(cbv))
    for n in range(N):
        for k in range(K):
            assert got[n, k] == brute_argmin(W[n, k], cbv[n]), (n, k)


def test_nearest_centroid_on_badly_scaled_values():
    """|w - c| computed in floating point ties where the exact distances differ; the midpoint form does not."""
    cbv = np.array([[-1.0, 1.0], [-2.0 ** -100, 2.0 ** 100], [-1.0, 2.0 ** -120]], dtype=np.float32)
    W = np.array([[1e-30, -1e-30, 0.0, -0.0], [1.0, 2.0 ** 99, 2.0 ** 99 * (1 + 2.0 ** -23), -1.0],
                  [-0.5, -0.5 + 2.0 ** -24, -0.5 - 2.0 ** -24, 1.0]], dtype=np.float32)
    got = q.nearest_centroid(W, bf16_bits(cbv))
    for n in range(3):
        for k in range(4):
            assert got[n, k] == brute_argmin(W[n, k], cbv[n]), (n, k)


def test_nearest_centroid_planted_mistakes_fail():
    cbv = np.array([[-1.0, 0.0, 0.0, 1.0]], dtype=np.float32)
    W = np.array([[-0.5, 0.5, 0.25, 0.0]], dtype=np.float32)
    want = [brute_argmin(w, cbv[0]) for w in W[0]]
    assert want == [0, 1, 1, 1]
    assert list(q.nearest_centroid(W, bf16_bits(cbv))[0]) == want
    # tie to the upper centroid
    mids = 0.5 * (cbv[0, :-1] + cbv[0, 1:])
    upper = [int(np.sum(w >= mids)) for w in W[0]]
    assert upper != want
    # duplicates not folded to the lowest index
    nofold = [int(np.sum(w > mids)) for w in W[0]]
    assert nofold != want


# ---------------------------------------------------------------- start and iteration
@pytest.mark.parametrize("Q", (2, 4, 16, 256))
def test_quantile_start_equals_numpy_quantiles(Q):
    rng = np.random.default_rng(Q)
    v = rng.standard_normal(1000)
    want = np.quantile(v, (np.arange(Q) + 0.5) / Q, method="linear")
    np.testing.assert_allclose(q.quantile_start(v, Q), want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("bits,K,iters", ((1, 5000, 2), (2, 1000, 4), (4, 4096, 7)))
def test_lloyd_equals_sklearn_lloyd_from_the_same_start(bits, K, iters):
    cluster = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(10 + bits)
    v = (rng.standard_normal(K) * 0.02).astype(np.float32)
    Q = 1 << bits
    start = q.quantile_start(v, Q)
    km = cluster.KMeans(n_clusters=Q, init=start.reshape(-1, 1), n_init=1, max_iter=iters, tol=0.0, algorithm="lloyd")
    km.fit(v.astype(np.float64).reshape(-1, 1))
    assert km.n_iter_ == iters, "the library stopped early; pick a case that has not converged"
    got = q.lloyd_1d(v, bits, iters)
    np.testing.assert_allclose(got, km.cluster_centers_[:, 0], rtol=1e-10, atol=1e-14)


def sse(v, c):
    return float(np.min((v[:, None] - c[None, :]) ** 2, axis=1).sum())


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_lloyd_error_never_increases_and_ends_in_a_fixed_point(bits):
    rng = np.random.default_rng(20 + bits)
    v = rng.laplace(0, 0.014, 2000)
    errs = [sse(v, q.lloyd_1d(v, bits, it)) for it in range(0, 12)]
    assert all(b <= a * (1 + 1e-12) for a, b in zip(errs, errs[1:]))
    assert errs[-1] < errs[0]
    c = q.lloyd_1d(v, bits, 400)
    nearest = np.argmin(np.abs(v[:, None] - c[None, :]), axis=1)
    for j in range(1 << bits):
        assert np.any(nearest == j)
        np.testing.assert_allclose(c[j], v[nearest == j].mean(), rtol=1e-9)
    assert np.all(np.diff(c) > 0)


def test_lloyd_closed_forms():
    # two separated clusters: the 1-bit fit is the pair of cluster means, after one iteration
    rng = np.random.default_rng(3)
    a, b = rng.uniform(-2, -1, 500), rng.uniform(3, 5, 300)
    c = q.lloyd_1d(np.concatenate([a, b]), 1, 1)
    np.testing.assert_allclose(c, [a.mean(), b.mean()], rtol=1e-12)
    # values on a uniform grid of 4 levels, any multiplicities: the 2-bit fit is the grid
    v = np.repeat([-3.0, -1.0, 1.0, 3.0], [5, 9, 2, 7])
    np.testing.assert_allclose(q.lloyd_1d(v, 2, 20), [-3, -1, 1, 3], rtol=0, atol=1e-15)
    # 1-bit optimum of a Gaussian: +- sigma * sqrt(2 / pi) (Lloyd-Max), to sampling error
    g = np.random.default_rng(4).standard_normal(400000) * 0.02
    c = q.lloyd_1d(g, 1, 30)
    np.testing.assert_allclose(c, [-0.02 * np.sqrt(2 / np.pi), 0.02 * np.sqrt(2 / np.pi)], rtol=1e-2)
    # fewer distinct values than centroids: nothing breaks, every value is reproduced exactly
    v = np.array([0.5] * 10 + [-0.25] * 3)
    c = q.lloyd_1d(v, 2, 5)
    assert np.all(np.diff(c) >= 0)
    idx = np.argmin(np.abs(v[:, None] - c[None, :]), axis=1)
    np.testing.assert_array_equal(c[idx], v)


def test_lloyd_empty_cluster_keeps_its_centroid():
    v = np.array([0.0] * 8 + [1.0] * 8)
    start = np.array([0.0, 0.4, 0.45, 1.0])          # nothing is nearest to 0.4 or 0.45
    c = q.lloyd_1d(v, 2, 3, start=start)
    np.testing.assert_array_equal(c, start)


def test_lloyd_planted_mistakes_fail():
    rng = np.random.default_rng(5)
    v = rng.standard_normal(777)
    good = q.lloyd_1d(v, 2, 6)

    def variant(assign_upper=False, median=False):
        c = q.quantile_start(v, 4)
        for _ in range(6):
            mids = 0.5 * (c[:-1] + c[1:])
            idx = np.sum(v[:, None] >= mids[None, :], axis=1) if assign_upper else np.sum(v[:, None] > mids[None, :], axis=1)
            for j in range(4):
                m = v[idx == j]
                if m.size:
                    c[j] = np.median(m) if median else m.mean()
        return c
    np.testing.assert_allclose(variant(), good, rtol=1e-13)          # the restatement itself agrees
    assert np.max(np.abs(variant(median=True) - good)) > 1e-6
    start_shifted = q.lloyd_1d(v, 2, 6, start=np.quantile(v, np.arange(4) / 4))
    assert np.max(np.abs(start_shifted - good)) > 1e-9


def test_centroids_to_bf16_is_round_to_nearest_even():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(6)
    c = np.concatenate([rng.standard_normal(4000) * 0.02, [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 0.0, 2.0 ** -130]])
    want = torch.from_numpy(c).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(q.centroids_to_bf16(c), want)
    # a zero of either sign, and a negative value that rounds to zero, are stored as +0
    np.testing.assert_array_equal(q.centroids_to_bf16(np.array([-0.0, 0.0, -1e-60])), [0, 0, 0])


# ---------------------------------------------------------------- block scales and normalisation
def test_block_scales_against_exact_arithmetic():
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((3, 128)) * 0.02).astype(np.float32)
    W[1, 64:] = 0.0
    W[2, :64] = 2.0 ** -140                        # absmean and absmax far below the bf16 normal range
    for mode in (q.ABSMAX, q.ABSMEAN):
        got = q.block_scales(W, mode)
        for n in range(3):
            for g in range(2):
                blk = [abs(frac_of_f32(w)) for w in W[n, 64 * g:64 * g + 64]]
                lam = max(blk) if mode == q.ABSMAX else sum(blk) / 64
                f = np.float32(float(lam))             # Fraction -> double is correctly rounded, then -> float32
                want = q.f32_to_bf16_rne(np.array([f]))[0]
                if lam == 0 or (int(want) << 16) == 0:
                    want = 0x3F80
                assert got[n, g] == want, (mode, n, g)
    assert q.block_scales(W, q.ABSMAX)[1, 1] == 0x3F80


def test_normalise_and_block_assign_by_brute_force():
    rng = np.random.default_rng(8)
    W = (rng.standard_normal((2, 128)) * 0.02).astype(np.float32)
    s = q.block_scales(W, q.ABSMAX)
    norm = q.normalise(W, s)
    assert np.max(np.abs(norm)) <= 1.0 + 2.0 ** -8
    cbv = np.array([-1.0, -0.25, 0.25, 0.75], dtype=np.float32)
    idx = q.block_assign(W, s, bf16_bits(cbv))
    sv = (s.astype(np.uint32) << 16).view(np.float32)
    for n in range(2):
        for k in range(128):
            r = frac_of_f32(W[n, k]) / frac_of_f32(sv[n, k // 64])
            d = [abs(r - Fraction(float(c))) for c in cbv]
            # the float64 quotient is within 2^-53 of r; no distance pair here is that close to a tie
            srt = sorted(d)
            assert srt[1] - srt[0] > Fraction(1, 2 ** 40)
            assert idx[n, k] == d.index(min(d))
            assert abs(Fraction(norm[n, k]) - r) <= Fraction(1, 2 ** 52)
    # under absmean the normalised weights leave [-1, 1]; nothing is clipped
    assert np.max(np.abs(q.normalise(W, q.block_scales(W, q.ABSMEAN)))) > 2.0


def test_strided_sample_rule():
    W = np.arange(4 * 128, dtype=np.float32).reshape(4, 128) / 512 - 0.5
    s = np.full((4, 2), 0x3F80, dtype=np.uint16)     # all scales 1
    got = q.strided_sample(W, s, 100)
    want = W.reshape(-1)[::5][:100]
    np.testing.assert_array_equal(got, want)
    assert q.strided_sample(W, s, 10 ** 6).size == 512
