"""GPU parity of the quantiser side (kmq_kmeans_rows, kmq_assign_pack, kmq_quantize_rows, kmq_block_scales,
kmq_block_sample, kmq_block_assign_pack, kmq_block_quantize) against oracle/kmq_quant_oracle.py.

Bars: indices, packed words, scales and samples bit-exact; fitted centroids within 1e-10 of the row's largest
magnitude in float64 (the two sides add the same numbers in a different order) and the stored bf16 codebooks equal,
except that a centroid whose unrounded value sits within 1e-9 (relative) of a rounding boundary may differ by one
step."""
import numpy as np
import pytest
import torch

from oracle import kmq_block_oracle as borc
from oracle import kmq_oracle as orc
from oracle import kmq_quant_oracle as qorc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
C, T, L = kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TUNED, kmq.KMQ_LAYOUT_TABLE


def bf16_to_f64(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def draw_rows(dist, N, K, seed):
    rng = np.random.default_rng(seed)
    if dist == "normal":
        return (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    if dist == "laplace":
        return rng.laplace(0, 0.014, (N, K)).astype(np.float32)
    if dist == "student_t":
        return (rng.standard_t(5, (N, K)) * 0.02 / np.sqrt(5 / 3)).astype(np.float32)
    raise ValueError(dist)


def degenerate_rows(K, Q, seed):
    """Rows on which a fit can go wrong: constant, two values, fewer distinct values than centroids, sorted and
    reversed input, signed zeros, one outlier, a few values repeated many times."""
    rng = np.random.default_rng(seed)
    rows = [np.full(K, 0.25), np.where(np.arange(K) % 3 == 0, -1.0, 2.0), np.sort(rng.standard_normal(K)),
            np.sort(rng.standard_normal(K))[::-1], np.where(np.arange(K) % 2 == 0, 0.0, -0.0),
            np.concatenate([[1000.0], rng.standard_normal(K - 1) * 1e-3]),
            rng.choice(rng.standard_normal(max(2, Q // 2)), K), rng.integers(-3, 4, K) / 4.0,
            rng.standard_normal(K) * 2.0 ** rng.integers(-20, 20, K)]
    return np.stack(rows).astype(np.float32)


def gpu_fit(W, bits, iters=20):
    N, K = W.shape
    Q = 1 << bits
    d_w = torch.from_numpy(W).cuda()
    cbuf, coff = gu.dev_bytes(N * Q * 2)
    fbuf, foff = gu.dev_bytes(N * Q * 8)
    kmq.kmq_kmeans_rows(d_w, N, K, bits, iters, cbuf.data_ptr() + coff, fbuf.data_ptr() + foff)
    torch.cuda.synchronize()
    assert gu.canaries_intact(cbuf, coff, N * Q * 2) and gu.canaries_intact(fbuf, foff, N * Q * 8)
    cb = cbuf[coff:coff + N * Q * 2].cpu().numpy().view(np.uint16).reshape(N, Q)
    cent = fbuf[foff:foff + N * Q * 8].cpu().numpy().view(np.float64).reshape(N, Q)
    return cb, cent


def check_fit(W, bits, iters=20):
    cb, cent = gpu_fit(W, bits, iters)
    want = qorc.lloyd_rows(W, bits, iters)
    scale = np.abs(W).max(axis=1, keepdims=True).astype(np.float64) + 1e-300
    err = np.abs(cent - want) / scale
    assert err.max() <= 1e-10, f"centroids differ: {err.max()} (row {np.argmax(err.max(axis=1))})"
    assert np.all(np.diff(cent, axis=1) >= 0)
    want_cb = qorc.centroids_to_bf16(want)
    bad = np.argwhere(cb != want_cb)
    for n, j in bad:
        # only a value on a rounding boundary may land on either side
        lo, hi = sorted((bf16_to_f64(cb[n, j]), bf16_to_f64(want_cb[n, j])))
        assert abs(int(cb[n, j]) - int(want_cb[n, j])) == 1 and abs(want[n, j] - 0.5 * (lo + hi)) <= 1e-9 * abs(hi)
    assert len(bad) <= 1
    return cb


@pytest.mark.parametrize("dist", ("normal", "laplace", "student_t"))
@pytest.mark.parametrize("K", (64, 1000, 4096))
@pytest.mark.parametrize("bits", (1, 2, 4))
def test_kmeans_rows_matches_the_oracle(bits, K, dist):
    check_fit(draw_rows(dist, 20, K, 7 * bits + K), bits)


@pytest.mark.parametrize("bits,K,N", ((1, 28672, 3), (4, 28672, 3), (8, 32768, 1), (8, 5000, 2), (8, 256, 2), (8, 300, 1), (4, 1024, 2), (4, 1025, 2), (2, 2, 3), (1, 3, 2)))
def test_kmeans_rows_long_short_and_8_bit(bits, K, N):
    if K < (1 << bits):
        pytest.skip("fewer values than centroids")
    check_fit(draw_rows("laplace", N, K, K + bits), bits)


@pytest.mark.parametrize("iters", (0, 1, 3))
def test_kmeans_rows_iteration_count(iters):
    check_fit(draw_rows("normal", 5, 777, iters), 2, iters)


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_kmeans_rows_degenerate_rows(bits):
    check_fit(degenerate_rows(520, 1 << bits, bits), bits)


def test_kmeans_rows_more_rows_than_resident_ctas_and_rerun_identical():
    W = draw_rows("normal", 700, 256, 3)
    cb1, cent1 = gpu_fit(W, 2)
    cb2, cent2 = gpu_fit(W, 2)
    np.testing.assert_array_equal(cent1, cent2)
    want = qorc.lloyd_rows(W[::37], 2)
    np.testing.assert_allclose(cent1[::37], want, rtol=0, atol=1e-10 * 0.1)
    np.testing.assert_array_equal(cb1[::37], qorc.centroids_to_bf16(want))


# ------------------------------------------------------------------------------------------- assignment + packing
def skewed_codebooks(bits, N, rng):
    """Sorted bf16 codebooks: k-means-like, with duplicates, with zeros of both signs, badly scaled."""
    Q = 1 << bits
    cb = np.sort(rng.standard_normal((N, Q)) * 0.02, axis=1)
    cb[0] = 0.5
    if Q >= 4:
        cb[1, 1] = cb[1, 2]
        cb[2, :2] = (-0.0, 0.0)
        cb[2] = np.sort(cb[2])
    cb[3] = np.sort(np.concatenate([[-2.0 ** -100, 2.0 ** 100], np.linspace(-1, 1, Q)[: Q - 2]]))[:Q]
    return synth.f32_to_bf16_bits(np.sort(cb, axis=1).astype(np.float32))


def weights_near_midpoints(cb_bits, K, rng):
    """Random weights; a third of them exactly on a midpoint of two stored centroids or one float32 step off."""
    N, Q = cb_bits.shape
    cb = bf16_to_f64(cb_bits)
    W = (rng.standard_normal((N, K)) * 0.03).astype(np.float32)
    mids = (0.5 * (cb[:, :-1] + cb[:, 1:])).astype(np.float32)
    pick = rng.integers(0, Q - 1, (N, K)) if Q > 2 else np.zeros((N, K), dtype=np.int64)
    on = np.take_along_axis(mids, pick, axis=1)
    step = rng.integers(-1, 2, (N, K))
    near = np.where(step == 0, on, np.nextafter(on, np.where(step > 0, np.float32(np.inf), np.float32(-np.inf))))
    use = rng.random((N, K)) < 0.33
    return np.where(use, near, W).astype(np.float32)


@pytest.mark.parametrize("layout", (C, T, L))
@pytest.mark.parametrize("N,K", ((37, 256), (16, 2048 + 128), (5, 96 * 4)))
@pytest.mark.parametrize("bits", (1, 2, 4))
def test_assign_pack_is_bit_exact(bits, N, K, layout):
    rng = np.random.default_rng(bits * 1000 + N + K)
    cb = skewed_codebooks(bits, N, rng)
    W = weights_near_midpoints(cb, K, rng)
    want_idx = qorc.nearest_centroid(W, cb)
    nbytes = kmq.kmq_packed_bytes(N, K, bits, layout)
    buf, off = gu.dev_bytes(nbytes)
    kmq.kmq_assign_pack(torch.from_numpy(W).cuda(), gu.to_dev_u16(cb), N, K, bits, layout, buf.data_ptr() + off)
    torch.cuda.synchronize()
    assert gu.canaries_intact(buf, off, nbytes)
    got = buf[off:off + nbytes].view(torch.int32)
    np.testing.assert_array_equal(gu.gpu_unpack(got, N, K, bits, layout), want_idx)
    # and the packed bytes themselves, padding included, equal kmq_pack of the oracle's indices
    ref = gu.gpu_pack(want_idx, bits, layout)
    assert torch.equal(got, ref)
    if layout == C:
        np.testing.assert_array_equal(gu.packed_to_numpy(got, N), orc.pack_canonical(want_idx, bits))


@pytest.mark.parametrize("bits,layout", ((1, L), (2, T), (4, T), (4, C)))
def test_quantize_rows_then_linear(bits, layout):
    """The whole chain on the GPU (fit, assign, pack, layer) against the whole chain of oracles, and against the
    seeded input generator, which follows the same recipe with its own code."""
    N, K, M = 64, 1024, 2
    layer = synth.make_layer(N, K, bits, M, dist="student_t", config_id=3, keep_weights=True)
    W = layer["W"]
    d_cb = torch.empty(N * (1 << bits), dtype=torch.int16, device="cuda")
    nbytes = kmq.kmq_packed_bytes(N, K, bits, layout)
    packed = torch.empty(nbytes // 4, dtype=torch.int32, device="cuda")
    kmq.kmq_quantize_rows(torch.from_numpy(W).cuda(), N, K, bits, 20, layout, d_cb, packed)
    torch.cuda.synchronize()
    cb = d_cb.cpu().numpy().view(np.uint16).reshape(N, -1)
    want_cb = qorc.centroids_to_bf16(qorc.lloyd_rows(W, bits))
    np.testing.assert_array_equal(cb, want_cb)
    want_idx = qorc.nearest_centroid(W, want_cb)
    np.testing.assert_array_equal(gu.gpu_unpack(packed, N, K, bits, layout), want_idx)
    np.testing.assert_array_equal(cb, layer["codebooks"])
    np.testing.assert_array_equal(want_idx, layer["idx"])
    y = gu.gpu_linear(packed, cb, layer["x"], N, K, bits, layout)
    y_ref, s = orc.linear_f64(orc.pack_canonical(want_idx, bits), want_cb, layer["x"], K, bits)
    assert orc.check_linear(y, y_ref, s) <= 1.0
    # the quantised layer is close to the unquantised one: relative error of W^ against W as 1-D k-means predicts
    w_hat = bf16_to_f64(np.take_along_axis(cb, want_idx.astype(np.int64), axis=1))
    rel = np.linalg.norm(w_hat - W) / np.linalg.norm(W)
    assert rel < {1: 0.75, 2: 0.5, 4: 0.2}[bits], rel


@pytest.mark.parametrize("N,K,bits", ((4096, 4096, 4), (4096, 4096, 1), (8192, 28672, 1), (3072, 8192, 2)))
def test_quantize_rows_full_size_sampled_rows(N, K, bits):
    g = torch.Generator(device="cuda").manual_seed(N + K + bits)
    d_w = torch.randn((N, K), generator=g, device="cuda", dtype=torch.float32) * 0.02
    layout = kmq.kmq_preferred_layout(N, K, bits, 1)
    Q = 1 << bits
    d_cb = torch.full((N * Q,), -1, dtype=torch.int16, device="cuda")
    packed = torch.empty(kmq.kmq_packed_bytes(N, K, bits, layout) // 4, dtype=torch.int32, device="cuda")
    kmq.kmq_quantize_rows(d_w, N, K, bits, 20, layout, d_cb, packed)
    torch.cuda.synchronize()
    cb = d_cb.cpu().numpy().view(np.uint16).reshape(N, Q)
    assert np.all(np.diff(bf16_to_f64(cb), axis=1) >= 0)
    rows = np.unique(np.concatenate([[0, 1, 15, 16, N - 17, N - 1], np.random.default_rng(1).integers(0, N, 10)]))
    W = d_w[torch.from_numpy(rows).cuda()].cpu().numpy()
    want_cb = qorc.centroids_to_bf16(qorc.lloyd_rows(W, bits))
    np.testing.assert_array_equal(cb[rows], want_cb)
    idx = torch.empty((N, K), dtype=torch.uint8, device="cuda")
    kmq.kmq_unpack(packed, N, K, bits, idx, layout=layout)
    got_idx = idx[torch.from_numpy(rows).cuda()].cpu().numpy()
    np.testing.assert_array_equal(got_idx, qorc.nearest_centroid(W, want_cb))
    # every row: the assignment is the nearest centroid (property checked on the device, all N*K weights)
    cbf = torch.from_numpy(cb.view(np.int16)).cuda().view(torch.bfloat16).to(torch.float64).reshape(N, Q)
    for r0 in range(0, N, 512):
        w = d_w[r0:r0 + 512].to(torch.float64)
        d_all = (w[:, :, None] - cbf[r0:r0 + 512, None, :]).abs() if Q <= 4 else None
        chosen = torch.gather(cbf[r0:r0 + 512], 1, idx[r0:r0 + 512].long())
        if d_all is not None:
            assert torch.all((w - chosen).abs() <= d_all.min(dim=2).values)
        else:
            for j in range(Q):
                assert torch.all((w - chosen).abs() <= (w - cbf[r0:r0 + 512, j:j + 1]).abs())


# ------------------------------------------------------------------------------------------------- block format
@pytest.mark.parametrize("lam", (kmq.KMQ_LAMBDA_ABSMAX, kmq.KMQ_LAMBDA_ABSMEAN))
def test_block_scales_bit_exact(lam):
    rng = np.random.default_rng(lam)
    W = (rng.standard_normal((33, 64 * 7)) * 0.02 * 2.0 ** rng.integers(-30, 30, (33, 1))).astype(np.float32)
    W[1, 64:128] = 0.0
    W[2, :64] = 2.0 ** -140
    N, K = W.shape
    buf, off = gu.dev_bytes(N * K // 64 * 2)
    kmq.kmq_block_scales(torch.from_numpy(W).cuda(), N, K, lam, buf.data_ptr() + off)
    torch.cuda.synchronize()
    assert gu.canaries_intact(buf, off, N * K // 64 * 2)
    got = buf[off:off + N * K // 64 * 2].cpu().numpy().view(np.uint16).reshape(N, K // 64)
    np.testing.assert_array_equal(got, qorc.block_scales(W, lam))


@pytest.mark.parametrize("samples", (100, 4096, 10 ** 6))
def test_block_sample_bit_exact(samples):
    rng = np.random.default_rng(samples)
    W = (rng.standard_normal((24, 256)) * 0.02).astype(np.float32)
    N, K = W.shape
    s = qorc.block_scales(W, qorc.ABSMAX)
    want = qorc.strided_sample(W, s, samples)
    assert kmq.kmq_block_sample_count(N, K, samples) == want.size
    buf, off = gu.dev_bytes(want.size * 4)
    kmq.kmq_block_sample(torch.from_numpy(W).cuda(), gu.to_dev_u16(s), N, K, samples, buf.data_ptr() + off)
    torch.cuda.synchronize()
    assert gu.canaries_intact(buf, off, want.size * 4)
    got = buf[off:off + want.size * 4].cpu().numpy().view(np.float32)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("bits", (1, 2, 4, 8))
def test_block_assign_pack_bit_exact(bits):
    rng = np.random.default_rng(40 + bits)
    N, K = 19, 64 * 5
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    s = qorc.block_scales(W, qorc.ABSMAX)
    Q = 1 << bits
    cbv = np.sort(np.clip(rng.standard_normal(Q) * 0.4, -1, 1))
    if Q >= 4:
        cbv[1] = cbv[2]
    cb = synth.f32_to_bf16_bits(np.sort(cbv).astype(np.float32))
    # put a fifth of the weights exactly on a midpoint of the normalised grid (scale * midpoint, where that is exact)
    c64 = bf16_to_f64(cb)
    mids = 0.5 * (c64[:-1] + c64[1:])
    sv = bf16_to_f64(s).repeat(64, axis=1)
    on = (sv * mids[rng.integers(0, Q - 1, (N, K))]).astype(np.float32)
    W = np.where(rng.random((N, K)) < 0.2, on, W).astype(np.float32)
    want = qorc.block_assign(W, s, cb)
    nbytes = kmq.kmq_block_packed_bytes(N, K, bits)
    buf, off = gu.dev_bytes(nbytes)
    kmq.kmq_block_assign_pack(torch.from_numpy(W).cuda(), gu.to_dev_u16(s), gu.to_dev_u16(cb), N, K, bits,
                              buf.data_ptr() + off)
    torch.cuda.synchronize()
    assert gu.canaries_intact(buf, off, nbytes)
    got = buf[off:off + nbytes].cpu().numpy().reshape(N, -1)
    np.testing.assert_array_equal(got, borc.pack_bytes(want, bits))


@pytest.mark.parametrize("bits,lam", ((1, 0), (2, 1), (4, 0), (8, 0)))
def test_block_quantize_end_to_end(bits, lam):
    rng = np.random.default_rng(50 + bits)
    N, K, samples = 96, 1024, 20000
    W = (rng.standard_t(5, (N, K)) * 0.02).astype(np.float32)
    d_s = torch.empty(N * K // 64, dtype=torch.int16, device="cuda")
    d_cb = torch.empty(max(8, 1 << bits), dtype=torch.int16, device="cuda")
    d_wq = torch.empty(kmq.kmq_block_packed_bytes(N, K, bits), dtype=torch.uint8, device="cuda")
    d_ws = torch.empty(samples, dtype=torch.float32, device="cuda")
    kmq.kmq_block_quantize(torch.from_numpy(W).cuda(), N, K, bits, lam, 20, samples, d_s, d_cb, d_wq, d_ws)
    torch.cuda.synchronize()
    s = qorc.block_scales(W, lam)
    np.testing.assert_array_equal(d_s.cpu().numpy().view(np.uint16).reshape(N, -1), s)
    sample = qorc.strided_sample(W, s, samples)
    cb = qorc.centroids_to_bf16(qorc.lloyd_1d(sample, bits, 20))
    np.testing.assert_array_equal(d_cb.cpu().numpy().view(np.uint16)[:1 << bits], cb)
    if lam == kmq.KMQ_LAMBDA_ABSMAX:
        assert np.all(np.abs(bf16_to_f64(cb)) <= 1.0 + 2.0 ** -8)
    idx = qorc.block_assign(W, s, cb)
    np.testing.assert_array_equal(d_wq.cpu().numpy().reshape(N, -1), borc.pack_bytes(idx, bits))
    # the quantised tensor reproduces W to the accuracy the bit width allows
    w_hat = bf16_to_f64(cb)[idx] * bf16_to_f64(s).repeat(64, axis=1)
    rel = np.linalg.norm(w_hat - W) / np.linalg.norm(W)
    assert rel < {1: 0.8, 2: 0.5, 4: 0.2, 8: 0.03}[bits], rel
