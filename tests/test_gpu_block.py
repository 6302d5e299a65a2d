"""GPU parity of the paper's k-means block format (kmq_block_*) against oracle/kmq_block_oracle.py: packed bytes
and dequantised weights bit for bit, outputs of both scale orders within |y - y_ref| <= 2^-7 * sum_k |x_k * w_k| +
1e-6, for b = 1, 2, 4, 8."""
import numpy as np
import pytest
import torch

from oracle import kmq_block_oracle as blk
from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
BITS = (1, 2, 4, 8)


def run_all(idx, scales, cb, x, bits, what):
    N, K = idx.shape
    M = x.shape[0]
    ref_wq = blk.pack_bytes(idx, bits)
    d_idx = torch.from_numpy(np.ascontiguousarray(idx)).cuda()
    nbytes = kmq.kmq_block_packed_bytes(N, K, bits)
    assert nbytes == ref_wq.size
    buf, off = gu.dev_bytes(nbytes)
    kmq.kmq_block_pack(d_idx, N, K, bits, buf.data_ptr() + off)
    torch.cuda.synchronize()
    assert gu.canaries_intact(buf, off, nbytes), f"{what}: pack wrote outside its buffer"
    wq = buf[off:off + nbytes]
    assert np.array_equal(wq.cpu().numpy().reshape(N, -1), ref_wq), f"{what}: packed bytes differ"

    d_s, d_cb, d_x = gu.to_dev_u16(scales), gu.to_dev_u16(cb), gu.to_dev_u16(x)
    wbuf, woff = gu.dev_bytes(N * K * 2)
    kmq.kmq_block_dequant_to_bf16(wq, d_s, d_cb, wbuf.data_ptr() + woff, N, K, bits)
    torch.cuda.synchronize()
    assert gu.canaries_intact(wbuf, woff, N * K * 2), f"{what}: dequant wrote outside W"
    got_w = wbuf[woff:woff + N * K * 2].cpu().numpy().view(np.uint16).reshape(N, K)
    assert np.array_equal(got_w, blk.dequant_scaled_bits(ref_wq, scales, cb, K, bits)), f"{what}: weights differ"

    y_ref, s_abs = blk.block_linear_f64(ref_wq, scales, cb, x, K, bits)
    worst = 0.0
    for order in (kmq.KMQ_SCALE_DIRECT, kmq.KMQ_SCALE_DEFERRED):
        ybuf, yoff = gu.dev_bytes(M * N * 2)
        kmq.kmq_block_linear(wq, d_s, d_cb, d_x, ybuf.data_ptr() + yoff, N, K, bits, M, scale_order=order)
        torch.cuda.synchronize()
        assert gu.canaries_intact(ybuf, yoff, M * N * 2), f"{what}: linear wrote outside y"
        y = ybuf[yoff:yoff + M * N * 2].cpu().numpy().view(np.uint16).reshape(M, N)
        ratio = orc.check_linear(y, y_ref, s_abs)
        assert ratio <= 1.0, f"{what} order={order}: error/tolerance = {ratio}"
        worst = max(worst, ratio)
    if bits != 8:
        worst = max(worst, run_table(wq, ref_wq, d_s, scales, d_cb, d_x, y_ref, s_abs, N, K, M, bits, what))
    return worst


def run_table(wq, ref_wq, d_s, scales, d_cb, d_x, y_ref, s_abs, N, K, M, bits, what):
    """The activation-table path: layout bytes against the documented formulas, round trip, parity of the layer."""
    tbytes = kmq.kmq_block_table_bytes(N, K, bits)
    tbuf, toff = gu.dev_bytes(tbytes)
    kmq.kmq_block_table_pack(wq, d_s, N, K, bits, tbuf.data_ptr() + toff)
    torch.cuda.synchronize()
    assert gu.canaries_intact(tbuf, toff, tbytes), f"{what}: table pack wrote outside its buffer"
    tab = tbuf[toff:toff + tbytes]
    if N * K <= 1 << 21:
        want = gu.block_table_from_bytes(ref_wq, scales, K, bits)
        assert want.size == tbytes
        assert np.array_equal(tab.cpu().numpy(), want), f"{what}: table bytes differ from the documented layout"
    wq2, s2 = torch.zeros_like(wq), torch.zeros_like(d_s)
    kmq.kmq_block_table_unpack(tab, N, K, bits, wq2, s2)
    torch.cuda.synchronize()
    assert torch.equal(wq2, wq) and torch.equal(s2, d_s), f"{what}: table unpack is not the inverse of pack"
    wsb = kmq.kmq_block_table_workspace_bytes(N, K, bits)
    ws = torch.full((max(wsb, 16),), 0xFF, dtype=torch.uint8, device="cuda")     # NaN patterns: contents are ignored
    ybuf, yoff = gu.dev_bytes(M * N * 2)
    kmq.kmq_block_table_linear(tab, d_cb, d_x, ybuf.data_ptr() + yoff, N, K, bits, M, ws, wsb)
    torch.cuda.synchronize()
    assert gu.canaries_intact(ybuf, yoff, M * N * 2), f"{what}: table linear wrote outside y"
    assert kmq.kmq_device_error_flags() == 0
    y = ybuf[yoff:yoff + M * N * 2].cpu().numpy().view(np.uint16).reshape(M, N)
    ratio = orc.check_linear(y, y_ref, s_abs)
    assert ratio <= 1.0, f"{what} table: error/tolerance = {ratio}"
    y2 = torch.empty(M * N, dtype=torch.int16, device="cuda")
    kmq.kmq_block_table_linear(tab, d_cb, d_x, y2, N, K, bits, M, ws, wsb)
    torch.cuda.synchronize()
    assert np.array_equal(y2.cpu().numpy().view(np.uint16).reshape(M, N), y), f"{what}: table linear not reproducible"
    return ratio


@pytest.mark.parametrize("bits", BITS)
def test_tiny_layer_of_the_block_format(bits):
    L = synth.make_block_layer(256, 256, bits, 1, "normal", config_id=1)
    run_all(L["idx"], L["scales"], L["codebook"], L["x"], bits, f"256x256 b={bits}")


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("N,K,M", [(1, 64, 1), (3, 128, 2), (17, 192, 3), (130, 2112, 4), (259, 4096, 5), (64, 64, 8),
                                   (1000, 1024, 1), (33, 28672, 2)])
def test_ragged_shapes_random_inputs(bits, N, K, M):
    rng = np.random.default_rng(100 * bits + N + M)
    idx = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    cb = synth.f32_to_bf16_bits(np.sort(rng.uniform(-1, 1, 1 << bits)).astype(np.float32))
    scales = synth.f32_to_bf16_bits(np.abs(rng.standard_normal((N, K // 64)) * 0.02).astype(np.float32))
    x = synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    run_all(idx, scales, cb, x, bits, f"N={N} K={K} M={M} b={bits}")


@pytest.mark.parametrize("bits", BITS)
def test_degenerate_scales_and_codebooks(bits):
    """Blocks with scale 0, 2^-40 and 2^20 side by side; a codebook with -0.0, duplicates and +-1; activations of
    very different magnitudes."""
    rng = np.random.default_rng(bits)
    N, K, M = 48, 1024, 2
    Q = 1 << bits
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    vals = np.array([-1.0, -0.0, 0.0, 1.0, 0.5, 0.5, -2.0 ** -20, 2.0 ** -20], np.float32)
    cb = synth.f32_to_bf16_bits(np.sort(np.resize(vals, Q)))
    sc = rng.choice(np.array([0.0, 2.0 ** -40, 2.0 ** 20, 1.0, 0.0123], np.float32), size=(N, K // 64))
    x = synth.f32_to_bf16_bits((rng.standard_normal((M, K)) * 2.0 ** rng.uniform(-10, 6, (M, K))).astype(np.float32))
    run_all(idx, synth.f32_to_bf16_bits(sc), cb, x, bits, f"degenerate b={bits}")


@pytest.mark.parametrize("bits", (1, 4))
def test_square_4096_every_row(bits):
    L = synth.make_block_layer(4096, 4096, bits, 1, "normal", config_id=2)
    run_all(L["idx"], L["scales"], L["codebook"], L["x"], bits, f"4096x4096 b={bits}")


def test_validation():
    a = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    assert kmq.kmq_block_linear(a, a, a, a, a, 4, 64, 3, 1, check=False) == kmq.KMQ_ERR_BITS
    assert kmq.kmq_block_linear(a, a, a, a, a, 4, 96, 4, 1, check=False) == kmq.KMQ_ERR_SHAPE
    assert kmq.kmq_block_linear(a, a, a, a, a, 4, 64, 4, 1, scale_order=5, check=False) == kmq.KMQ_ERR_LAYOUT
    assert kmq.kmq_block_linear(a, None, a, a, a, 4, 64, 4, 1, check=False) == kmq.KMQ_ERR_NULL
    assert kmq.kmq_block_packed_bytes(4, 96, 4) == 0


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_table_path_skewed_shared_codebooks(bits):
    """Codebooks whose entries differ by many orders of magnitude, rows that use one centroid only: a table entry must
    be the sum of the selected products, not a difference of sums."""
    rng = np.random.default_rng(70 + bits)
    N, K, M = 80, 2048, 1
    Q = 1 << bits
    for vals in ([-1.0, 2.0 ** -20], [0.0, 1.0], [-300.0, 2.0 ** -10], [0.5, 0.5]):
        cbv = np.sort(np.resize(np.array(vals, np.float32), Q))
        cb = synth.f32_to_bf16_bits(cbv)
        idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
        for v in range(min(Q, 4)):
            idx[v] = v                                  # constant rows
            idx[8 + v] = v
            idx[8 + v, rng.integers(0, K)] = (v + 1) % Q   # one odd element in the row
        scales = synth.f32_to_bf16_bits(np.abs(rng.standard_normal((N, K // 64)) * 0.02).astype(np.float32))
        x = synth.f32_to_bf16_bits((rng.standard_normal((M, K)) * 2.0 ** rng.uniform(-12, 4, (M, K))).astype(np.float32))
        run_all(idx, scales, cb, x, bits, f"skewed {vals} b={bits}")


@pytest.mark.parametrize("bits,N,K", ((1, 8192, 8192), (4, 8192, 8192), (2, 16384, 3072), (1, 3072, 8192)))
def test_table_path_large_shapes_sampled_rows(bits, N, K):
    g = torch.Generator(device="cuda").manual_seed(bits + N)
    idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device="cuda", generator=g)
    wq = torch.empty(kmq.kmq_block_packed_bytes(N, K, bits), dtype=torch.uint8, device="cuda")
    kmq.kmq_block_pack(idx, N, K, bits, wq)
    scales = (torch.rand(N, K // 64, device="cuda", generator=g) * 0.05 + 0.01).to(torch.bfloat16)
    cb = torch.linspace(-1, 1, 1 << bits, device="cuda").to(torch.bfloat16)
    x = torch.randn(1, K, device="cuda", generator=g).to(torch.bfloat16)
    tab = torch.empty(kmq.kmq_block_table_bytes(N, K, bits), dtype=torch.uint8, device="cuda")
    kmq.kmq_block_table_pack(wq, scales, N, K, bits, tab)
    wsb = kmq.kmq_block_table_workspace_bytes(N, K, bits)
    ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
    y = torch.full((N,), float("nan"), dtype=torch.bfloat16, device="cuda")
    kmq.kmq_block_table_linear(tab, cb, x, y, N, K, bits, 1, ws, wsb)
    torch.cuda.synchronize()
    assert kmq.kmq_device_error_flags() == 0
    assert bool(torch.isfinite(y.float()).all())
    rows = np.unique(np.concatenate([np.arange(40), np.arange(N - 40, N), np.random.default_rng(0).integers(0, N, 64)]))
    sel = torch.from_numpy(rows).cuda()
    ref_wq = blk.pack_bytes(idx[sel].cpu().numpy(), bits)
    y_ref, s_abs = blk.block_linear_f64(ref_wq, scales[sel].view(torch.int16).cpu().numpy().view(np.uint16),
                                        cb.view(torch.int16).cpu().numpy().view(np.uint16),
                                        x.view(torch.int16).cpu().numpy().view(np.uint16), K, bits)
    got = y[sel].view(torch.int16).cpu().numpy().view(np.uint16).reshape(1, -1)
    assert orc.check_linear(got, y_ref, s_abs) <= 1.0
