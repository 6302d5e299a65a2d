"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Integer and lookup work (packing,
dequantised weights) must match bit for bit; layer outputs must satisfy
|y - y_ref| <= 2^-7 * sum_k |x_k * w_k| + 1e-6 elementwise."""
import numpy as np
import pytest
import torch

from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
BITS = (1, 2, 4)


def random_layer(rng, N, K, bits, M):
    Q = 1 << bits
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    cb = synth.f32_to_bf16_bits(np.sort(rng.standard_normal((N, Q)) * 0.02, axis=1).astype(np.float32))
    x = synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    return idx, cb, x


LAYOUTS = (kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TUNED, kmq.KMQ_LAYOUT_TABLE)


def check_all(idx, cb, x, bits, what=""):
    """Every packed layout.  The canonical words must equal the oracle's bit for bit; the tuned and the table layout
    are defined only through what they decode to (indices, weights), which must be exact; their bytes must also be
    the documented arrangement of the oracle's indices, padding zero."""
    N, K = idx.shape
    ref_packed = orc.pack_canonical(idx, bits)
    ref_w = orc.dequant_bits(ref_packed, cb, K, bits)
    y_ref, s = orc.linear_f64(ref_packed, cb, x, K, bits)
    worst = 0.0
    for layout in LAYOUTS:
        tag = f"{what} layout={layout}"
        packed = gu.gpu_pack(idx, bits, layout)
        if layout == kmq.KMQ_LAYOUT_CANONICAL:
            assert np.array_equal(gu.packed_to_numpy(packed, N), ref_packed), f"{tag}: packed words differ"
        else:
            assert np.array_equal(gu.gpu_unpack(packed, N, K, bits, layout), idx), f"{tag}: unpack(pack(idx)) != idx"
            if layout == kmq.KMQ_LAYOUT_TABLE and bits != 4:
                assert np.array_equal(packed.cpu().numpy().view(np.uint8),
                                      gu.table_from_indices(orc.unpack_canonical(ref_packed, K, bits), bits)), \
                    f"{tag}: bit planes differ from the documented layout"
            else:
                assert np.array_equal(packed.cpu().numpy().view(np.uint32), gu.tuned_from_canonical(ref_packed, bits)), \
                    f"{tag}: tuned words differ from the documented layout"
        w = gu.gpu_dequant(packed, cb, N, K, bits, layout)
        assert np.array_equal(w, ref_w), f"{tag}: dequantised weights differ"
        y = gu.gpu_linear(packed, cb, x, N, K, bits, layout)
        ratio = orc.check_linear(y, y_ref, s)
        assert ratio <= 1.0, (f"{tag}: error/tolerance = {ratio} "
                              f"[{kmq.kmq_linear_variant(N, K, bits, x.shape[0], layout)}]")
        worst = max(worst, ratio)
    return worst


# ---- configuration 1 (tiny correctness layer), all bit widths ----
@pytest.mark.parametrize("bits", BITS)
def test_config1_tiny_layer(bits):
    L = synth.make_layer(256, 256, bits, 1, "normal", config_id=1)
    check_all(L["idx"], L["codebooks"], L["x"], bits, f"config1 b={bits}")


# ---- pack / unpack ----
@pytest.mark.parametrize("bits", BITS)
def test_pack_unpack_round_trip_and_adversarial_patterns(bits):
    per, Q = 32 // bits, 1 << bits
    rng = np.random.default_rng(bits)
    K = per * 37
    pats = [rng.integers(0, 256, size=(19, K), dtype=np.uint8),          # high bits must be dropped
            np.zeros((3, K), np.uint8), np.full((3, K), Q - 1, np.uint8),
            (np.arange(3 * K).reshape(3, K) % 2 * (Q - 1)).astype(np.uint8)]
    one_hot = np.zeros((per, K), np.uint8)
    for p in range(per):
        one_hot[p, per * (p % 37) + p] = Q - 1                            # one field per word position
    pats.append(one_hot)
    for idx in pats:
        N = idx.shape[0]
        packed = gu.gpu_pack(idx, bits)
        assert np.array_equal(gu.packed_to_numpy(packed, N), orc.pack_canonical(idx, bits))
        out = torch.empty(N * K, dtype=torch.uint8, device="cuda")
        kmq.kmq_unpack(packed, N, K, bits, out)
        assert np.array_equal(out.cpu().numpy().reshape(N, K), idx % Q)


# ---- dequant special cases ----
@pytest.mark.parametrize("bits", BITS)
def test_dequant_identity_codebook_reveals_indices_and_keeps_negative_zero(bits):
    Q = 1 << bits
    rng = np.random.default_rng(20 + bits)
    N, K = 37, (32 // bits) * 9
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    ident = synth.f32_to_bf16_bits(np.tile(np.arange(Q, dtype=np.float32), (N, 1)))
    packed = gu.gpu_pack(idx, bits)
    w = gu.gpu_dequant(packed, ident, N, K, bits)
    assert np.array_equal(synth.bf16_bits_to_f32(w).astype(np.uint8), idx)
    odd = np.tile(np.array([0x8000, 0x0000, 0x0001, 0x7F7F] * (Q // 4 + 1), np.uint16)[:Q], (N, 1))
    w2 = gu.gpu_dequant(packed, odd, N, K, bits)
    assert np.array_equal(w2, orc.dequant_bits(orc.pack_canonical(idx, bits), odd, K, bits))


# ---- ragged and small shapes, every batch size of interest ----
@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("N,Kmul,M", [
    (1, 1, 1), (3, 1, 2), (17, 3, 3), (130, 5, 5), (259, 16, 7), (64, 64, 8), (100, 33, 9),
    (257, 40, 15), (48, 128, 16), (61, 24, 17), (33, 12, 31), (40, 10, 33), (16, 8, 63), (129, 20, 64),
    (70, 4, 65), (1000, 96, 1), (2051, 32, 2),
])
def test_linear_ragged_shapes(bits, N, Kmul, M):
    K = (32 // bits) * Kmul
    rng = np.random.default_rng(1000 * bits + N + M)
    idx, cb, x = random_layer(rng, N, K, bits, M)
    check_all(idx, cb, x, bits, f"N={N} K={K} M={M} b={bits}")


# ---- invariants on the GPU path too ----
def test_one_bit_sign_codebook_on_gpu():
    rng = np.random.default_rng(5)
    N, K, M = 300, 1024, 3
    idx = rng.integers(0, 2, size=(N, K), dtype=np.uint8)
    a = synth.f32_to_bf16_bits((rng.integers(128, 256, size=N) * 2.0 ** -13).astype(np.float32))
    cb = np.stack([a | np.uint16(0x8000), a], axis=1)
    x = synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    packed = gu.gpu_pack(idx, 1)
    y = synth.bf16_bits_to_f32(gu.gpu_linear(packed, cb, x, N, K, 1)).astype(np.float64)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    expect = (xf @ (2.0 * idx - 1.0).T) * synth.bf16_bits_to_f32(a).astype(np.float64)[None, :]
    bound = 2.0 ** -7 * (np.abs(xf).sum(axis=1)[:, None] * synth.bf16_bits_to_f32(a)[None, :]) + 1e-6
    assert np.all(np.abs(y - expect) <= bound)


def test_repeated_calls_are_bit_identical():
    rng = np.random.default_rng(9)
    N, K, M, bits = 512, 2048, 4, 2
    idx, cb, x = random_layer(rng, N, K, bits, M)
    packed = gu.gpu_pack(idx, bits)
    y1 = gu.gpu_linear(packed, cb, x, N, K, bits)
    y2 = gu.gpu_linear(packed, cb, x, N, K, bits)
    assert np.array_equal(y1, y2)


def test_host_entry_point_matches_device_entry_point():
    rng = np.random.default_rng(10)
    N, K, M, bits = 384, 1024, 3, 4
    idx, cb, x = random_layer(rng, N, K, bits, M)
    packed = gu.gpu_pack(idx, bits)
    y_dev = gu.gpu_linear(packed, cb, x, N, K, bits)
    xh = torch.from_numpy(x.view(np.int16)).pin_memory()
    yh = torch.empty(M * N, dtype=torch.int16).pin_memory()
    xs = torch.empty(M * K, dtype=torch.int16, device="cuda")
    ys = torch.empty(M * N, dtype=torch.int16, device="cuda")
    ws_bytes = kmq.kmq_workspace_bytes(N, K, bits, M)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    kmq.kmq_linear_host(packed, gu.to_dev_u16(cb), xh.data_ptr(), yh.data_ptr(), N, K, bits, M, xs, ys, ws, ws_bytes)
    assert np.array_equal(yh.numpy().view(np.uint16).reshape(M, N), y_dev)


def test_workspace_is_checked_on_the_host():
    N, K, bits, M, T = 8192, 16384, 4, 1, kmq.KMQ_LAYOUT_TUNED
    need = kmq.kmq_workspace_bytes(N, K, bits, M, T)
    if need == 0:
        pytest.skip("this shape needs no workspace on this device")
    a = torch.zeros(16, dtype=torch.uint8, device="cuda")
    big = torch.zeros(N * K // 4, dtype=torch.uint8, device="cuda")
    st = kmq.kmq_linear(big, big, big, big, N, K, bits, M, a, need - 1, layout=T, check=False)
    assert st == kmq.KMQ_ERR_WORKSPACE
    st = kmq.kmq_linear(big, big, big, big, N, K, bits, M, None, 0, layout=T, check=False)
    assert st == kmq.KMQ_ERR_WORKSPACE


# ---- more tiles than resident CTAs: equal step ranges per CTA, partial tiles added by the fix-up kernel ----
@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("Kmul,M", [(512, 1), (517, 3)])
def test_linear_balanced_split_variant(bits, Kmul, M):
    N, K = 16 * 460 + 5, (128 // bits) * Kmul          # 461 tiles (the last one ragged), Kmul 16-byte chunks per row
    if bits == 1:
        M = 1                                          # b = 1 goes to the multi-tile kernel from 2 batch rows on here
    rng = np.random.default_rng(7000 + 10 * bits + Kmul)
    idx, cb, x = random_layer(rng, N, K, bits, M)
    T = kmq.KMQ_LAYOUT_TUNED
    if kmq.kmq_workspace_bytes(N, K, bits, M, T) == 0:
        pytest.skip("the balanced variant is not selected on this device")
    assert kmq.kmq_linear_num_launches(N, K, bits, M, T) == 2
    ref_packed = orc.pack_canonical(idx, bits)
    y_ref, s = orc.linear_f64(ref_packed, cb, x, K, bits)
    packed = gu.gpu_pack(idx, bits, T)
    y1 = gu.gpu_linear(packed, cb, x, N, K, bits, T)
    ratio = orc.check_linear(y1, y_ref, s)
    assert ratio <= 1.0, f"error/tolerance = {ratio} [{kmq.kmq_linear_variant(N, K, bits, M, T)}]"
    assert np.array_equal(y1, gu.gpu_linear(packed, cb, x, N, K, bits, T)), "repeated call differs"
