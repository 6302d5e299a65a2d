"""GPU parity of kmq_linear_tcgen05 (tensor-memory kernel, tuned layout) against the CPU oracle: same tolerance as
kmq_linear, |y - y_ref| <= 2^-7 * sum_k |x_k * w_k| + 1e-6; every wait inside the kernel is bounded, so the device
error word must stay 0; outputs outside [0, M) x [0, N) must not be touched."""
import numpy as np
import pytest
import torch

from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
T = kmq.KMQ_LAYOUT_TUNED


def random_layer(rng, N, K, bits, M):
    Q = 1 << bits
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    cb = synth.f32_to_bf16_bits(np.sort(rng.standard_normal((N, Q)) * 0.02, axis=1).astype(np.float32))
    x = synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    return idx, cb, x


def run(idx, cb, x, bits):
    N, K = idx.shape
    M = x.shape[0]
    packed = gu.gpu_pack(idx, bits, T)
    nbytes = M * N * 2
    buf, off = gu.dev_bytes(nbytes)
    kmq.kmq_linear_tcgen05(packed, gu.to_dev_u16(cb), gu.to_dev_u16(x), buf.data_ptr() + off, N, K, bits, M)
    assert kmq.kmq_device_error_flags() == 0, "a bounded wait inside the kernel ran out"
    assert gu.canaries_intact(buf, off, nbytes), "the kernel wrote outside y"
    return buf[off:off + nbytes].cpu().numpy().view(np.uint16).reshape(M, N)


# ragged row counts (not a multiple of 16 or 128), K that is not a whole number of stages, every width of the MMA's N
@pytest.mark.parametrize("bits", (1, 2, 4))
@pytest.mark.parametrize("N,Kmul,M", [(128, 4, 16), (200, 9, 48), (333, 5, 64), (77, 12, 17), (1000, 32, 33),
                                      (129, 2, 31), (16, 1, 1), (48, 1, 64), (520, 16, 130), (2048, 64, 20), (300, 8, 90),
                                      (1100, 32, 128),
                                      (520, 128, 64), (300, 131, 33)])   # >= 32 steps of K: cluster of 4 CTAs
def test_tcgen05_linear_matches_oracle(bits, N, Kmul, M):
    K = (128 // bits) * Kmul          # Kmul 16-byte chunks per row
    rng = np.random.default_rng(9000 + 100 * bits + N + M)
    idx, cb, x = random_layer(rng, N, K, bits, M)
    y_ref, s = orc.linear_f64(orc.pack_canonical(idx, bits), cb, x, K, bits)
    y = run(idx, cb, x, bits)
    ratio = orc.check_linear(y, y_ref, s)
    assert ratio <= 1.0, f"error/tolerance = {ratio}"


def test_tcgen05_matches_kmq_linear_on_a_k_means_layer():
    L = synth.make_layer(512, 2048, 2, 24, "normal", config_id=4)
    y = run(L["idx"], L["codebooks"], L["x"], 2)
    y_ref, s = orc.linear_f64(orc.pack_canonical(L["idx"], 2), L["codebooks"], L["x"], 2048, 2)
    assert orc.check_linear(y, y_ref, s) <= 1.0
    packed = gu.gpu_pack(L["idx"], 2, T)
    y2 = gu.gpu_linear(packed, L["codebooks"], L["x"], 512, 2048, 2, T)
    assert orc.check_linear(y2, y_ref, s) <= 1.0


def test_tcgen05_argument_errors():
    a = torch.zeros(4096, dtype=torch.int32, device="cuda")
    assert kmq.kmq_linear_tcgen05(0, a, a, a, 128, 256, 2, 16, check=False) == kmq.KMQ_ERR_NULL
    assert kmq.kmq_linear_tcgen05(a, a, a, a, 128, 256, 3, 16, check=False) == kmq.KMQ_ERR_BITS
    assert kmq.kmq_linear_tcgen05(a, a, a, a, 128, 16, 2, 16, check=False) == kmq.KMQ_ERR_SHAPE   # K * bits % 128 != 0
    assert kmq.kmq_linear_tcgen05(a.data_ptr() + 4, a, a, a, 128, 256, 2, 16, check=False) == kmq.KMQ_ERR_ALIGN
