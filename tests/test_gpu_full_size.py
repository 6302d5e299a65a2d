"""GPU parity at the full sizes of the benchmark configurations, in the launch configurations bench.py times
(tuned and table layouts, packed by kmq_pack; the canonical layout as well).  The oracle is evaluated on every
output row of the layers it finishes in seconds (configurations 2 and 3) and on a sample of rows (first tile, last
tile and random rows) of the larger ones, each row computed on its own: canonical packed words and dequantised
weights must match bit for bit, outputs within |y - y_ref| <= 2^-7 * sum_k |x_k * w_k| + 1e-6."""
import functools

import numpy as np
import pytest
import torch

from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
T, C, L = kmq.KMQ_LAYOUT_TUNED, kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TABLE
ALL_ROWS_MAX_WEIGHTS = 1 << 26          # the float64 oracle takes a second or two on a layer of this size


@functools.lru_cache(maxsize=2)
def layer(config_id, name, bits):
    (N, K, dist), = [(n_, k_, d_) for (nm, n_, k_, d_) in synth.CONFIG_LAYERS[config_id] if nm == name]
    L = synth.make_layer(N, K, bits, 1, dist, config_id=config_id)
    return L["idx"], L["codebooks"]


def sample_rows(N, K, seed):
    if N * K <= ALL_ROWS_MAX_WEIGHTS:
        return np.arange(N)
    rng = np.random.default_rng(seed)
    rows = np.concatenate([np.arange(16), np.arange(N - 16, N), rng.choice(N, size=32, replace=False)])
    return np.unique(rows)


def run_case(config_id, name, bits, M, check_dequant):
    idx, cb = layer(config_id, name, bits)
    N, K = idx.shape
    x = synth.draw_activations(M, K, synth.rng_for(config_id, 1000 + M))
    rows = sample_rows(N, K, 17 * config_id + bits + M)
    layouts = (T, C, L) if (bits != 4 and M <= 2) else (T, C)       # the table kernel runs one pass per batch row
    ref_packed = orc.pack_canonical(idx[rows], bits)                       # the sampled rows only
    y_ref, s = orc.linear_f64(ref_packed, cb[rows], x, K, bits)

    d_idx = torch.from_numpy(idx).cuda()
    packed = {}
    for layout in layouts:
        p = torch.empty(kmq.kmq_packed_bytes(N, K, bits, layout) // 4, dtype=torch.int32, device="cuda")
        kmq.kmq_pack(d_idx, N, K, bits, p, layout=layout)
        packed[layout] = p
    del d_idx
    got = packed[C].view(N, -1)[torch.from_numpy(rows).cuda()].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, ref_packed), "canonical packed words differ on the sampled rows"

    d_cb, d_x = gu.to_dev_u16(cb), gu.to_dev_u16(x)
    for layout in layouts:
        y = torch.full((M * N,), 0x7FC0, dtype=torch.int16, device="cuda")
        ws_bytes = kmq.kmq_workspace_bytes(N, K, bits, M, layout)
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
        kmq.kmq_linear(packed[layout], d_cb, d_x, y, N, K, bits, M, ws, ws_bytes, layout=layout)
        yh = y.cpu().numpy().view(np.uint16).reshape(M, N)
        assert np.all(np.isfinite(synth.bf16_bits_to_f32(yh))), f"layout {layout}: some outputs were not written"
        ratio = orc.check_linear(yh[:, rows], y_ref, s)
        assert ratio <= 1.0, (f"layout {layout}: error/tolerance = {ratio} "
                              f"[{kmq.kmq_linear_variant(N, K, bits, M, layout)}]")
    if check_dequant:
        ref_w = orc.dequant_bits(ref_packed, cb[rows], K, bits)
        for layout in layouts:
            W = torch.empty(N * K, dtype=torch.int16, device="cuda")
            kmq.kmq_dequant_to_bf16(packed[layout], d_cb, W, N, K, bits, layout=layout)
            got_w = W.view(N, K)[torch.from_numpy(rows).cuda()].cpu().numpy().view(np.uint16)
            assert np.array_equal(got_w, ref_w), f"layout {layout}: dequantised weights differ on the sampled rows"
            del W
    torch.cuda.empty_cache()


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_config2_square_4096(bits):
    run_case(2, "square4096", bits, 1, check_dequant=True)


@pytest.mark.parametrize("M", (1, 8))
@pytest.mark.parametrize("name", ("qkv", "o", "gate_up", "down"))
def test_config3_decoder_linear_set(name, M):
    run_case(3, name, 2, M, check_dequant=(M == 1))


def test_large_batch_on_many_rows_goes_through_tcgen05():
    """16384 rows are 128 blocks of 128: from 33 batch rows on kmq_linear picks the tensor-memory kernel there."""
    assert kmq.kmq_linear_variant(16384, 3072, 2, 64, T).startswith("tcgen05")
    assert kmq.kmq_linear_num_launches(16384, 3072, 2, 64, T) == 1
    assert kmq.kmq_workspace_bytes(16384, 3072, 2, 64, T) == 0
    run_case(3, "gate_up", 2, 64, check_dequant=False)
    assert kmq.kmq_device_error_flags() == 0


def test_no_kernel_reported_an_error():
    """Collected after the full-size cases above: no bounded wait ran out, no shared-memory window was misplaced."""
    assert kmq.kmq_device_error_flags() == 0


@pytest.mark.parametrize("M", (1, 2, 4, 8, 16, 32, 64))
def test_config4_batch_sweep_8192(M):
    run_case(4, "square8192", 2, M, check_dequant=(M == 1))


@pytest.mark.parametrize("M", (1, 5, 16))
@pytest.mark.parametrize("bits", (1, 4))
def test_config5_large_down_projection(bits, M):
    run_case(5, "down_large", bits, M, check_dequant=(M == 1))
