"""GPU parity on inputs chosen to break an evaluation that is not the definition: skewed codebooks (one centroid
zero, tiny, or hundreds of times the other; equal centroids), index rows that use one centroid everywhere or almost
everywhere, activations spanning many orders of magnitude.  The stated tolerance |y - y_ref| <= 2^-7 * sum_k |x_k *
w_k| + 1e-6 is relative to the terms a row really has, so any rewrite of the sum that cancels large terms against
each other (a sign decomposition, a sum over all activations minus a part) fails here unless it is done with care.
Every kernel variant the dispatcher can pick for b = 1 and b = 2 is reached."""
import numpy as np
import pytest

from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
C, T, L = kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TUNED, kmq.KMQ_LAYOUT_TABLE


def bf16(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def skewed_codebooks(bits):
    """One codebook per row pattern; every value is exactly representable in bf16."""
    if bits == 1:
        return [(0.0, 1.0), (1.0, 0.0), (2.0 ** -10, 1.0), (-1.0, 300.0), (300.0, -1.0), (0.75, 0.75),
                (-0.0, 2.0 ** -20), (1.0, -1.0)]
    return [(0.0, 0.0, 0.0, 1.0), (1.0, 0.0, 0.0, 0.0), (-300.0, 2.0 ** -10, 0.0, 1.0), (0.5, 0.5, 0.5, 0.5),
            (0.0, 1.0, -1.0, 0.0), (2.0 ** -12, -2.0 ** -12, 256.0, -0.0), (-1.0, -0.5, 0.5, 1.0),
            (7.0, 2.0 ** -9, -7.0, 2.0 ** -9)]


def index_rows(rng, K, Q):
    """Index patterns: constant rows, one odd element in 4096, one odd element in the row, uniform."""
    rows = []
    for v in range(Q):
        rows.append(np.full(K, v, np.uint8))
        r = np.full(K, v, np.uint8)
        r[rng.integers(0, 4096) % K::4096] = (v + 1) % Q
        rows.append(r)
        r = np.full(K, v, np.uint8)
        r[rng.integers(0, K)] = (v + Q - 1) % Q
        rows.append(r)
    rows.append(rng.integers(0, Q, K).astype(np.uint8))
    return rows


def adversarial_layer(bits, K, M, seed):
    rng = np.random.default_rng(seed)
    Q = 1 << bits
    cbs = skewed_codebooks(bits)
    pats = index_rows(rng, K, Q)
    idx = np.stack([p for _ in cbs for p in pats])
    cb = bf16(np.stack([np.array(c) for c in cbs for _ in pats]))
    # activations: N(0,1) scaled by 2^u, u uniform in [-12, 4] -> small and large values side by side
    x = bf16(rng.standard_normal((M, K)) * 2.0 ** rng.uniform(-12, 4, size=(M, K)))
    return idx, cb, x


def check(idx, cb, x, bits, layout):
    N, K = idx.shape
    M = x.shape[0]
    ref_packed = orc.pack_canonical(idx, bits)
    y_ref, s = orc.linear_f64(ref_packed, cb, x, K, bits)
    packed = gu.gpu_pack(idx, bits, layout)
    y = gu.gpu_linear(packed, cb, x, N, K, bits, layout)
    ratio = orc.check_linear(y, y_ref, s)
    variant = kmq.kmq_linear_variant(N, K, bits, M, layout)
    assert ratio <= 1.0, f"b={bits} K={K} M={M} layout={layout} [{variant}]: error/tolerance = {ratio}"
    return variant


@pytest.mark.parametrize("layout", (C, T, L))
@pytest.mark.parametrize("M", (1, 3, 8, 16))
@pytest.mark.parametrize("K", (4096, 28672))
@pytest.mark.parametrize("bits", (1, 2))
def test_skewed_codebooks_and_degenerate_rows(bits, K, M, layout):
    if layout == L and M > 3:
        pytest.skip("the table kernel runs one pass per batch row: M = 1 and 3 cover it")
    idx, cb, x = adversarial_layer(bits, K, M, 100 * bits + M + K)
    check(idx, cb, x, bits, layout)


@pytest.mark.parametrize("bits", (1, 2))
def test_skewed_codebooks_on_the_balanced_split_variant(bits):
    """More 16-row tiles than resident CTAs and long rows: the balanced kernel pair of the tuned layout."""
    K, M = (128 // bits) * 512, 1
    idx, cb, x = adversarial_layer(bits, K, M, 7 + bits)
    reps = -(-(16 * 460 + 5) // idx.shape[0])
    idx, cb = np.tile(idx, (reps, 1))[:16 * 460 + 5], np.tile(cb, (reps, 1))[:16 * 460 + 5]
    if kmq.kmq_workspace_bytes(idx.shape[0], K, bits, M, T) == 0:
        pytest.skip("the balanced variant is not selected on this device")
    assert check(idx, cb, x, bits, T).startswith("split")


def test_every_b1_b2_variant_was_reached():
    names = set()
    for bits in (1, 2):
        for K in (4096, 28672):
            for M in (1, 3, 8, 16):
                for layout in (C, T, L):
                    names.add(kmq.kmq_linear_variant(64, K, bits, M, layout))
    for want in ("tiled_", "multi_", "staged_", "table_lookup_"):
        assert any(n.startswith(want) for n in names), f"no case reaches a {want}* kernel: {sorted(names)}"
