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


@pytest.mark.parametrize("M", (1, 2))
@pytest.mark.parametrize("N,K", ((16, 512), (50, 1024), (700, 2048), (4096 + 7, 4096), (130, 6144 + 256), (9216, 3072)))
@pytest.mark.parametrize("bits", (1, 2))
def test_table_kernel_with_the_slices_of_a_row_block_as_one_cluster(bits, N, K, M):
    """Shapes whose K range splits into 2, 4 or 8 slices: the table kernel then adds the slices inside a thread-block
    cluster (one launch, no scratch).  Ragged row counts, more row blocks than one, skewed codebooks on the first
    rows; the output must not depend on which of the two forms ran."""
    if kmq.kmq_workspace_bytes(N, K, bits, M, L) != 0 or kmq.kmq_linear_num_launches(N, K, bits, M, L) != M:
        pytest.skip("the planner adds the slices with a second kernel for this shape on this device")
    rng = np.random.default_rng(bits * 100 + N + K + M)
    Q = 1 << bits
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    cbv = np.sort(rng.standard_normal((N, Q)) * 0.02, axis=1)
    sk = skewed_codebooks(bits)
    for i, c in enumerate(sk[:min(N, len(sk))]):
        cbv[i] = c
        idx[i] = i % Q
    cb = bf16(cbv)
    x = bf16(rng.standard_normal((M, K)) * 2.0 ** rng.uniform(-8, 3, size=(M, K)))
    assert check(idx, cb, x, bits, L).startswith("table_lookup")
