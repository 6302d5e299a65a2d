"""kmq_linear_static_scratch, the entry point for callers that may not allocate device memory (its scratch is a fixed
array inside the library): on a shape that really uses scratch it must give what kmq_linear gives with a
caller-provided workspace, on two calls in a row that share the array.  The file name sorts last on purpose: with
`pytest -x` a failure here cannot keep any other test from running."""
import numpy as np
import pytest
import torch

from paper_2602_15563_b200 import kmq

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_entry_point_twice():
    N, K, bits, M, T = 8192, 16384, 4, 3, kmq.KMQ_LAYOUT_TUNED
    need = kmq.kmq_workspace_bytes(N, K, bits, M, T)
    if need == 0:
        pytest.skip("no kernel of kmq_linear uses scratch for this shape on this device")
    assert need <= kmq.kmq_static_scratch_capacity()
    g = torch.Generator(device="cuda").manual_seed(1234)
    words = kmq.kmq_packed_bytes(N, K, bits, T) // 4
    packed = torch.randint(-2**31, 2**31 - 1, (words,), dtype=torch.int32, device="cuda", generator=g)
    cb = (torch.randn(N, 1 << bits, device="cuda", generator=g) * 0.02).sort(dim=1).values.to(torch.bfloat16)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    for call in range(2):                                   # second call: other activations, same shared array
        x = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
        y_ref = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        y = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        kmq.kmq_linear(packed, cb, x, y_ref, N, K, bits, M, ws, need, layout=T)
        kmq.kmq_linear_static_scratch(packed, cb, x, y, N, K, bits, M, layout=T)
        torch.cuda.synchronize()
        a, b = y.float().cpu().numpy(), y_ref.float().cpu().numpy()
        assert np.all(np.isfinite(b)) and np.abs(b).max() > 0
        # same kernels, same order of additions: the tolerance of the parity tests (2^-7 of the sum of magnitudes,
        # here bounded from below by |y_ref|) is met with room to spare; in fact the results are identical
        assert np.all(np.abs(a - b) <= 2.0 ** -7 * np.abs(b) + 1e-6), f"call {call}: outputs differ"
        assert np.array_equal(a, b), f"call {call}: outputs are not bit-identical"


def test_static_scratch_passes_through_shapes_without_scratch_and_bad_arguments():
    N, K, bits, M = 64, 256, 2, 2
    assert kmq.kmq_workspace_bytes(N, K, bits, M) == 0
    g = torch.Generator(device="cuda").manual_seed(5)
    packed = torch.randint(-2**31, 2**31 - 1, (kmq.kmq_packed_bytes(N, K, bits) // 4,), dtype=torch.int32,
                           device="cuda", generator=g)
    cb = (torch.randn(N, 1 << bits, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    x = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    y1 = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    y2 = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    kmq.kmq_linear(packed, cb, x, y1, N, K, bits, M)
    kmq.kmq_linear_static_scratch(packed, cb, x, y2, N, K, bits, M)
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    assert kmq.kmq_linear_static_scratch(packed, cb, x, y2, N, K, 3, M, check=False) == kmq.KMQ_ERR_BITS
    assert kmq.kmq_linear_static_scratch(0, cb, x, y2, N, K, bits, M, check=False) == kmq.KMQ_ERR_NULL
