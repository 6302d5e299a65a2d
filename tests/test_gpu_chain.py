"""Calls chained on one stream without any synchronisation in between, every call reading the previous call's output:
the kernels start before their predecessors have finished (programmatic dependent launch, early release of the next
kernel) and must still see finished inputs.  The chain mixes every kernel variant of kmq_linear; its results must be
bit-identical to the same chain run with a device synchronisation after every call, and the first link is checked
against the oracle."""
import numpy as np
import pytest
import torch

from oracle import kmq_oracle as orc
from paper_2602_15563_b200 import kmq

pytestmark = pytest.mark.gpu
C, T, L = kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TUNED, kmq.KMQ_LAYOUT_TABLE


def build_chain(widths, bits_layouts, M, seed):
    """Layers widths[i] -> widths[i + 1] with random indices and small codebooks (so that activations stay finite)."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    layers = []
    for i, (bits, layout) in enumerate(bits_layouts):
        K, N = widths[i], widths[i + 1]
        idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device="cuda", generator=g)
        packed = torch.empty(kmq.kmq_packed_bytes(N, K, bits, layout) // 4, dtype=torch.int32, device="cuda")
        kmq.kmq_pack(idx, N, K, bits, packed, layout=layout)
        cb = (torch.randn(N, 1 << bits, device="cuda", generator=g) * (2.0 / K ** 0.5)).sort(dim=1).values
        cb = cb.to(torch.bfloat16).view(torch.int16)
        wsb = kmq.kmq_workspace_bytes(N, K, bits, M, layout)
        layers.append({"N": N, "K": K, "bits": bits, "layout": layout, "packed": packed, "cb": cb, "idx": idx,
                       "ws_bytes": wsb, "variant": kmq.kmq_linear_variant(N, K, bits, M, layout)})
    return layers


def run_chain(layers, x0, M, sync):
    ws = torch.empty(max([l["ws_bytes"] for l in layers] + [16]), dtype=torch.uint8, device="cuda")
    outs, x = [], x0
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for l in layers:
            y = torch.full((M * l["N"],), 0x7FC0, dtype=torch.int16, device="cuda")     # NaN patterns
            outs.append(y)
        stream.synchronize()
        for l, y in zip(layers, outs):
            kmq.kmq_linear(l["packed"], l["cb"], x, y, l["N"], l["K"], l["bits"], M, ws, l["ws_bytes"], layout=l["layout"])
            if sync:
                stream.synchronize()
            x = y
        stream.synchronize()
    return [o.clone() for o in outs]


@pytest.mark.parametrize("M", (1, 3, 16, 40))
def test_chained_calls_see_finished_inputs(M):
    widths = [4096, 3072, 8192, 4096, 2048, 6144, 4096, 3072, 4096]
    bl = [(2, T), (4, T), (1, T), (1, L), (2, L), (4, T), (2, C), (1, T)]
    layers = build_chain(widths, bl, M, seed=M)
    g = torch.Generator(device="cuda").manual_seed(99)
    x0 = torch.randn(M * widths[0], device="cuda", generator=g).to(torch.bfloat16).view(torch.int16)
    ref = run_chain(layers, x0, M, sync=True)
    for rep in range(3):
        got = run_chain(layers, x0, M, sync=False)
        for i, (a, b) in enumerate(zip(got, ref)):
            assert torch.equal(a, b), f"M={M} rep={rep}: link {i} [{layers[i]['variant']}] differs from the synchronised chain"
    assert kmq.kmq_device_error_flags() == 0
    # the first link against the oracle, the last against finiteness (every link consumed a finished input)
    l = layers[0]
    rows = np.arange(0, l["N"], 61)
    ref_packed = orc.pack_canonical(l["idx"][torch.from_numpy(rows).cuda()].cpu().numpy(), l["bits"])
    y_ref, s = orc.linear_f64(ref_packed, l["cb"].cpu().numpy().view(np.uint16)[rows],
                              x0.cpu().numpy().view(np.uint16).reshape(M, -1), l["K"], l["bits"])
    y0 = ref[0].cpu().numpy().view(np.uint16).reshape(M, -1)[:, rows]
    assert orc.check_linear(y0, y_ref, s) <= 1.0
    assert bool(torch.isfinite(ref[-1].view(torch.bfloat16).float()).all())
    assert len({l["variant"].split("_")[0] for l in layers}) >= 3 or M > 8


def test_large_layers_chained_with_the_table_and_split_kernels():
    """8192 x 28672 at b = 1 (table kernel + the kernel that adds its slices) and b = 4 (balanced split + fix-up)
    feeding a 4096-wide layer and each other."""
    M = 1
    widths = [28672, 8192, 28672, 8192, 4096]
    bl = [(1, L), (4, T), (4, T), (2, T)]
    layers = build_chain(widths, bl, M, seed=5)
    g = torch.Generator(device="cuda").manual_seed(7)
    x0 = torch.randn(M * widths[0], device="cuda", generator=g).to(torch.bfloat16).view(torch.int16)
    ref = run_chain(layers, x0, M, sync=True)
    for rep in range(2):
        got = run_chain(layers, x0, M, sync=False)
        for i, (a, b) in enumerate(zip(got, ref)):
            assert torch.equal(a, b), f"rep={rep}: link {i} [{layers[i]['variant']}] differs from the synchronised chain"
    assert kmq.kmq_device_error_flags() == 0
