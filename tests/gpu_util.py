"""Helpers shared by the GPU parity tests: move a synthetic layer to the device,
run the library through its C ABI, bring the results back as NumPy arrays."""
import numpy as np
import torch

from paper_2602_15563_b200 import kmq

CANARY = 0x5A


def dev_bytes(nbytes: int, pad: int = 256):
    """A device buffer of `nbytes` with canary bands on both sides.
    Returns (whole uint8 tensor, offset of the payload)."""
    total = nbytes + 2 * pad
    buf = torch.full((total,), CANARY, dtype=torch.uint8, device="cuda")
    return buf, pad


def canaries_intact(buf: torch.Tensor, off: int, nbytes: int) -> bool:
    head = buf[:off]
    tail = buf[off + nbytes:]
    return bool((head == CANARY).all().item() and (tail == CANARY).all().item())


def to_dev_u16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def gpu_pack(idx: np.ndarray, bits: int, layout: int = kmq.KMQ_LAYOUT_CANONICAL) -> torch.Tensor:
    """Pack on the GPU into a buffer with canary bands; returns the payload view."""
    N, K = idx.shape
    d_idx = torch.from_numpy(np.ascontiguousarray(idx)).cuda()
    nbytes = kmq.kmq_packed_bytes(N, K, bits, layout)
    buf, off = dev_bytes(nbytes)
    assert (buf.data_ptr() + off) % 16 == 0
    kmq.kmq_pack(d_idx, N, K, bits, buf.data_ptr() + off, layout=layout)
    torch.cuda.synchronize()
    assert canaries_intact(buf, off, nbytes), "pack wrote outside its buffer"
    return buf[off:off + nbytes].view(torch.int32)


def gpu_unpack(packed: torch.Tensor, N: int, K: int, bits: int, layout: int = kmq.KMQ_LAYOUT_CANONICAL) -> np.ndarray:
    nbytes = N * K
    buf, off = dev_bytes(nbytes)
    kmq.kmq_unpack(packed, N, K, bits, buf.data_ptr() + off, layout=layout)
    torch.cuda.synchronize()
    assert canaries_intact(buf, off, nbytes), "unpack wrote outside idx"
    return buf[off:off + nbytes].cpu().numpy().reshape(N, K)


def packed_to_numpy(packed: torch.Tensor, N: int) -> np.ndarray:
    return packed.cpu().numpy().view(np.uint32).reshape(N, -1)


def gpu_dequant(packed: torch.Tensor, cb: np.ndarray, N: int, K: int, bits: int,
                layout: int = kmq.KMQ_LAYOUT_CANONICAL) -> np.ndarray:
    d_cb = to_dev_u16(cb)
    nbytes = N * K * 2
    buf, off = dev_bytes(nbytes)
    kmq.kmq_dequant_to_bf16(packed, d_cb, buf.data_ptr() + off, N, K, bits, layout=layout)
    torch.cuda.synchronize()
    assert canaries_intact(buf, off, nbytes), "dequant wrote outside W"
    return buf[off:off + nbytes].cpu().numpy().view(np.uint16).reshape(N, K)


def gpu_linear(packed: torch.Tensor, cb: np.ndarray, x: np.ndarray, N: int, K: int, bits: int,
               layout: int = kmq.KMQ_LAYOUT_CANONICAL) -> np.ndarray:
    M = x.shape[0]
    d_cb, d_x = to_dev_u16(cb), to_dev_u16(x)
    nbytes = M * N * 2
    buf, off = dev_bytes(nbytes)
    ws_bytes = kmq.kmq_workspace_bytes(N, K, bits, M, layout)
    wsbuf, wsoff = dev_bytes(max(ws_bytes, 16))
    kmq.kmq_linear(packed, d_cb, d_x, buf.data_ptr() + off, N, K, bits, M,
                   wsbuf.data_ptr() + wsoff, ws_bytes, layout=layout)
    torch.cuda.synchronize()
    assert canaries_intact(buf, off, nbytes), "linear wrote outside y"
    assert canaries_intact(wsbuf, wsoff, max(ws_bytes, 16)), "linear wrote outside its workspace"
    return buf[off:off + nbytes].cpu().numpy().view(np.uint16).reshape(M, N)


def tuned_from_canonical(words: np.ndarray, bits: int) -> np.ndarray:
    """The documented tuned layout (include/kmq.h) applied to canonical words [N, wpr]: flat uint32 array of
    kmq_packed_bytes(..., TUNED) / 4 words, padding zero.  Written from the header's formulas, not from the library."""
    N, wpr = words.shape
    per = 32 // bits
    if bits == 4:
        shifts = [4 * i for i in range(per)]
    elif bits == 2:
        shifts = [2 * (i // 4) + 8 * (i % 4) for i in range(per)]
    else:
        shifts = [(31 - i // 2) if i % 2 else (15 - i // 2) for i in range(per)]
    mask = np.uint32((1 << bits) - 1)
    perm = np.zeros_like(words)
    for i in range(per):
        perm |= ((words >> np.uint32(i * bits)) & mask) << np.uint32(shifts[i])
    steps = -(-wpr // 16)
    out = np.zeros(-(-N // 16) * steps * 256, dtype=np.uint32)
    n = np.arange(N)[:, None]
    j = np.arange(wpr)[None, :]
    out[(((n // 16) * steps + j // 16) * 16 + n % 16) * 16 + j % 16] = perm
    return out


def table_from_indices(idx: np.ndarray, bits: int) -> np.ndarray:
    """The documented bit-plane layout KMQ_LAYOUT_TABLE (include/kmq.h) applied to indices [N, K] (bits = 1, 2):
    uint8 array of kmq_packed_bytes(..., TABLE) bytes, padding zero.  Written from the header's formulas."""
    N, K = idx.shape
    assert bits in (1, 2) and K % 8 == 0
    chunks, tiles = -(-K // 256), -(-N // 16)
    out = np.zeros(tiles * chunks * bits * 512, dtype=np.uint8)
    n = np.arange(N)[:, None]
    g = np.arange(K // 8)[None, :]
    weights = (1 << np.arange(8)).astype(np.uint16)
    for p in range(bits):
        plane = ((idx.reshape(N, K // 8, 8) >> p) & 1).astype(np.uint16)
        byte = (plane * weights).sum(axis=2).astype(np.uint8)                 # weight 8g + t in bit t
        off = ((n // 16 * chunks + g // 32) * bits + p) * 512 + (2 * (n % 16) + g % 2) * 16 + ((g % 32) // 2 - n % 16) % 16
        out[off] = byte
    return out


def block_table_from_bytes(wq: np.ndarray, scales: np.ndarray, K: int, bits: int) -> np.ndarray:
    """The block-format table layout restated from the formulas of include/kmq.h: uint8 [total bytes].
    wq uint8 [N, K*bits/8] (layout of kmq_block_pack), scales uint16 [N, K/64]."""
    N = wq.shape[0]
    bpc, S = 4 // bits, 4 * bits
    unit = 512 + 32 * bpc
    row_bytes, row_blocks = K * bits // 8, K // 64
    chunks = -(-row_bytes // 32)
    tiles = -(-N // 16)
    out = np.zeros(tiles * chunks * unit, dtype=np.uint8)
    sc = np.zeros(tiles * chunks * unit // 2, dtype=np.uint16)
    for T in range(tiles):
        for c in range(chunks):
            base = (T * chunks + c) * unit
            for r in range(16):
                n = 16 * T + r
                if n >= N:
                    continue
                r_hi, r_lo = divmod(r, S)
                for a in range(2):
                    L = 2 * r + a
                    for i in range(16):
                        j, f = divmod(i, S)
                        byte = c * 32 + (8 * bits) * ((j + r_hi) % bpc) + a + 2 * ((f + r_lo) % S)
                        if byte < row_bytes:
                            out[base + 16 * L + i] = wq[n, byte]
                for q in range(bpc):
                    blk = c * bpc + q
                    if blk < row_blocks:
                        sc[(base + 512) // 2 + r * bpc + q] = scales[n, blk]
    scb = sc.view(np.uint8)
    mask = scb != 0
    out[mask] = scb[mask]
    return out
