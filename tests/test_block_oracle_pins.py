"""Pins of the block-format oracle (oracle/kmq_block_oracle.py) against things other than itself: pure-Python brute
force, the per-row oracle in the special case where the two formats coincide, the paper's first listing restated
literally with a 256-entry table, the agreement of the two scale orders, the printed bits per weight and the bytes
behind the paper's effective-bandwidth figures, and planted mistakes that must fail."""
import math
import struct

import numpy as np
import pytest

from oracle import kmq_block_oracle as blk
from oracle import kmq_oracle as orc


def bf16_f(b):                                  # bf16 bit pattern -> Python float, by the format's definition
    return struct.unpack("<f", struct.pack("<I", int(b) << 16))[0]


def to_bf16(a):                                 # float32 -> bf16 bits, truncation-free inputs only (tests pick exact values)
    u = np.asarray(a, dtype=np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "test values must be exact in bf16"
    return (u >> 16).astype(np.uint16)


def rand_bf16(rng, shape, scale=1.0):
    u = (rng.standard_normal(shape) * scale).astype(np.float32).view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def make(rng, N, K, bits, M):
    idx = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    cb = np.sort(rand_bf16(rng, (1 << bits,), 0.5).view(np.int16)).view(np.uint16)
    scales = rand_bf16(rng, (N, K // 64), 0.02)
    x = rand_bf16(rng, (M, K))
    return idx, cb, scales, x


def slow_bf16_round(val: float) -> int:
    """Nearest bf16 of a float, ties to even, from the value alone (frexp), not from float32 bit tricks."""
    if val == 0.0:
        return 0x8000 if math.copysign(1.0, val) < 0 else 0
    m, e = math.frexp(abs(val))
    e_b = e - 1
    if e_b < -126:
        bits = int(round(abs(val) / 2.0 ** -133))            # Python's round: half to even
    else:
        bits = ((e_b + 127) << 7) + int(round((2.0 * m - 1.0) * 128.0))
    return (0x8000 if val < 0 else 0) | bits


@pytest.mark.parametrize("bits", (1, 2, 4, 8))
def test_brute_force_tiny(bits):
    rng = np.random.default_rng(bits)
    N, K, M = 5, 128, 2
    idx, cb, scales, x = make(rng, N, K, bits, M)
    wq = blk.pack_bytes(idx, bits)
    per = 8 // bits
    for order in ("direct", "deferred"):
        y, a = blk.block_linear_f64(wq, scales, cb, x, K, bits, order)
        for m in range(M):
            for n in range(N):
                terms = []
                for k in range(K):
                    byte = int(wq[n, k // per])
                    i = (byte >> ((k % per) * bits)) & ((1 << bits) - 1)          # LSB-first field
                    assert i == idx[n, k]
                    terms.append(bf16_f(x[m, k]) * bf16_f(scales[n, k // 64]) * bf16_f(cb[i]))
                ref = math.fsum(terms)
                assert abs(y[m, n] - ref) <= 1e-12 * max(1.0, math.fsum(abs(t) for t in terms))
                assert abs(a[m, n] - math.fsum(abs(t) for t in terms)) <= 1e-12 * max(1.0, a[m, n])


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_unit_scales_reduce_to_the_per_row_oracle(bits):
    """All scales 1 and every row using the tensor's codebook: the per-row format with equal codebooks."""
    rng = np.random.default_rng(10 + bits)
    N, K, M = 33, 256, 3
    idx, cb, _, x = make(rng, N, K, bits, M)
    ones = np.full((N, K // 64), 0x3F80, np.uint16)
    y_b, a_b = blk.block_linear_f64(blk.pack_bytes(idx, bits), ones, cb, x, K, bits)
    y_r, a_r = orc.linear_f64(orc.pack_canonical(idx, bits), np.tile(cb, (N, 1)), x, K, bits)
    assert np.allclose(y_b, y_r, rtol=1e-13, atol=1e-15) and np.allclose(a_b, a_r, rtol=1e-13)
    # the bytes are the canonical words seen as little-endian bytes
    assert np.array_equal(blk.pack_bytes(idx, bits), orc.pack_canonical(idx, bits).view(np.uint8).reshape(N, -1))


@pytest.mark.parametrize("bits", (1, 2, 4, 8))
def test_direct_and_deferred_agree_in_float64(bits):
    rng = np.random.default_rng(20 + bits)
    idx, cb, scales, x = make(rng, 40, 512, bits, 4)
    wq = blk.pack_bytes(idx, bits)
    y1, a1 = blk.block_linear_f64(wq, scales, cb, x, 512, bits, "direct")
    y2, a2 = blk.block_linear_f64(wq, scales, cb, x, 512, bits, "deferred")
    assert np.all(np.abs(y1 - y2) <= 1e-12 * a1) and np.array_equal(a1, a2)


@pytest.mark.parametrize("bits", (1, 4, 8))
def test_equals_the_first_listing_restated(bits):
    """Gather from a 256-entry byte table, scale every block, contract: the listing's steps in loops."""
    rng = np.random.default_rng(30 + bits)
    N, K, M = 7, 192, 2
    idx, cb, scales, x = make(rng, N, K, bits, M)
    wq = blk.pack_bytes(idx, bits)
    per = 8 // bits
    table = [[bf16_f(cb[(byte >> (i * bits)) & ((1 << bits) - 1)]) for i in range(per)] for byte in range(256)]
    W = np.zeros((N, K))
    for n in range(N):
        wu = [v for byte in wq[n] for v in table[int(byte)]]
        for k in range(K):
            W[n, k] = wu[k] * bf16_f(scales[n, k // 64])
    xf = np.array([[bf16_f(v) for v in row] for row in x])
    y, _ = blk.block_linear_f64(wq, scales, cb, x, K, bits)
    assert np.allclose(y, xf @ W.T, rtol=1e-13, atol=1e-15)
    assert np.array_equal(blk.lut8(cb, bits).shape, (256, per))


def test_bits_per_weight_and_the_papers_micro_benchmark_bytes():
    """P_w = b + 16/64 (Section 2.1, the 4.25-bit example) and the micro-benchmark table of Section 3.3: a 1 x 8192
    by 8192 x 8192 product in 49.5 us at 721 GB/s (4.25 bits) and 24.0 us at 438 GB/s (1.25 bits) moves P_w / 8
    bytes per weight."""
    assert blk.block_bits_per_weight(4) == 4.25 and blk.block_bits_per_weight(1) == 1.25
    assert blk.block_bits_per_weight(2) == 2.25 and blk.block_bits_per_weight(8) == 8.25
    for bits, us, gbs in ((4, 49.5, 721.0), (1, 24.0, 438.0)):
        weight_bytes = 8192 * 8192 * blk.block_bits_per_weight(bits) / 8
        assert abs(weight_bytes / (us * 1e-6) / 1e9 - gbs) / gbs < 0.012       # the table rounds to 3 digits


def test_scaled_dequant_rounding_matches_a_value_based_rounding():
    rng = np.random.default_rng(5)
    idx, cb, scales, _ = make(rng, 9, 128, 4, 1)
    wq = blk.pack_bytes(idx, 4)
    got = blk.dequant_scaled_bits(wq, scales, cb, 128, 4)
    for n in range(9):
        for k in range(128):
            exact = bf16_f(scales[n, k // 64]) * bf16_f(cb[idx[n, k]])
            assert got[n, k] == slow_bf16_round(exact)
    # ties: 1.00390625 * 1.0 = 1 + 2^-8 lies between two bf16 values -> even mantissa (1.0)
    assert blk.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert blk.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    assert blk.f64_to_bf16_bits(np.array([-0.0]))[0] == 0x8000


def test_pack_unpack_round_trip_and_field_order():
    for bits in (1, 2, 4, 8):
        per = 8 // bits
        rng = np.random.default_rng(bits)
        idx = rng.integers(0, 256, size=(6, per * 24), dtype=np.uint8)
        wq = blk.pack_bytes(idx, bits)
        assert np.array_equal(blk.unpack_bytes(wq, idx.shape[1], bits), idx & ((1 << bits) - 1))
        one = np.zeros((1, per), np.uint8)
        for i in range(per):
            one[:] = 0
            one[0, i] = (1 << bits) - 1
            assert blk.pack_bytes(one, bits)[0, 0] == ((1 << bits) - 1) << (i * bits)   # field i at bits [i*b, (i+1)*b)
    assert np.array_equal(blk.pack_bytes(np.array([[1, 0, 0, 0, 0, 0, 0, 1]], np.uint8), 1), [[0x81]])
    assert np.array_equal(blk.pack_bytes(np.array([[0x3, 0xA]], np.uint8), 4), [[0xA3]])   # low nibble first


def test_planted_mistakes_are_caught():
    rng = np.random.default_rng(77)
    N, K, M, bits = 6, 256, 2, 2
    idx, cb, scales, x = make(rng, N, K, bits, M)
    wq = blk.pack_bytes(idx, bits)
    y, a = blk.block_linear_f64(wq, scales, cb, x, K, bits)
    tol = 1e-9 * a

    def differs(y2):
        return np.any(np.abs(y2 - y) > tol)
    # MSB-first fields inside a byte
    rev = idx.reshape(N, K // 4, 4)[:, :, ::-1].reshape(N, K)
    assert differs(blk.block_linear_f64(blk.pack_bytes(rev, bits), scales, cb, x, K, bits)[0])
    # the scale of the neighbouring block
    assert differs(blk.block_linear_f64(wq, np.roll(scales, 1, axis=1), cb, x, K, bits)[0])
    # scales indexed by the wrong row
    assert differs(blk.block_linear_f64(wq, scales[::-1].copy(), cb, x, K, bits)[0])
    # a codebook with two entries swapped
    cb2 = cb.copy()
    cb2[[0, 1]] = cb2[[1, 0]]
    assert differs(blk.block_linear_f64(wq, scales, cb2, x, K, bits)[0])
