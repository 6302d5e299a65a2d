"""Pins for the CPU oracle: each test ties one part of it to something that is
not the oracle itself (pure-Python brute force, a closed form, a special case
that collapses to a textbook operation, an exactly rounded sum)."""
import math
import struct

import numpy as np
import pytest

from oracle import kmq_oracle as orc

BITS = (1, 2, 4)


# ---------- independent helpers (pure Python, no NumPy arithmetic) ----------
def py_bf16(u16: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (int(u16) & 0xFFFF) << 16))[0]


def py_field(word: int, i: int, bits: int) -> int:
    return (int(word) >> (i * bits)) % (1 << bits)


def py_index(packed_row, k: int, bits: int) -> int:
    per = 32 // bits
    return py_field(packed_row[k // per], k % per, bits)


def random_case(rng, N, K, bits, M):
    idx = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    cb = rng.integers(0, 1 << 16, size=(N, 1 << bits), dtype=np.uint16)
    # keep exponents moderate so every value is finite and sums do not overflow
    cb = (cb & np.uint16(0x80FF)) | np.uint16(0x3C00) | (cb & np.uint16(0x0300))
    x = rng.integers(0, 1 << 16, size=(M, K), dtype=np.uint16)
    x = (x & np.uint16(0x80FF)) | np.uint16(0x3E00) | (x & np.uint16(0x0180))
    return idx, cb, x


# ---------- 1. brute force on tiny shapes ----------
@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("N,K,M", [(1, 32, 1), (3, 64, 2), (5, 96, 3), (7, 32, 1)])
def test_brute_force_tiny(bits, N, K, M):
    rng = np.random.default_rng(100 + bits + N + K)
    idx, cb, x = random_case(rng, N, K, bits, M)
    packed = orc.pack_canonical(idx, bits)
    w_bits = orc.dequant_bits(packed, cb, K, bits)
    y, s = orc.linear_f64(packed, cb, x, K, bits)
    for n in range(N):
        prow = [int(v) for v in packed[n]]
        for k in range(K):
            i = py_index(prow, k, bits)
            assert i == int(idx[n, k])
            assert int(w_bits[n, k]) == int(cb[n, i])
    for m in range(M):
        for n in range(N):
            prow = [int(v) for v in packed[n]]
            terms = [py_bf16(x[m, k]) * py_bf16(cb[n, py_index(prow, k, bits)]) for k in range(K)]
            ref = math.fsum(terms)
            ref_abs = math.fsum(abs(t) for t in terms)
            assert abs(y[m, n] - ref) <= 1e-12 * ref_abs + 1e-300
            assert abs(s[m, n] - ref_abs) <= 1e-12 * ref_abs + 1e-300


# ---------- 2. one-bit codebook {-a, +a} is a scaled sign matmul ----------
@pytest.mark.parametrize("order", ["neg_first", "pos_first"])
def test_one_bit_symmetric_codebook_is_sign_matmul(order):
    rng = np.random.default_rng(7)
    N, K, M = 33, 256, 4
    idx = rng.integers(0, 2, size=(N, K), dtype=np.uint8)
    # a_n exactly representable in bf16: 8 significant bits
    a = (rng.integers(128, 256, size=N).astype(np.float64)) * 2.0 ** -13
    a_bits = (a.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    neg = a_bits | np.uint16(0x8000)
    cb = np.stack([neg, a_bits], axis=1) if order == "neg_first" else np.stack([a_bits, neg], axis=1)
    x = (rng.standard_normal((M, K)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    sign = 2.0 * idx.astype(np.float64) - 1.0
    if order == "pos_first":
        sign = -sign
    expect = (xf @ sign.T) * a[None, :]
    y, s = orc.linear_f64(orc.pack_canonical(idx, 1), cb, x, K, 1)
    np.testing.assert_allclose(y, expect, rtol=0, atol=1e-12 * np.abs(xf).sum(axis=1).max())
    np.testing.assert_allclose(s, np.abs(xf).sum(axis=1)[:, None] * a[None, :], rtol=1e-13)


# ---------- 3. uniform-grid codebook is integer quantisation ----------
@pytest.mark.parametrize("bits", BITS)
def test_uniform_grid_codebook_is_integer_quantisation(bits):
    rng = np.random.default_rng(11 + bits)
    N, K, M = 17, 128, 3
    Q = 1 << bits
    z = Q // 2
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    scale = 2.0 ** rng.integers(-9, -3, size=N).astype(np.float64)     # powers of two
    grid = (np.arange(Q, dtype=np.float64)[None, :] - z) * scale[:, None]
    cb = (grid.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    assert np.array_equal((cb.astype(np.uint32) << 16).view(np.float32).astype(np.float64), grid)
    x = (rng.standard_normal((M, K)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ints = idx.astype(np.int64) - z
    expect = (xf @ ints.astype(np.float64).T) * scale[None, :]
    y, _ = orc.linear_f64(orc.pack_canonical(idx, bits), cb, x, K, bits)
    np.testing.assert_allclose(y, expect, rtol=0, atol=1e-12 * np.abs(xf).sum(axis=1).max())
    # the paper's symmetric grid {-(2^(b-1)-1) .. 2^(b-1)-1} with the spare code duplicated
    if bits >= 2:
        lim = Q // 2 - 1
        sym = np.clip(np.arange(Q) - z, -lim, lim).astype(np.float64)
        cb2 = np.tile((sym.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16), (N, 1))
        y2, _ = orc.linear_f64(orc.pack_canonical(idx, bits), cb2, x, K, bits)
        expect2 = xf @ np.clip(ints, -lim, lim).astype(np.float64).T
        np.testing.assert_allclose(y2, expect2, rtol=0, atol=1e-12 * np.abs(xf).sum(axis=1).max())


# ---------- 4. pack / unpack round trip, bit positions ----------
@pytest.mark.parametrize("bits", BITS)
def test_round_trip_random_and_adversarial(bits):
    per = 32 // bits
    Q = 1 << bits
    rng = np.random.default_rng(bits)
    K = per * 5
    cases = [rng.integers(0, Q, size=(9, K), dtype=np.uint8),
             np.zeros((2, K), np.uint8), np.full((2, K), Q - 1, np.uint8),
             (np.arange(2 * K).reshape(2, K) % Q).astype(np.uint8),
             (np.arange(2 * K).reshape(2, K) % 2 * (Q - 1)).astype(np.uint8)]
    for idx in cases:
        packed = orc.pack_canonical(idx, bits)
        assert packed.dtype == np.uint32 and packed.shape == (idx.shape[0], K // per)
        assert np.array_equal(orc.unpack_canonical(packed, K, bits), idx)
    # a single non-zero field lands at the documented bit position
    for pos in range(K):
        idx = np.zeros((1, K), np.uint8)
        idx[0, pos] = Q - 1
        packed = orc.pack_canonical(idx, bits)
        expect = np.zeros(K // per, dtype=np.uint64)
        expect[pos // per] = (Q - 1) << ((pos % per) * bits)
        assert np.array_equal(packed[0].astype(np.uint64), expect)
    # all-zero / all-one words
    assert np.all(orc.pack_canonical(np.full((1, K), Q - 1, np.uint8), bits) == np.uint32(0xFFFFFFFF))
    # values above 2^bits - 1 are reduced to their low bits
    big = rng.integers(0, 256, size=(3, K), dtype=np.uint8)
    assert np.array_equal(orc.unpack_canonical(orc.pack_canonical(big, bits), K, bits), big % Q)


def test_canonical_words_match_little_endian_byte_stream():
    """b=4: word bytes in memory order carry (low nibble, high nibble) pairs;
    b=1: numpy's little-bit-order packbits gives the same stream."""
    rng = np.random.default_rng(3)
    idx = rng.integers(0, 2, size=(4, 96), dtype=np.uint8)
    by = np.packbits(idx, axis=1, bitorder="little")
    assert np.array_equal(orc.pack_canonical(idx, 1).view(np.uint8).reshape(4, -1), by)
    idx4 = rng.integers(0, 16, size=(4, 64), dtype=np.uint8)
    by4 = (idx4[:, 0::2] | (idx4[:, 1::2] << 4)).astype(np.uint8)
    assert np.array_equal(orc.pack_canonical(idx4, 4).view(np.uint8).reshape(4, -1), by4)


# ---------- 5. shared codebook == byte-table formulation of the paper ----------
@pytest.mark.parametrize("bits", BITS)
def test_shared_codebook_equals_byte_table_gather(bits):
    """With one codebook for all rows (and unit block scales) the layer is the
    paper's reference semantics: a 256-entry table maps each packed byte to
    its 8/bits decoded values, the decoded matrix multiplies x."""
    rng = np.random.default_rng(40 + bits)
    N, K, M = 12, 128, 2
    Q = 1 << bits
    epb = 8 // bits
    idx = rng.integers(0, Q, size=(N, K), dtype=np.uint8)
    c = np.sort(rng.standard_normal(Q)).astype(np.float32)
    c_bits = (c.view(np.uint32) >> 16).astype(np.uint16)
    c64 = (c_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    table = np.empty((256, epb), dtype=np.float64)
    for byte in range(256):
        for e in range(epb):
            table[byte, e] = c64[(byte >> (e * bits)) & (Q - 1)]
    wq = orc.pack_canonical(idx, bits).view(np.uint8).reshape(N, K // epb)   # little-endian host
    w = table[wq].reshape(N, K)
    x = (rng.standard_normal((M, K)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    y, _ = orc.linear_f64(orc.pack_canonical(idx, bits), np.tile(c_bits, (N, 1)), x, K, bits)
    np.testing.assert_allclose(y, xf @ w.T, rtol=0, atol=1e-12 * np.abs(xf).sum())
    assert np.array_equal(orc.bf16_bits_to_f64(orc.dequant_bits(orc.pack_canonical(idx, bits),
                                                                 np.tile(c_bits, (N, 1)), K, bits)), w)


# ---------- 6. bf16 widening and -0.0 ----------
def test_bf16_widening_matches_struct_and_keeps_negative_zero():
    pats = np.array([0x0000, 0x8000, 0x3F80, 0xBF80, 0x0080, 0x7F7F, 0xFF7F, 0x0001, 0x3C23], np.uint16)
    wide = orc.bf16_bits_to_f64(pats)
    for p, v in zip(pats, wide):
        assert v == py_bf16(p)
    assert math.copysign(1.0, wide[1]) == -1.0
    cb = np.array([[0x8000, 0x0000]], np.uint16)
    idx = np.array([[0, 1] * 16], np.uint8)
    out = orc.dequant_bits(orc.pack_canonical(idx, 1), cb, 32, 1)
    assert np.array_equal(out[0, :4], np.array([0x8000, 0x0000, 0x8000, 0x0000], np.uint16))


# ---------- 7. acceptance rule ----------
def test_tolerance_rule_and_checker():
    s = np.array([[0.0, 1.0, 128.0]])
    np.testing.assert_allclose(orc.tolerance(s), [[1e-6, 2 ** -7 + 1e-6, 1.0 + 1e-6]])
    y_ref = np.array([[0.0, 1.0, -2.0]])
    good = np.array([[0x0000, 0x3F80, 0xC000]], np.uint16)          # 0, 1, -2 exactly
    assert orc.check_linear(good, y_ref, s) == 0.0
    off = np.array([[0x0000, 0x3F81, 0xC000]], np.uint16)           # 1 + 2^-7
    r = orc.check_linear(off, y_ref, s)
    assert 0.99 < r < 1.0
    bad = np.array([[0x0000, 0x3F82, 0xC000]], np.uint16)           # 1 + 2^-6
    assert orc.check_linear(bad, y_ref, s) > 1.0
    nan = np.array([[0x7FC0, 0x3F80, 0xC000]], np.uint16)
    assert orc.check_linear(nan, y_ref, s) == float("inf")


# ---------- 8. planted mistakes are caught by the pins above ----------
def test_pins_catch_planted_mistakes(monkeypatch):
    """Break the oracle in plausible ways (on the CPU) and check that the
    brute-force pin notices each of them."""
    def run_pin():
        test_brute_force_tiny(2, 3, 64, 2)
        test_brute_force_tiny(4, 5, 96, 3)
        test_brute_force_tiny(1, 5, 96, 3)

    run_pin()
    real_unpack = orc.unpack_canonical

    def msb_first(packed, K, bits):
        per = 32 // bits
        out = real_unpack(packed, K, bits).reshape(packed.shape[0], -1, per)
        return out[:, :, ::-1].reshape(packed.shape[0], K)
    monkeypatch.setattr(orc, "unpack_canonical", msb_first)
    with pytest.raises(AssertionError):
        run_pin()
    monkeypatch.setattr(orc, "unpack_canonical", real_unpack)

    real_take = np.take_along_axis

    def shifted_rows(a, i, axis):
        return real_take(np.roll(a, 1, axis=0), i, axis)
    monkeypatch.setattr(np, "take_along_axis", shifted_rows)      # wrong row's codebook
    with pytest.raises(AssertionError):
        run_pin()
    monkeypatch.setattr(np, "take_along_axis", real_take)

    real_widen = orc.bf16_bits_to_f64
    monkeypatch.setattr(orc, "bf16_bits_to_f64", lambda b: np.abs(real_widen(b)))   # dropped sign
    with pytest.raises(AssertionError):
        run_pin()
    monkeypatch.setattr(orc, "bf16_bits_to_f64", real_widen)
    run_pin()
