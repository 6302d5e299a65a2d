"""Host-side arithmetic of the two packed layouts (no GPU): the word index map of the tuned layout is injective,
stays inside kmq_packed_bytes, follows the documented formula, and the field shifts of every bit width are a
permutation of the canonical ones."""
import numpy as np
import pytest

from paper_2602_15563_b200 import build as kb
from paper_2602_15563_b200 import kmq

C, T = kmq.KMQ_LAYOUT_CANONICAL, kmq.KMQ_LAYOUT_TUNED


@pytest.fixture(scope="module", autouse=True)
def built():
    kb.build()


@pytest.mark.parametrize("bits", (1, 2, 4))
@pytest.mark.parametrize("N,Kwords", [(1, 1), (16, 16), (17, 17), (50, 33), (33, 4)])
def test_tuned_word_index_is_injective_and_documented(bits, N, Kwords):
    K = Kwords * (32 // bits)
    total = kmq.kmq_packed_bytes(N, K, bits, T) // 4
    steps = -(-Kwords // 16)
    assert total == -(-N // 16) * steps * 256
    seen = set()
    for n in range(N):
        for j in range(Kwords):
            w = kmq.kmq_packed_word_index(n, j, N, K, bits, T)
            assert w == (((n // 16) * steps + j // 16) * 16 + n % 16) * 16 + j % 16
            assert 0 <= w < total and w not in seen
            seen.add(w)
            assert kmq.kmq_packed_word_index(n, j, N, K, bits, C) == n * Kwords + j
    assert kmq.kmq_packed_word_index(N, 0, N, K, bits, T) == -1
    assert kmq.kmq_packed_word_index(0, Kwords, N, K, bits, T) == -1


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_field_shifts(bits):
    per = 32 // bits
    canon = [kmq.kmq_packed_field_shift(i, bits, C) for i in range(per)]
    tuned = [kmq.kmq_packed_field_shift(i, bits, T) for i in range(per)]
    assert canon == [i * bits for i in range(per)]
    assert sorted(tuned) == canon                                  # same fields, other order
    covered = np.zeros(32, int)
    for s in tuned:
        covered[s:s + bits] += 1
    assert np.all(covered == 1)                                    # fields tile the word exactly
    if bits == 4:
        assert tuned == canon
    if bits == 2:
        assert tuned == [2 * (i // 4) + 8 * (i % 4) for i in range(per)]
    if bits == 1:
        assert tuned == [(31 - i // 2) if i % 2 else (15 - i // 2) for i in range(per)]
    assert kmq.kmq_packed_field_shift(per, bits, T) == -1 and kmq.kmq_packed_field_shift(0, 3, T) == -1


@pytest.mark.parametrize("bits", (1, 2))
@pytest.mark.parametrize("N,K", [(1, 32), (16, 256), (37, 544), (33, 288)])
def test_table_layout_bit_index_is_injective_and_documented(bits, N, K):
    """KMQ_LAYOUT_TABLE: every index bit has its own position inside kmq_packed_bytes, at the place the header's
    formula gives; the word-based helpers do not describe this layout."""
    L = kmq.KMQ_LAYOUT_TABLE
    chunks, tiles = -(-K // 256), -(-N // 16)
    total = kmq.kmq_packed_bytes(N, K, bits, L)
    assert total == tiles * chunks * bits * 512
    seen = set()
    for n in range(N):
        for k in range(K):
            g = k // 8
            for p in range(bits):
                pos = kmq.kmq_packed_bit_index(n, k, p, N, K, bits, L)
                byte = (((n // 16) * chunks + g // 32) * bits + p) * 512 + (2 * (n % 16) + g % 2) * 16 \
                    + ((g % 32) // 2 - n % 16) % 16
                assert pos == byte * 8 + k % 8
                assert 0 <= pos < total * 8 and pos not in seen
                seen.add(pos)
    assert kmq.kmq_packed_word_index(0, 0, N, K, bits, L) == -1
    assert kmq.kmq_packed_field_shift(0, bits, L) == -1
    assert kmq.kmq_packed_bit_index(N, 0, 0, N, K, bits, L) == -1
    assert kmq.kmq_packed_bit_index(0, K, 0, N, K, bits, L) == -1
    assert kmq.kmq_packed_bit_index(0, 0, bits, N, K, bits, L) == -1


@pytest.mark.parametrize("bits", (1, 2, 4))
def test_bit_index_agrees_with_word_index_and_shift(bits):
    N, K = 19, (32 // bits) * 5
    per = 32 // bits
    for layout in (C, T) + ((kmq.KMQ_LAYOUT_TABLE,) if bits == 4 else ()):
        for n in (0, 7, 18):
            for k in (0, 1, per - 1, per, K - 1):
                w = kmq.kmq_packed_word_index(n, k // per, N, K, bits, layout)
                sh = kmq.kmq_packed_field_shift(k % per, bits, layout)
                for p in range(bits):
                    assert kmq.kmq_packed_bit_index(n, k, p, N, K, bits, layout) == w * 32 + sh + p
    assert kmq.kmq_packed_bytes(N, K, 4, kmq.KMQ_LAYOUT_TABLE) == kmq.kmq_packed_bytes(N, K, 4, T)


@pytest.mark.parametrize("bits", (1, 2, 4))
@pytest.mark.parametrize("N,K", ((16, 256), (37, 64 * 7), (5, 1024)))
def test_block_table_offsets_are_injective_and_documented(bits, N, K):
    """kmq_block_table_index_offset / _scale_offset against the layout of include/kmq.h restated here."""
    bpc, S = 4 // bits, 4 * bits
    unit = 512 + 32 * bpc
    per = 8 // bits
    chunks = -(-(K * bits // 8) // 32)
    total = kmq.kmq_block_table_bytes(N, K, bits)
    assert total == -(-N // 16) * chunks * unit
    seen = set()
    for n in range(N):
        for k in range(0, K, per):
            byte = k // per
            c, b = divmod(byte, 32)
            q, w = divmod(b, 8 * bits)
            a, m = w & 1, w >> 1
            r = n % 16
            r_hi, r_lo = divmod(r, S)
            j, f = (q - r_hi) % bpc, (m - r_lo) % S
            want = ((n // 16) * chunks + c) * unit + 16 * (2 * r + a) + S * j + f
            got = kmq.kmq_block_table_index_offset(n, k, N, K, bits)
            assert got == want == kmq.kmq_block_table_index_offset(n, k + per - 1, N, K, bits)
            assert got % unit < 512 and got not in seen
            seen.add(got)
        for blk in range(K // 64):
            want = ((n // 16) * chunks + blk // bpc) * unit + 512 + ((n % 16) * bpc + blk % bpc) * 2
            got = kmq.kmq_block_table_scale_offset(n, 64 * blk + 63, N, K, bits)
            assert got == want and got not in seen and got + 1 not in seen
            seen.update((got, got + 1))
    assert max(seen) < total
    assert kmq.kmq_block_table_index_offset(N, 0, N, K, bits) == -1
    assert kmq.kmq_block_table_scale_offset(0, K, N, K, bits) == -1
    assert kmq.kmq_block_table_bytes(N, K, 8) == 0 and kmq.kmq_block_table_bytes(N, K + 32, bits) == 0
