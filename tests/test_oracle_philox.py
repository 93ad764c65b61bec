"""Pins for the oracle's Philox4x32-10 and its stream layout (CPU only)."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ctr, key, out = [[int(w, 16) for w in part.split()] for part in line.split("|")]
        rows.append((ctr, key, out))
    assert len(rows) == 3
    return rows


def test_known_answer_vectors():
    for ctr, key, out in _kat():
        assert oracle.philox4x32_10(ctr, key).tolist() == out


def test_stream_starts_with_first_known_answer():
    # seed 0 -> key (0, 0); elements 0..3 are block 0 = counter (0, 0, 0, 0)
    assert oracle.gen_u32(0, 0, 4).tolist() == _kat()[0][2]


def test_stream_layout_blocks_and_key_words():
    seed = 0x299F31D0A4093822          # key words (a4093822, 299f31d0)
    key = [0xA4093822, 0x299F31D0]
    for block in (0, 1, 7, 0xFFFFFFFF, 0x100000000, 0x123456789A, (1 << 62) - 1):
        want = oracle.philox4x32_10([block & 0xFFFFFFFF, block >> 32, 0, 0], key)
        got = oracle.gen_u32(seed, 4 * block, 4)
        assert got.tolist() == want.tolist(), hex(block)


def test_slicing_invariant_any_offset():
    whole = oracle.gen_u32(77, 0, 4096)
    for a, n in [(0, 1), (1, 5), (2, 17), (3, 1000), (1023, 1025), (4095, 1), (10, 0)]:
        assert np.array_equal(oracle.gen_u32(77, a, n), whole[a:a + n])
    far = 0xFFFFFFFF0
    big = oracle.gen_u32(5, far - 8, 64)
    assert np.array_equal(oracle.gen_u32(5, far + 3, 11), big[11:22])


def test_seeds_and_blocks_are_distinct_and_uniform():
    # A counter-based generator is a bijection per key: no repeated blocks; and
    # the words look uniform (chi-square over bytes, 255 d.o.f.).
    w = oracle.gen_u32(123, 0, 1 << 16).reshape(-1, 4)
    assert len({tuple(r) for r in w.tolist()}) == w.shape[0]
    assert not np.array_equal(oracle.gen_u32(123, 0, 64), oracle.gen_u32(124, 0, 64))
    assert not np.array_equal(oracle.gen_u32(123, 0, 64), oracle.gen_u32(123 + (1 << 32), 0, 64))
    counts = np.bincount(w.reshape(-1).view(np.uint8), minlength=256).astype(np.float64)
    expected = counts.sum() / 256
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert 150 < chi2 < 380      # far tails of chi-square(255)
