"""Pins for the oracle's packed b-bit layout (8 int4 per uint32; 32 int3 per three uint32)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "packed_layout_vectors.txt")


def _vectors():
    with open(GOLD) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, codes, words = [p.strip() for p in line.split("|")]
            yield int(bits), [int(c) for c in codes.split(",")], [int(w, 16) for w in words.split(",")]


def test_hand_vectors():
    for bits, codes, words in _vectors():
        c = np.array(codes, np.uint8)[None, :]
        w = oracle.pack(c, bits)
        assert [int(x) for x in w[0]] == words
        assert np.array_equal(oracle.unpack(np.array(words, np.uint32)[None, :], 32, bits), c)


@pytest.mark.parametrize("bits", [3, 4])
def test_against_python_big_integers(bits):
    rng = np.random.default_rng(bits)
    K = 160
    codes = rng.integers(0, 1 << bits, size=(5, K), dtype=np.uint8)
    words = oracle.pack(codes, bits)
    for i in range(5):
        v = sum(int(c) << (bits * j) for j, c in enumerate(codes[i]))
        expect = [(v >> (32 * w)) & 0xFFFFFFFF for w in range(K * bits // 32)]
        assert [int(x) for x in words[i]] == expect


@pytest.mark.parametrize("bits", [3, 4])
def test_roundtrips(bits):
    rng = np.random.default_rng(100 + bits)
    codes = rng.integers(0, 1 << bits, size=(9, 256), dtype=np.uint8)
    words = oracle.pack(codes, bits)
    assert words.shape == (9, 256 * bits // 32)
    assert np.array_equal(oracle.unpack(words, 256, bits), codes)
    raw = rng.integers(0, 2 ** 32, size=(9, 256 * bits // 32), dtype=np.uint64).astype(np.uint32)
    assert np.array_equal(oracle.pack(oracle.unpack(raw, 256, bits), bits), raw)


def test_rows_do_not_share_words():
    codes = np.zeros((2, 32), np.uint8)
    codes[1, :] = 7
    w = oracle.pack(codes, 3)
    assert np.all(w[0] == 0) and np.all(w[1] == 0xFFFFFFFF)
