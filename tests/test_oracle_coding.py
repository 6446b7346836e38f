"""Pins of the CPU oracle's prefix code (Huffman lengths, canonical words, block encode / decode)."""
import itertools
import math

import numpy as np
import pytest


def _expected(w, lengths):
    w = np.asarray(w, np.float64)
    return float((w / w.sum() * lengths).sum())


def test_textbook_examples(orc):
    assert orc.huffman_lengths([0.4, 0.3, 0.2, 0.1]).tolist() == [1, 2, 3, 3]
    # dyadic probabilities: the expected length equals the entropy
    w = [0.5, 0.25, 0.125, 0.125]
    l = orc.huffman_lengths(w)
    assert l.tolist() == [1, 2, 3, 3] and _expected(w, l) == 1.75
    assert orc.huffman_lengths([1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0]).tolist() == [3] * 8
    assert orc.huffman_lengths([7.0]).tolist() == [1]
    # canonical words of lengths (1,2,3,3): 0, 10, 110, 111
    assert orc.canonical_codes([1, 2, 3, 3]).tolist() == [0b0, 0b10, 0b110, 0b111]
    assert orc.canonical_codes([3, 3, 2, 1]).tolist() == [0b110, 0b111, 0b10, 0b0]


@pytest.mark.parametrize("n", [2, 3, 4, 5, 6])
def test_optimal_against_brute_force(orc, n):
    """Minimum expected length over all length vectors that satisfy Kraft's inequality (small alphabets)."""
    rng = np.random.default_rng(n)
    for _ in range(20):
        w = rng.dirichlet(np.ones(n) * 0.5) + 1e-6
        l = orc.huffman_lengths(w)
        best = min(_expected(w, np.array(c)) for c in itertools.product(range(1, n + 1), repeat=n)
                   if sum(2.0 ** -x for x in c) <= 1.0 + 1e-12)
        assert abs(_expected(w, l) - best) < 1e-12


def test_kraft_entropy_bounds_and_prefix_freedom(orc):
    rng = np.random.default_rng(3)
    for n in (2, 8, 16, 32, 256):
        w = rng.dirichlet(np.ones(n) * 0.3)
        w[rng.integers(0, n)] = 0.0                       # a symbol of probability zero still gets a word
        l = orc.huffman_lengths(w).astype(int)
        assert np.all(l >= 1) and l.max() <= 12
        assert abs(sum(2.0 ** -x for x in l) - 1.0) < 1e-12                      # a complete code
        p = w / w.sum(); H = -sum(x * math.log2(x) for x in p if x > 0)
        if l.max() < 12:                                                         # not length-limited: optimal
            assert H - 1e-9 <= _expected(w, l) <= H + 1                              # H <= E[L] <= H + 1
        codes = orc.canonical_codes(l)
        words = sorted(format(int(c), "b").zfill(int(x)) for c, x in zip(codes, l))
        assert all(not b.startswith(a) for a, b in zip(words, words[1:]))        # prefix free
    # a geometric tail would need words longer than the limit: the limit holds and the code stays complete
    w = 0.5 ** np.arange(40)
    l = orc.huffman_lengths(w, 12).astype(int)
    assert l.max() == 12 and abs(sum(2.0 ** -x for x in l) - 1.0) < 1e-12
    assert orc.huffman_lengths(w, 32).astype(int).max() > 12


def test_block_layout_by_hand_and_round_trip(orc):
    lengths = np.uint8([1, 2, 3, 3]); codes = orc.canonical_codes(lengths)
    # coordinates 0..5 of a block: lane 0 holds c = 0,1,2,3 (p = 0..3), lane 1 holds c = 4,5 (p = 0,1): the stream
    # visits lane 0 first.  idx = [1,0,3,2,0,1], sign = [1,0,0,1,0,0]:
    #   c0: 10 + sign 1 | c1: 0 | c2: 111 + sign 0 | c3: 110 + sign 1 | c4: 0 | c5: 10 + sign 0
    idx = np.uint8([1, 0, 3, 2, 0, 1]); sg = np.uint8([1, 0, 0, 1, 0, 0])
    words, bits = orc.entropy_encode_block(idx, sg, lengths, codes)
    want = "101" + "0" + "1110" + "1101" + "0" + "100"
    assert bits == len(want) and words.size == 1
    assert format(int(words[0]), "b").zfill(bits)[::-1] == want                 # stream bit t = bit t of the word
    rng = np.random.default_rng(5)
    for n, count in [(16, 1024), (16, 1), (8, 1000), (256, 513), (2, 77)]:
        l = orc.huffman_lengths(rng.dirichlet(np.ones(n) * 0.4)); c = orc.canonical_codes(l)
        idx = rng.integers(0, n, count).astype(np.uint8); sg = (rng.integers(0, 2, count) * (idx != 0)).astype(np.uint8)
        words, bits = orc.entropy_encode_block(idx, sg, l, c)
        assert bits == int(l[idx].astype(int).sum() + np.count_nonzero(idx))
        i2, s2, used = orc.entropy_decode_block(words, count, l, c)
        assert used == bits and np.array_equal(i2, idx) and np.array_equal(s2, sg)


def test_elias_recursive_code_words(orc):
    """Elias' recursive code against the words its definition gives by hand, prefix-freeness, Kraft's inequality and
    the round trip through the decoder."""
    by_hand = {1: "0", 2: "100", 3: "110", 4: "101000", 7: "101110", 8: "1110000", 15: "1111110",
               16: "10100100000", 100: "1011011001000"}
    for v, w in by_hand.items():
        assert orc.elias_omega(v) == w, v
    words = [orc.elias_omega(v) for v in range(1, 300)]
    assert sum(2.0 ** -len(w) for w in words) < 1.0
    for i, a in enumerate(words):
        for j, b in enumerate(words):
            assert i == j or not b.startswith(a)
    lens = [len(w) for w in words]
    assert all(x <= y for x, y in zip(lens, lens[1:]))                 # smaller values never get longer words
    stream = "".join(words[v - 1] for v in [5, 1, 299, 64, 2])
    pos, out = 0, []
    while pos < len(stream):
        v, used = orc.elias_omega_decode(stream[pos:])
        out.append(v); pos += used
    assert out == [5, 1, 299, 64, 2]
