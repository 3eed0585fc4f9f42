"""Pins of the oracle's Huffman code lengths: a textbook worked example, the Kraft equality, the entropy bounds,
dyadic and uniform distributions (closed form), and brute force over all prefix-code length vectors on tiny alphabets."""
import itertools
import math

import numpy as np
import pytest

import oracle


def kraft(lengths):
    return sum(2.0 ** -int(l) for l in lengths if l > 0)


def test_textbook_example():
    # frequencies 45, 13, 12, 16, 9, 5 (the six-letter example of Cormen et al., Introduction to Algorithms,
    # ch. "Huffman codes"): code lengths 1, 3, 3, 3, 4, 4 and 224 bits per 100 letters
    lengths, total = oracle.huffman_lengths([45, 13, 12, 16, 9, 5])
    assert list(lengths) == [1, 3, 3, 3, 4, 4] and total == 224


def test_dyadic_and_uniform_distributions_have_closed_forms():
    lengths, total = oracle.huffman_lengths([8, 4, 2, 1, 1])           # p = 1/2, 1/4, 1/8, 1/16, 1/16
    assert list(lengths) == [1, 2, 3, 4, 4] and total == 8 + 8 + 6 + 4 + 4
    for b in (1, 2, 4, 8):
        lengths, total = oracle.huffman_lengths([7] * (1 << b))
        assert set(lengths) == {b} and total == 7 * b * (1 << b)


def test_degenerate_alphabets():
    assert oracle.huffman_lengths([0, 0, 0])[1] == 0
    lengths, total = oracle.huffman_lengths([0, 9, 0])
    assert list(lengths) == [0, 1, 0] and total == 9
    lengths, total = oracle.huffman_lengths([3, 0, 5])
    assert list(lengths) == [1, 0, 1] and total == 8


@pytest.mark.parametrize("seed", range(6))
def test_kraft_equality_and_entropy_bounds(seed):
    rng = np.random.default_rng(seed)
    nlev = int(rng.integers(2, 257))
    h = rng.integers(0, 1000, nlev) * (rng.random(nlev) < 0.8)
    h[rng.integers(0, nlev)] += 5
    h[rng.integers(0, nlev)] += 3
    if (h > 0).sum() < 2:
        h[:2] += 1
    lengths, total = oracle.huffman_lengths(h)
    assert abs(kraft(lengths) - 1.0) < 1e-12                        # a full binary tree
    assert all((l > 0) == (c > 0) for l, c in zip(lengths, h))
    n = int(h.sum())
    H = -sum(c / n * math.log2(c / n) for c in h if c > 0)
    assert H - 1e-12 <= total / n < H + 1.0                         # Shannon's bounds for an optimal prefix code


def test_optimal_among_all_prefix_codes_on_tiny_alphabets():
    # brute force: every length vector with Kraft sum <= 1 is realisable as a prefix code; none beats Huffman
    rng = np.random.default_rng(42)
    for m in (2, 3, 4, 5):
        for _ in range(6):
            h = rng.integers(1, 40, m)
            best = min(sum(int(c) * l for c, l in zip(h, ls))
                       for ls in itertools.product(range(1, m + 1), repeat=m) if kraft(ls) <= 1.0 + 1e-12)
            assert oracle.huffman_lengths(h)[1] == best
