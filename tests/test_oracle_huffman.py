"""Pins of the oracle's Huffman code (Sect. IV-B): Kraft equality, the bound
H <= average length <= H + 1 the paper quotes, optimality by brute force on tiny
alphabets, and the closed forms for equiprobable sources."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import hac_oracle as orc


def kraft(lengths):
    return sum(Fraction(1, 2 ** int(l)) for l in lengths)


def brute_force_best_cost(counts):
    """Minimum of sum(count * length) over all length vectors that some prefix code has
    (Kraft sum <= 1), by plain enumeration."""
    k = len(counts)
    best = None
    for lens in itertools.product(range(1, k + 1), repeat=k):
        if kraft(lens) <= 1:
            cost = sum(c * l for c, l in zip(counts, lens))
            best = cost if best is None else min(best, cost)
    return best


@pytest.mark.parametrize("seed", range(12))
def test_optimal_on_tiny_alphabets(seed):
    rng = np.random.default_rng(seed)
    k = int(rng.integers(2, 7))
    counts = rng.integers(1, 30, size=k).tolist()
    if seed % 3 == 0:
        counts = [int(c) for c in rng.integers(1, 4, size=k)]          # many ties
    lengths = orc.huffman_lengths(counts)
    assert sum(c * int(l) for c, l in zip(counts, lengths)) == brute_force_best_cost(counts)


@pytest.mark.parametrize("seed", range(8))
def test_kraft_equality_and_entropy_bound(seed):
    rng = np.random.default_rng(100 + seed)
    k = int(rng.integers(2, 400))
    counts = np.maximum(1, (rng.pareto(1.2, size=k) * 50).astype(np.int64))
    lengths = orc.huffman_lengths(counts)
    assert kraft(lengths) == 1
    H = orc.entropy_bits(counts)
    avg = float((counts * lengths.astype(np.int64)).sum() / counts.sum())
    assert H - 1e-12 <= avg <= H + 1 + 1e-12
    # a more frequent symbol never has a longer code word
    order = np.argsort(counts, kind="stable")
    assert all(lengths[order[i]] >= lengths[order[i + 1]] or counts[order[i]] == counts[order[i + 1]]
               for i in range(k - 1))


@pytest.mark.parametrize("j", [1, 2, 5, 8])
def test_equiprobable_power_of_two_gives_fixed_length(j):
    # Table III: the equiprobable quantizer at k = 256 costs 8 bits per weight (psi = 0.2500)
    lengths = orc.huffman_lengths([7] * (2 ** j))
    assert set(lengths.tolist()) == {j}
    if j == 8:
        assert round(8 / 32.0, 4) == 0.2500


def test_degenerate_alphabets():
    assert orc.huffman_lengths([5]).tolist() == [1]
    assert orc.huffman_lengths([1, 1000]).tolist() == [1, 1]
    with pytest.raises(ValueError):
        orc.huffman_lengths([3, 0, 2])


def test_fibonacci_counts_give_a_comb():
    # textbook worst case: Fibonacci frequencies produce lengths 1,2,...,k-1,k-1
    counts = [1, 1, 2, 3, 5, 8, 13, 21]
    lengths = orc.huffman_lengths(counts)
    assert sorted(lengths.tolist()) == [1, 2, 3, 4, 5, 6, 7, 7]


def test_canonical_codes_are_a_prefix_code_in_order():
    rng = np.random.default_rng(9)
    counts = rng.integers(1, 1000, size=57)
    lengths = orc.huffman_lengths(counts)
    codes = orc.canonical_codes(lengths)
    words = [format(int(c), f"0{int(l)}b") for c, l in zip(codes, lengths)]
    assert len(set(words)) == len(words)
    for a in words:
        for b in words:
            assert a == b or not b.startswith(a)
    # ordered by (length, id): as left-aligned binary fractions the code words increase
    order = sorted(range(len(words)), key=lambda s: (int(lengths[s]), s))
    frac = [Fraction(int(codes[s]), 2 ** int(lengths[s])) for s in order]
    assert all(frac[i] < frac[i + 1] for i in range(len(frac) - 1))
    assert int(codes[order[0]]) == 0
    # a complete code: the last code word is all ones
    assert words[order[-1]] == "1" * int(lengths[order[-1]])


def test_tie_rule_keeps_codes_shallow():
    # counts 1,1,1,1: taking leaves before merged nodes gives 2,2,2,2 (not 1,2,3,3)
    assert orc.huffman_lengths([1, 1, 1, 1]).tolist() == [2, 2, 2, 2]
    # counts 1,1,2: the merged node (weight 2) ties with the leaf of weight 2; the leaf goes first
    assert orc.huffman_lengths([1, 1, 2]).tolist() == [2, 2, 1]
