"""Pins for the oracle's quantiser, statistics and Huffman code (Section 3.1 "Quantization"
and "Variable length coding"; Appendix D).  Hand-made values, closed forms, invariants and
brute force over every Kraft-feasible length vector."""
import itertools
import math

import numpy as np
import pytest

import oracle


def _model(lo, step, bits):
    return oracle.Model(1, 1, bits, np.zeros(1), np.eye(1), np.ones(1), lo, step, "f64")


def test_quantizer_hand_values_ties_and_clamps():
    m = _model(0.0, 1.0, 3)               # levels 0..7
    y = np.array([0.0, 0.49, 0.5, 1.5, 2.5, 3.5, 6.5, 7.0, 7.49, 7.5, 9.0, -0.5, -3.0, 2.51])
    want = [0, 0, 0, 2, 2, 4, 6, 7, 7, 7, 7, 0, 0, 3]     # halves go to the even level
    assert oracle.quantize(m, y).tolist() == want
    m = _model(-1.0, 0.25, 4)
    assert oracle.quantize(m, np.array([-1.0, 2.75, -0.875, -0.625])).tolist() == [0, 15, 0, 2]
    q, u = oracle.quantize(m, np.array([-0.9, 0.0]), with_units=True)
    assert np.allclose(u, [0.4, 4.0])


def test_quantizer_idempotent_on_levels():
    m = _model(-2.3, 0.37, 5)
    levels = m.lo + np.arange(32) * m.step
    assert oracle.quantize(m, levels).tolist() == list(range(32))


def test_high_rate_mse_and_step_rate_relation():
    # Appendix D: for a unit Gaussian and rate R >= 2 the step obeys step * 2^R ~= 4.2184
    # (fitted in the paper); high-rate theory gives sqrt(2 pi e) = 4.1327, and the quantiser
    # noise is step^2 / 12.
    rng = np.random.default_rng(7)
    y = rng.standard_normal(2_000_000)
    theory = math.sqrt(2 * math.pi * math.e)
    gaps = []
    for step in (0.5, 0.25, 0.125):
        m = _model(-127.5 * step, step, 8)
        q = oracle.quantize(m, y)
        hist = oracle.histogram(q[:, None], 8, False)
        rate = oracle.entropy(hist[0])
        assert rate >= 2.0
        prod = step * 2.0 ** rate
        assert prod == pytest.approx(theory, rel=0.015)
        assert prod == pytest.approx(4.2184, rel=0.03)
        gaps.append(abs(prod - theory))
        err = y - (m.lo + q * m.step)
        assert np.mean(err ** 2) == pytest.approx(step ** 2 / 12, rel=0.01)
    assert gaps[0] > gaps[1] > gaps[2]          # the finer the step, the closer to theory


def test_entropy_closed_forms():
    assert oracle.entropy(np.array([5, 5, 5, 5])) == pytest.approx(2.0)
    assert oracle.entropy(np.array([8, 4, 2, 2])) == pytest.approx(1.75)
    assert oracle.entropy(np.array([9, 0, 0, 0])) == 0.0
    assert oracle.mean_length(np.array([8, 4, 2, 2]), np.array([1, 2, 3, 3])) == pytest.approx(1.75)


def test_histogram_groups():
    q = np.array([[0, 1], [0, 3], [2, 3]], dtype=np.uint8)
    assert oracle.histogram(q, 2, False).tolist() == [[2, 1, 1, 2]]
    assert oracle.histogram(q, 2, True).tolist() == [[2, 0, 1, 0], [0, 1, 0, 2]]


def _kraft(lengths, lmax):
    return sum(1 << (lmax - int(l)) for l in lengths)


def _brute_force_cost(w, lmax):
    best = None
    for ls in itertools.product(range(1, lmax + 1), repeat=len(w)):
        if _kraft(ls, lmax) <= (1 << lmax):
            cost = sum(a * b for a, b in zip(w, ls))
            best = cost if best is None else min(best, cost)
    return best


@pytest.mark.parametrize("seed", range(12))
def test_huffman_optimal_by_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 7))
    w = rng.integers(1, 40, n).tolist()
    if seed % 3 == 0:
        w = sorted(w)
        w[-1] = sum(w) * 3          # very skewed: a deep tree
    ln = oracle.huffman_lengths_raw(w, lmax=n)
    assert _kraft(ln, 8) == 1 << 8                              # Kraft equality
    assert sum(a * int(b) for a, b in zip(w, ln)) == _brute_force_cost(w, n)


@pytest.mark.parametrize("seed", range(10))
def test_length_limited_optimal_by_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(3, 7))
    w = [int(2 ** i * rng.integers(1, 3)) for i in range(n)]    # forces deep plain trees
    lmax = max(2, math.ceil(math.log2(n))) + int(seed % 2)
    ln = oracle.huffman_lengths_raw(w, lmax=lmax, force_limited=True)
    assert max(ln) <= lmax
    assert _kraft(ln, lmax) == 1 << lmax
    assert sum(a * int(b) for a, b in zip(w, ln)) == _brute_force_cost(w, lmax)


def test_limited_equals_plain_when_limit_is_loose():
    rng = np.random.default_rng(5)
    for _ in range(20):
        w = rng.integers(1, 1000, 16).tolist()
        a = oracle.huffman_lengths_raw(w, lmax=31)
        b = oracle.huffman_lengths_raw(w, lmax=15, force_limited=True)
        assert sum(x * int(y) for x, y in zip(w, a)) == sum(x * int(y) for x, y in zip(w, b))


def test_huffman_dyadic_and_uniform():
    # dyadic probabilities: lengths are exactly -log2 p
    assert oracle.huffman_lengths_raw([8, 4, 2, 1, 1]).tolist() == [1, 2, 3, 4, 4]
    assert oracle.huffman_lengths_raw([3] * 16).tolist() == [4] * 16
    # the public entry adds one to every count (all symbols get a code)
    assert oracle.huffman_lengths(np.array([7, 3, 1, 0]), 12).tolist() == [[1, 2, 3, 3]]
    assert oracle.huffman_lengths(np.zeros(8, dtype=np.uint64), 12).tolist() == [[3] * 8]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_huffman_rate_bound_and_length_limit(bits):
    # H <= L < H + 1 on the distribution the code was built from (Section 3.1).
    rng = np.random.default_rng(bits)
    n = 1 << bits
    counts = np.floor(1e6 * np.exp(-0.5 * ((np.arange(n) - n / 3) / (n / 10)) ** 2)).astype(np.uint64)
    ln = oracle.huffman_lengths(counts, 31)[0]
    smoothed = counts + 1
    h = oracle.entropy(smoothed)
    l = oracle.mean_length(smoothed, ln)
    assert h <= l < h + 1
    assert _kraft(ln, 32) == 1 << 32
    lim = oracle.huffman_lengths(counts, 12)[0]
    assert max(lim) <= 12 and _kraft(lim, 12) == 1 << 12
    assert oracle.mean_length(smoothed, lim) >= l - 1e-12
    if max(ln) <= 12:
        assert lim.tolist() == ln.tolist()


def test_huffman_tie_break_is_deterministic():
    # equal weights: leaves before internal nodes, lower symbols first
    assert oracle.huffman_lengths_raw([1, 1, 1]).tolist() == [2, 2, 1]
    assert oracle.huffman_lengths_raw([1, 1, 1, 1, 1]).tolist() == [3, 3, 2, 2, 2]


def test_canonical_codes_hand_example_and_prefix_freeness():
    # lengths 2 1 3 3 -> order (len, symbol): s1, s0, s2, s3 -> 0, 10, 110, 111
    assert oracle.canonical_codes(np.array([2, 1, 3, 3])).tolist() == [0b10, 0b0, 0b110, 0b111]
    rng = np.random.default_rng(1)
    counts = rng.integers(0, 5000, 64)
    ln = oracle.huffman_lengths(counts, 12)[0]
    code = oracle.canonical_codes(ln)
    words = [format(int(c), "b").zfill(int(l)) for c, l in zip(code, ln)]
    for i, a in enumerate(words):
        for j, b in enumerate(words):
            if i != j:
                assert not b.startswith(a)
    order = sorted(range(64), key=lambda s: (ln[s], s))
    vals = [int(words[s].ljust(12, "0"), 2) for s in order]
    assert vals == sorted(vals)                         # numeric order = (length, symbol) order
    for a, b in zip(order, order[1:]):
        if ln[a] == ln[b]:
            assert code[b] == code[a] + 1               # equal lengths are consecutive
