"""Pins for the oracle's bSPARQ (Section 3.1 of the paper).

The oracle walks the window algorithm.  These tests pin it to things that are
not the oracle: the examples the paper prints, a set-based definition written
here from scratch ("nearest member of the set of representable values"), and
the invariants the method promises, all by exhaustive enumeration of the 256
inputs.
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_examples.txt")

NAMED = {  # Section 3.1 (5opt/3opt/2opt) and Section 5.1 / Table 4 (6opt, 7opt)
    "5opt": (4, 0x1F),
    "3opt": (4, 0x15),
    "2opt": (4, 0x11),
    "6opt": (3, 0x3F),
    "7opt": (2, 0x7F),
}


def valid_masks(n):
    """Every placement set that contains shift 0 and the top shift 8-n and leaves
    no gap wider than n (so that no value falls between two windows)."""
    top = 8 - n
    out = []
    for bits in range(1 << (top + 1)):
        if not (bits & 1) or not (bits >> top) & 1:
            continue
        shifts = [s for s in range(top + 1) if (bits >> s) & 1]
        if all(b - a <= n for a, b in zip(shifts, shifts[1:])):
            out.append(bits)
    return out


def representable_set(n, mask):
    shifts = [s for s in range(8 - n + 1) if (mask >> s) & 1]
    return sorted({m << s for s in shifts for m in range(1 << n) if (m << s) <= 255})


ALL_CASES = [(n, m) for n in (4, 3, 2) for m in valid_masks(n)]


def test_golden_paper_examples():
    rows = 0
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            x, n, mask, rnd, value, window, shift = (int(t, 0) for t in line.split())
            assert oracle.bsparq(x, n, mask, rnd) == value
            assert oracle.bsparq_window(x, n, mask, rnd) == (window, shift)
            rows += 1
    assert rows >= 5


def test_named_sets_are_valid_and_region_counts():
    # Section 3.1: five placements for 4 bits; six and seven regions for 3 and 2 bits.
    for name, (n, mask) in NAMED.items():
        assert mask in valid_masks(n), name
    assert bin(NAMED["5opt"][1]).count("1") == 5
    assert bin(NAMED["6opt"][1]).count("1") == 6
    assert bin(NAMED["7opt"][1]).count("1") == 7
    # the number of distinct shifts actually used over all inputs equals the set size
    for name, (n, mask) in NAMED.items():
        used = {oracle.window_shift(x, n, mask) for x in range(1, 256)}
        assert used == {s for s in range(9 - n) if (mask >> s) & 1}, name


def test_window_follows_leading_one_full_set():
    # Section 3.1 (the window position comes from the leading-zero count): with every placement
    # allowed the window's top bit is the leading one (or the window sits at the bottom for small values).
    for n in (4, 3, 2):
        full = (1 << (9 - n)) - 1
        for x in range(1, 256):
            p = x.bit_length() - 1
            assert oracle.window_shift(x, n, full) == max(0, p - n + 1)


@pytest.mark.parametrize("n,mask", ALL_CASES)
def test_truncate_is_largest_representable_not_above(n, mask):
    R = representable_set(n, mask)
    for x in range(256):
        want = max(r for r in R if r <= x)
        assert oracle.bsparq(x, n, mask, 0) == want, (x, n, hex(mask))


@pytest.mark.parametrize("n,mask", ALL_CASES)
def test_round_is_nearest_representable_ties_up(n, mask):
    R = representable_set(n, mask)
    for x in range(256):
        best = min(R, key=lambda r: (abs(r - x), -r))  # ties resolved upwards
        assert oracle.bsparq(x, n, mask, 1) == best, (x, n, hex(mask))


@pytest.mark.parametrize("n,mask", ALL_CASES)
@pytest.mark.parametrize("rnd", [0, 1])
def test_invariants(n, mask, rnd):
    q = [oracle.bsparq(x, n, mask, rnd) for x in range(256)]
    top_sat = ((1 << n) - 1) << (8 - n)
    assert q[0] == 0                                        # zeros preserved
    for x in range(1, 256):
        v = q[x]
        assert 0 < v <= 255
        # at most n contiguous significant bits, at an allowed placement
        tz = (v & -v).bit_length() - 1
        assert v.bit_length() - tz <= n
        assert any((mask >> s) & 1 and (v >> s) < (1 << n) and v % (1 << s) == 0
                   for s in range(9 - n))
        if x < (1 << n):
            assert v == x                                   # small values unchanged
        s = oracle.window_shift(x, n, mask)
        if rnd == 0:
            assert v <= x and x - v < (1 << s)              # trim error below one window LSB
        else:
            if x + ((1 << s) >> 1) > 255 and s == 8 - n:
                assert v == top_sat                         # top of range saturates
                assert abs(v - x) < (1 << s)
            else:
                assert 2 * abs(v - x) <= (1 << s)           # error <= half the window LSB
        assert oracle.bsparq(v, n, mask, rnd) == v          # idempotent
    assert all(a <= b for a, b in zip(q, q[1:]))            # monotone


def test_values_below_16_unchanged_and_fourbit_budget():
    for mask in valid_masks(4):
        for rnd in (0, 1):
            for x in range(16):
                assert oracle.bsparq(x, 4, mask, rnd) == x


def test_noise_ordering():
    # Rounding lowers the noise of trimming, and more placements lower it further
    # (Section 3.1, Figure 1 caption; Section 5.1 observations (1) and (2)).
    def mse(n, mask, rnd):
        return np.mean([(oracle.bsparq(x, n, mask, rnd) - x) ** 2 for x in range(256)])
    for n, mask in ALL_CASES:
        assert mse(n, mask, 1) <= mse(n, mask, 0)
    for rnd in (0, 1):
        assert mse(4, 0x1F, rnd) <= mse(4, 0x15, rnd) <= mse(4, 0x11, rnd)
        assert mse(4, 0x1F, rnd) <= mse(3, 0x3F, rnd) <= mse(2, 0x7F, rnd)


def test_identity_width_and_invalid_set():
    for x in range(256):
        assert oracle.bsparq(x, 8, 0x1, 1) == x
    # a set without the top placement cannot hold large values
    assert oracle.window_shift(200, 4, 0x03) == -1


def test_eq3_two_nibble_products():
    # Eq. 3: x*w == 2^4 * x[7:4]*w + x[3:0]*w for every 8-bit x and signed 8-bit w.
    x = np.arange(256, dtype=np.int64)[:, None]
    w = np.arange(-128, 128, dtype=np.int64)[None, :]
    assert np.array_equal(x * w, ((x >> 4) * w << 4) + (x & 15) * w)


def test_eq4_value_is_window_times_power_of_two():
    # Eq. 4: each operand is a 4-bit value times 2^opt with opt from the placement set.
    for name, (n, mask) in NAMED.items():
        for rnd in (0, 1):
            for x in range(256):
                win, s = oracle.bsparq_window(x, n, mask, rnd)
                assert win < (1 << n) and (mask >> s) & 1
                assert win << s == oracle.bsparq(x, n, mask, rnd)


def test_transform_vector_matches_scalar():
    x = np.arange(256, dtype=np.uint8)
    for (n, mask), rnd in itertools.product(ALL_CASES[::7], (0, 1)):
        got = oracle.transform(x, oracle.MODE_BSPARQ, n, mask, rnd)
        want = np.array([oracle.bsparq(int(v), n, mask, rnd) for v in x], dtype=np.uint8)
        assert np.array_equal(got, want)
    assert np.array_equal(oracle.transform(x, oracle.MODE_NONE, 4, 0x1F, 1), x)
