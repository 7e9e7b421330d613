"""Pins for the oracle's vSPARQ (Section 3.2, Eq. 1-2): all 65,536 pairs."""
import numpy as np
import pytest

import oracle

CASES = [(4, 0x1F), (4, 0x15), (4, 0x11), (3, 0x3F), (2, 0x7F), (3, 0x29), (2, 0x55)]


def all_pairs():
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    return np.stack([a.ravel(), b.ravel()], axis=1)  # rows are pairs (a, b)


def widest(x, n, rnd):
    """What a lone non-zero keeps: the nearest (or next lower) value with at most
    2n contiguous significant bits -- written from the set definition, not the window walk."""
    wide = 2 * n
    if wide >= 8:
        return x
    R = sorted({m << s for s in range(8 - wide + 1) for m in range(1 << wide) if (m << s) <= 255})
    if rnd == 0:
        return max(r for r in R if r <= x)
    return min(R, key=lambda r: (abs(r - x), -r))


@pytest.mark.parametrize("n,mask", CASES)
@pytest.mark.parametrize("rnd", [0, 1])
def test_all_pairs_follow_eq2(n, mask, rnd):
    pairs = all_pairs()
    got = oracle.transform(pairs, oracle.MODE_VSPARQ, n, mask, rnd).reshape(256, 256, 2)
    b_tab = np.array([oracle.bsparq(x, n, mask, rnd) for x in range(256)], dtype=np.uint8)
    w_tab = np.array([widest(x, n, rnd) for x in range(256)], dtype=np.uint8)
    a = np.arange(256)[:, None]
    b = np.arange(256)[None, :]
    want_a = np.where(b == 0, w_tab[a], b_tab[a]) * np.ones_like(b)
    want_b = np.where(a == 0, w_tab[b], b_tab[b]) * np.ones_like(a)
    assert np.array_equal(got[..., 0], want_a.astype(np.uint8))
    assert np.array_equal(got[..., 1], want_b.astype(np.uint8))
    # zeros stay zero in every case of Eq. 2
    assert (got[0, :, 0] == 0).all() and (got[:, 0, 1] == 0).all()
    if n == 4:
        # a lone non-zero still has all of its 8 bits (Section 1)
        assert np.array_equal(got[:, 0, 0], np.arange(256, dtype=np.uint8))
        assert np.array_equal(got[0, :, 1], np.arange(256, dtype=np.uint8))
    else:
        # total window of 2n bits (Section 5.1): 6 bits for n=3, 4 bits for n=2
        for x in range(1, 256):
            v = int(got[x, 0, 0])
            tz = (v & -v).bit_length() - 1
            assert v.bit_length() - tz <= 2 * n
            assert 2 * abs(v - x) <= (1 << tz) or rnd == 0 or x > 255 - (1 << (8 - 2 * n - 1))


def test_scalar_pair_matches_vector_and_dot_product_form():
    rng = np.random.default_rng(7)
    for _ in range(200):
        a, b = (int(v) for v in rng.integers(0, 256, 2))
        if rng.random() < 0.3:
            a = 0
        if rng.random() < 0.3:
            b = 0
        qa, qb = oracle.vsparq_pair(a, b, 4, 0x1F, 1)
        v = oracle.transform(np.array([[a, b]], dtype=np.uint8), oracle.MODE_VSPARQ, 4, 0x1F, 1)
        assert (qa, qb) == (int(v[0, 0]), int(v[0, 1]))
        # Eq. 2, left-hand side, for an arbitrary weight pair
        w1, w2 = (int(v) for v in rng.integers(-128, 128, 2))
        if b == 0:
            assert qa * w1 + qb * w2 == a * w1
        elif a == 0:
            assert qa * w1 + qb * w2 == b * w2
        else:
            assert qa * w1 + qb * w2 == oracle.bsparq(a, 4, 0x1F, 1) * w1 + oracle.bsparq(b, 4, 0x1F, 1) * w2


def test_pairs_do_not_cross_rows_and_odd_tail():
    # rows of length 3: (x0,x1) is a pair, x2 is paired with an implicit zero.
    x = np.array([[200, 201, 203], [0, 77, 0], [99, 0, 0]], dtype=np.uint8)
    y = oracle.transform(x, oracle.MODE_VSPARQ, 4, 0x1F, 0)
    assert y[0, 0] == oracle.bsparq(200, 4, 0x1F, 0) and y[0, 1] == oracle.bsparq(201, 4, 0x1F, 0)
    assert y[0, 2] == 203           # lone tail keeps 8 bits, although the next row starts with 0/99
    assert list(y[1]) == [0, 77, 0]
    assert list(y[2]) == [99, 0, 0]
