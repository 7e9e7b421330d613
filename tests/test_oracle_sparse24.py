"""Pins for the oracle's sparse-tensor-core variant (Section 4 "Sparse TC" and Section 5.3):
2:4-compressed weights select two activations per group of four, and SPARQ's pair is that
selected pair.  Pinned by special cases that reduce to the dense oracle (already pinned
elsewhere), and by a brute-force restatement in Python on tiny shapes."""
import numpy as np
import pytest

import oracle
import sparq_synth as synth

P = dict(n=4, mask=0x1F, rnd=1)


def test_generator_is_2_of_4():
    vals, pos = synth.sparse24_weights(1, 8, 64)
    assert vals.shape == (8, 32) and pos.shape == (8, 32)
    p = pos.reshape(8, 16, 2)
    assert (p[..., 0] < p[..., 1]).all() and p.max() <= 3
    dense = synth.sparse24_dense(vals, pos)
    assert ((dense.reshape(8, 16, 4) != 0).sum(axis=2) <= 2).all()
    assert len({tuple(t) for t in p.reshape(-1, 2)}) == 6          # all six patterns occur


@pytest.mark.parametrize("mode", [0, 1])
def test_elementwise_modes_reduce_to_the_dense_product(mode):
    # without the pair rule the transform is per element and commutes with the selection
    A = synth.activations(2, (33, 64), 0.5)
    vals, pos = synth.sparse24_weights(3, 10, 64)
    dense = synth.sparse24_dense(vals, pos)
    got = oracle.gemm_sparse24(A, vals, pos, mode, **P)
    want = oracle.gemm(A, np.ascontiguousarray(dense.T), mode, **P)
    assert np.array_equal(got, want)


def test_aligned_patterns_reduce_to_dense_vsparq():
    # coordinates (0,1) or (2,3) select exactly a pair (2j, 2j+1) of the dense pairing
    A = synth.activations(4, (17, 48), 0.5)
    vals = synth.weights(5, (6, 24))
    rng = np.random.default_rng(0)
    pick = rng.integers(0, 2, size=(6, 12))
    pos = np.where(pick[..., None] == 0, np.array([0, 1], np.uint8), np.array([2, 3], np.uint8)).reshape(6, 24)
    dense = synth.sparse24_dense(vals, np.ascontiguousarray(pos))
    got = oracle.gemm_sparse24(A, vals, np.ascontiguousarray(pos), 2, **P)
    assert np.array_equal(got, oracle.gemm(A, np.ascontiguousarray(dense.T), 2, **P))


@pytest.mark.parametrize("n,mask", [(4, 0x1F), (4, 0x15), (3, 0x3F), (2, 0x7F)])
@pytest.mark.parametrize("rnd", [0, 1])
def test_brute_force_python(n, mask, rnd):
    A = synth.activations(6 + n, (5, 16), 0.5)
    vals, pos = synth.sparse24_weights(7, 4, 16)
    got = oracle.gemm_sparse24(A, vals, pos, 2, n, mask, rnd)
    for m in range(5):
        for j in range(4):
            s = 0
            for g in range(4):
                a, b = int(A[m, 4 * g + pos[j, 2 * g]]), int(A[m, 4 * g + pos[j, 2 * g + 1]])
                qa, qb = oracle.vsparq_pair(a, b, n, mask, rnd)
                s += qa * int(vals[j, 2 * g]) + qb * int(vals[j, 2 * g + 1])
            assert got[m, j] == s


def test_the_pair_depends_on_the_output_channel():
    # activations (200, 0, 0, 90): with coordinates (0,1) the 200 is a lone value and stays
    # exact; with (0,3) it is paired with 90 and both are trimmed to 4 bits (208, 88)
    A = np.array([[200, 0, 0, 90]], dtype=np.uint8)
    vals = np.array([[1, 1], [1, 1]], dtype=np.int8)
    pos = np.array([[0, 1], [0, 3]], dtype=np.uint8)
    got = oracle.gemm_sparse24(A, vals, pos, 2, **P)
    assert list(got[0]) == [200, 208 + 88]


def test_rejects_bad_coordinates():
    A = np.zeros((1, 4), np.uint8)
    with pytest.raises(ValueError):
        oracle.gemm_sparse24(A, np.ones((1, 2), np.int8), np.array([[2, 1]], np.uint8), 2, **P)
