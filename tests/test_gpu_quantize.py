"""CUDA transform kernel vs the CPU oracle, byte for byte (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

COMBOS = [
    (4, 0x1F), (4, 0x15), (4, 0x11), (4, 0x1B), (4, 0x13),
    (3, 0x3F), (3, 0x35), (3, 0x29), (2, 0x7F), (2, 0x55), (2, 0x6B),
]


def run_gpu(x: np.ndarray, rows, row_len, params, inplace=False, offset=0):
    total = rows * row_len
    buf = torch.zeros(total + offset + 64, dtype=torch.uint8, device="cuda")
    buf[offset:offset + total] = torch.from_numpy(x.reshape(-1)).cuda()
    src = buf[offset:offset + total]
    if inplace:
        dst = src
    else:
        dbuf = torch.full((total + offset + 64,), 0xAA, dtype=torch.uint8, device="cuda")
        dst = dbuf[offset:offset + total]
    sparq.sparq_quantize(src, dst, rows, row_len, params)
    sparq.sparq_check()
    if not inplace:
        # nothing outside the destination range was written
        assert (dbuf[:offset] == 0xAA).all() and (dbuf[offset + total:] == 0xAA).all()
    return dst.cpu().numpy().reshape(x.shape)


@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", [sparq.MODE_BSPARQ, sparq.MODE_VSPARQ])
def test_all_65536_pairs(n, mask, rnd, mode):
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    x = np.stack([a.ravel(), b.ravel()], axis=1).copy()      # 65536 rows of one pair
    want = oracle.transform(x, mode, n, mask, rnd)
    p = sparq.SparqParams(mode, n, mask, rnd)
    got_vec = run_gpu(x, 65536, 2, p)                         # vector path
    assert np.array_equal(got_vec, want)
    got_scalar = run_gpu(x, 65536, 2, p, offset=3)            # unaligned: per-pair path
    assert np.array_equal(got_scalar, want)


@pytest.mark.parametrize("rows,row_len", [(1, 16), (3, 1030), (7, 999), (5, 1), (1, 15), (129, 64),
                                           (2, 4098), (1, 1 << 20), (1000, 577)])
@pytest.mark.parametrize("mode", [sparq.MODE_NONE, sparq.MODE_BSPARQ, sparq.MODE_VSPARQ])
def test_ragged_shapes_and_in_place(rows, row_len, mode):
    x = synth.activations(rows * 31 + row_len, (rows, row_len), 0.5)
    for n, mask, rnd in [(4, 0x1F, 1), (3, 0x3F, 0), (2, 0x7F, 1)]:
        p = sparq.SparqParams(mode, n, mask, rnd)
        want = oracle.transform(x, mode, n, mask, rnd)
        assert np.array_equal(run_gpu(x, rows, row_len, p), want)
        assert np.array_equal(run_gpu(x, rows, row_len, p, inplace=True), want)
        assert np.array_equal(run_gpu(x, rows, row_len, p, offset=1), want)


def test_empty_and_errors():
    p = sparq.SparqParams()
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    sparq.sparq_quantize(z, z, 0, 16, p)
    sparq.sparq_quantize(z, z, 4, 0, p)
    with pytest.raises(sparq.SparqError):
        sparq.sparq_quantize(z, z, 1, 16, sparq.SparqParams(2, 4, 0x0F, 1))
    with pytest.raises(sparq.SparqError):   # partial overlap
        big = torch.zeros(64, dtype=torch.uint8, device="cuda")
        sparq.sparq_quantize(big[:32], big[16:48], 1, 32, p)


@pytest.mark.parametrize("mode", [sparq.MODE_BSPARQ, sparq.MODE_VSPARQ])
def test_full_size_2_30_sampled(mode):
    """The benchmark's launch configuration (2^20 rows of 1024) on 2^30 activations;
    the oracle checks the head, the tail and 64 random 64 KiB windows."""
    rows, row_len = 1 << 20, 1024
    total = rows * row_len
    x = synth.activations(4, (total,), 0.5)
    xd = torch.from_numpy(x).cuda()
    yd = torch.empty_like(xd)
    p = sparq.SparqParams(mode, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
    sparq.sparq_quantize(xd, yd, rows, row_len, p)
    sparq.sparq_check()
    rng = np.random.default_rng(0)
    win = 1 << 16
    starts = [0, total - win] + [int(s) * 1024 for s in rng.integers(0, (total - win) // 1024, 64)]
    for s in starts:
        got = yd[s:s + win].cpu().numpy()
        want = oracle.transform(x[s:s + win].reshape(-1, row_len), mode, 4, 0x1F, 1).reshape(-1)
        assert np.array_equal(got, want), s
    # properties that hold at any size, checked on the whole tensor on the device
    diff = yd.to(torch.int16) - xd.to(torch.int16)
    assert int(diff.max()) <= 8 and int(diff.min()) >= -15   # half a top-window LSB up; the saturating top loses < 16
    assert bool(((xd == 0) == (yd == 0)).all())              # zeros, and only zeros, map to zero
    small = xd < 16
    assert bool((yd[small] == xd[small]).all())              # values below 16 unchanged
