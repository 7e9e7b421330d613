"""Packed stream (Eq. 4's two 4-bit inputs per pair plus the pair's ShiftCtrl / MuxCtrl
state, Sections 3.1 and 5.1): the CUDA codec against the oracle, byte for byte."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

MASKS = [0x1F, 0x15, 0x11, 0x1B, 0x17]


def run(x, params):
    cb = sparq.sparq_packed_ctrl_bits(params)
    xg = torch.from_numpy(x).cuda()
    data = torch.zeros(x.size // 2, dtype=torch.uint8, device="cuda")
    ctrl = torch.zeros(x.size // 16 * cb, dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(xg)
    sparq.sparq_pack(xg, params, data, ctrl)
    sparq.sparq_unpack(data, ctrl, params, out)
    sparq.sparq_check()
    return cb, data.cpu().numpy(), ctrl.cpu().numpy(), out.cpu().numpy()


@pytest.mark.parametrize("mask", MASKS)
@pytest.mark.parametrize("mode", [sparq.MODE_BSPARQ, sparq.MODE_VSPARQ])
@pytest.mark.parametrize("rnd", [0, 1])
def test_every_pair(mask, mode, rnd):
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    x = np.ascontiguousarray(np.stack([a.ravel(), b.ravel()], axis=1).reshape(-1, 64))
    p = sparq.SparqParams(mode, 4, mask, rnd)
    cb, data, ctrl, out = run(x, p)
    assert cb == oracle.pack_ctrl_bits(mode, mask)
    wd, wc = oracle.pack(x, mode, mask, rnd)
    assert np.array_equal(data, wd)
    assert np.array_equal(ctrl, wc)
    assert np.array_equal(out, oracle.transform(x, mode, 4, mask, rnd))


@pytest.mark.parametrize("shape", [(1, 16), (3, 48), (1025, 16), (777, 1024 + 16), (4096 + 3, 4096)])
def test_shapes_with_ragged_tiles(shape):
    # tiles are 1024 units of 16 activations: one unit, a partial tile, a tile plus one unit,
    # several tiles with a tail that is not a multiple of four control bytes
    x = synth.activations(40 + shape[0], shape, 0.5)
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
    _, data, ctrl, out = run(x, p)
    wd, wc = oracle.pack(x, p.mode, p.placement_mask, p.rounding)
    assert np.array_equal(data, wd)
    assert np.array_equal(ctrl, wc)
    assert np.array_equal(out, oracle.transform(x, p.mode, 4, p.placement_mask, p.rounding))


def test_unpacked_stream_feeds_a_plain_gemm():
    # consumer with mode NONE on the unpacked tensor == fused vSPARQ GEMM on the raw one
    M, N, K = 512, 96, 256
    A = synth.activations(60, (M, K), 0.5)
    B = synth.weights(61, (K, N))
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x15, 1)
    _, _, _, out = run(A, p)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    sparq.sparq_gemm_s8(torch.from_numpy(out).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda(),
                        sparq.SparqParams(sparq.MODE_NONE), acc_out=acc)
    sparq.sparq_check()
    assert np.array_equal(acc.cpu().numpy(), oracle.gemm(A, B, p.mode, 4, p.placement_mask, p.rounding))


def test_empty_and_rejected():
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
    e = torch.zeros((0, 64), dtype=torch.uint8, device="cuda")
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    sparq.sparq_pack(e, p, z, z)                                   # no-op
    x = torch.zeros((2, 24), dtype=torch.uint8, device="cuda")
    big = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:                     # row_len not a multiple of 16
        sparq.sparq_pack(x, p, big, big)
    assert ei.value.code == -2
    assert sparq.sparq_packed_ctrl_bits(sparq.SparqParams(sparq.MODE_VSPARQ, 3, 0x3F, 1)) == 6
    with pytest.raises(sparq.SparqError) as ei:                     # nothing to pack without SPARQ
        sparq.sparq_packed_ctrl_bits(sparq.SparqParams(sparq.MODE_NONE))
    assert ei.value.code == -1
    x = torch.zeros((2, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:                     # misaligned plane
        sparq.sparq_pack(x, p, big[1:], big)
    assert ei.value.code == -2


# ---- 3- and 2-bit windows (Section 5.1) -------------------------------------------------------

NARROW = [(3, 0x3F), (3, 0x35), (3, 0x29), (2, 0x7F), (2, 0x55), (2, 0x6B)]


def run_n(x, params):
    n = params.window_bits
    cb = sparq.sparq_packed_ctrl_bits(params)
    xg = torch.from_numpy(x).cuda()
    data = torch.full((x.size // 16 * 2 * n + 16,), 0xAA, dtype=torch.uint8, device="cuda")
    ctrl = torch.full((x.size // 16 * cb + 16,), 0xAA, dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(xg)
    sparq.sparq_pack(xg, params, data, ctrl)
    sparq.sparq_unpack(data, ctrl, params, out)
    sparq.sparq_check()
    nd, nc = x.size // 16 * 2 * n, x.size // 16 * cb
    assert (data[nd:] == 0xAA).all() and (ctrl[nc:] == 0xAA).all()      # nothing written past the planes
    return cb, data[:nd].cpu().numpy(), ctrl[:nc].cpu().numpy(), out.cpu().numpy()


@pytest.mark.parametrize("n,mask", NARROW)
@pytest.mark.parametrize("mode", [sparq.MODE_BSPARQ, sparq.MODE_VSPARQ])
@pytest.mark.parametrize("rnd", [0, 1])
def test_every_pair_narrow_windows(n, mask, mode, rnd):
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    x = np.ascontiguousarray(np.stack([a.ravel(), b.ravel()], axis=1).reshape(-1, 64))
    p = sparq.SparqParams(mode, n, mask, rnd)
    cb, data, ctrl, out = run_n(x, p)
    assert cb == oracle.pack_ctrl_bits_n(mode, n, mask)
    wd, wc = oracle.pack_n(x, mode, n, mask, rnd)
    assert np.array_equal(data, wd)
    assert np.array_equal(ctrl, wc)
    assert np.array_equal(out, oracle.transform(x, mode, n, mask, rnd))


@pytest.mark.parametrize("shape", [(1, 16), (3, 48), (1025, 16), (777, 1024 + 16)])
@pytest.mark.parametrize("n,mask", [(3, 0x3F), (2, 0x7F)])
def test_ragged_shapes_narrow_windows(shape, n, mask):
    x = synth.activations(90 + shape[0] + n, shape, 0.5)
    p = sparq.SparqParams(sparq.MODE_VSPARQ, n, mask, 1)
    _, data, ctrl, out = run_n(x, p)
    wd, wc = oracle.pack_n(x, p.mode, n, mask, 1)
    assert np.array_equal(data, wd) and np.array_equal(ctrl, wc)
    assert np.array_equal(out, oracle.transform(x, p.mode, n, mask, 1))
