"""SPARQ on a 2:4 sparse tensor core (Sections 4 and 5.3): the expansion kernels and the
product over the expanded operands against the oracle's per-channel pair selection."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

PARAMS = [
    sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1),
    sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x15, 0),
    sparq.SparqParams(sparq.MODE_VSPARQ, 3, 0x3F, 1),
    sparq.SparqParams(sparq.MODE_VSPARQ, 2, 0x7F, 1),
    sparq.SparqParams(sparq.MODE_BSPARQ, 4, 0x1F, 1),
    sparq.SparqParams(sparq.MODE_NONE),
]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def expand_weights(vals, pos, p):
    N, half = vals.shape
    kx = sparq.sparq_sparse24_expanded_k(2 * half, p)
    w = torch.full((N, kx), 77, dtype=torch.int8, device="cuda")
    sparq.sparq_sparse24_expand_weights(dev(vals), dev(pos), p, w)
    return w


@pytest.mark.parametrize("p", PARAMS)
@pytest.mark.parametrize("shape", [(300, 64, 192), (129, 40, 64), (1000, 200, 256)])
def test_gemm_matches_the_per_channel_pair_selection(p, shape):
    M, N, K = shape
    A = synth.activations(70 + M, (M, K), 0.5)
    vals, pos = synth.sparse24_weights(71 + N, N, K)
    w = expand_weights(vals, pos, p)
    kx = sparq.sparq_sparse24_expanded_k(K, p)
    assert kx == (3 * K if p.mode == sparq.MODE_VSPARQ else K)
    ws = torch.zeros(M * kx, dtype=torch.uint8, device="cuda")
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    scale, bias = synth.scales(K, N), synth.bias(K, N)
    inv = synth.inv_out_scale(K // 2)
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    sparq.sparq_gemm_s8_sparse24(dev(A), w, p, workspace=ws, scale=dev(scale), bias=dev(bias), relu=True,
                                 inv_out_scale=inv, acc_out=acc, u8_out=u8)
    sparq.sparq_check()
    want = oracle.gemm_sparse24(A, vals, pos, p.mode, p.window_bits, p.placement_mask, p.rounding)
    assert np.array_equal(acc.cpu().numpy(), want)
    _, q = oracle.epilogue(want, scale, bias, True, inv)
    assert np.array_equal(u8.cpu().numpy(), q)


def test_expanded_operands_layout():
    # one group: activations (200, 0, 0, 90); pairs in the order (0,1) (0,2) (0,3) (1,2) (1,3) (2,3)
    p = PARAMS[0]
    A = np.zeros((1, 16), dtype=np.uint8)
    A[0, :4] = [200, 0, 0, 90]
    a_exp = torch.zeros((1, 48), dtype=torch.uint8, device="cuda")
    sparq.sparq_sparse24_expand_activations(dev(A), p, a_exp)
    assert list(a_exp.cpu().numpy()[0, :12]) == [200, 0, 200, 0, 208, 88, 0, 0, 0, 90, 0, 90]
    vals = np.array([[5, -7] + [0] * 6], dtype=np.int8)
    pos = np.array([[1, 3] + [0, 1] * 3], dtype=np.uint8)
    w = expand_weights(vals, pos, p)
    sparq.sparq_check()
    assert list(w.cpu().numpy()[0, :12]) == [0] * 8 + [5, -7, 0, 0]           # pattern (1,3) is the fifth pair
    wd = expand_weights(vals, pos, sparq.SparqParams(sparq.MODE_NONE))
    assert list(wd.cpu().numpy()[0, :4]) == [0, 5, 0, -7]


def test_convolution_on_expanded_channels():
    # 3x3 convolution with 2:4 weights along the input channels: expand both sides along C
    # and run the existing convolution with mode NONE
    p = PARAMS[0]
    nb, hw, c, cout = 2, 14, 64, 32
    x = synth.activations(80, (nb, hw, hw, c), 0.5)
    vals, pos = synth.sparse24_weights(81, cout, 9 * c)
    x_exp = torch.zeros((nb, hw, hw, 3 * c), dtype=torch.uint8, device="cuda")
    sparq.sparq_sparse24_expand_activations(dev(x), p, x_exp)
    w_exp = expand_weights(vals, pos, p).view(cout, 3, 3, 3 * c)
    acc = torch.zeros((nb, hw, hw, cout), dtype=torch.int32, device="cuda")
    sparq.sparq_conv2d_nhwc_s8(x_exp, w_exp, (1, 1), (1, 1), sparq.SparqParams(sparq.MODE_NONE), acc_out=acc)
    sparq.sparq_check()
    # oracle: explicit im2col rows (K order r, s, c) against the compressed weights
    xp = np.zeros((nb, hw + 2, hw + 2, c), dtype=np.uint8)
    xp[:, 1:-1, 1:-1] = x
    cols = np.stack([xp[:, r:r + hw, s:s + hw] for r in range(3) for s in range(3)], axis=3).reshape(-1, 9 * c)
    want = oracle.gemm_sparse24(cols, vals, pos, p.mode, p.window_bits, p.placement_mask, p.rounding)
    assert np.array_equal(acc.cpu().numpy().reshape(-1, cout), want)


def test_bad_coordinates_are_reported():
    p = PARAMS[0]
    vals = np.ones((1, 8), dtype=np.int8)
    pos = np.array([[0, 1, 2, 1, 0, 4, 1, 1]], dtype=np.uint8)       # groups 1, 2 and 3 are invalid
    w = expand_weights(vals, pos, p)
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_check()
    assert ei.value.code == -1
    got = w.cpu().numpy()[0]
    assert list(got[:2]) == [1, 1] and not got[2:].any()
    sparq.sparq_check()                                                # the record is cleared
    with pytest.raises(sparq.SparqError):
        sparq.sparq_sparse24_expanded_k(6, p)
