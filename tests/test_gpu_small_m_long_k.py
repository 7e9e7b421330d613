"""Few output tiles and long reductions: the deep 7x7 / 14x14 layers of the ResNet-50 stack
(M = 3136 rows against K up to 4608) and GEMMs with K up to the accepted maximum, where a CTA
runs dozens of reduction steps per tile and the stage ring wraps many times.  Every output
must match the oracle bit for bit, launch after launch, on any stream."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

VS = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
NONE = sparq.SparqParams(sparq.MODE_NONE)
V3 = sparq.SparqParams(sparq.MODE_VSPARQ, 3, 0x3F, 1)


def conv_check(cfg, p, seed, repeats=1, stream=None):
    nb, h, w, c, cout, r, stride = cfg
    pad = r // 2
    x = synth.activations(seed, (nb, h, w, c), 0.5)
    wt = synth.weights(seed, (cout, r, r, c))
    scale, bias = synth.scales(seed, cout), synth.bias(seed, cout)
    inv = synth.inv_out_scale(r * r * c)
    acc = oracle.conv2d_nhwc(x, wt, (stride, stride), (pad, pad), p.mode, p.window_bits, p.placement_mask, p.rounding)
    f, q = oracle.epilogue(acc, scale, bias, True, inv)
    xd, wd = torch.from_numpy(x).cuda(), torch.from_numpy(wt).cuda()
    sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
    for _ in range(repeats):
        a = torch.full(acc.shape, -3, dtype=torch.int32, device="cuda")
        f32 = torch.full(acc.shape, -3.0, dtype=torch.float32, device="cuda")
        u8 = torch.full(acc.shape, 3, dtype=torch.uint8, device="cuda")
        sparq.sparq_conv2d_nhwc_s8(xd, wd, (stride, stride), (pad, pad), p, scale=sd, bias=bd, relu=True, inv_out_scale=inv,
                                   acc_out=a, f32_out=f32, u8_out=u8, stream=stream)
        sparq.sparq_check(stream)
        assert np.array_equal(a.cpu().numpy(), acc)
        assert np.array_equal(u8.cpu().numpy(), q)
        assert np.allclose(f32.cpu().numpy(), f, rtol=1e-6, atol=1e-6)
        # bytes only: the straight-line epilogue
        u8.fill_(3)
        sparq.sparq_conv2d_nhwc_s8(xd, wd, (stride, stride), (pad, pad), p, scale=sd, bias=bd, relu=True, inv_out_scale=inv,
                                   u8_out=u8, stream=stream)
        sparq.sparq_check(stream)
        assert np.array_equal(u8.cpu().numpy(), q)


@pytest.mark.parametrize("cfg", [
    (64, 7, 7, 512, 512, 3, 1),       # 25 x 2 tiles, 36 reduction steps
    (64, 14, 14, 512, 512, 3, 2),     # the same GEMM shape through the strided im2col loader
    (64, 7, 7, 2048, 512, 1, 1),      # 1x1: the GEMM view, 16 steps
    (16, 7, 7, 512, 512, 3, 1),       # 7 row tiles, the last one ragged
    (9, 14, 14, 256, 320, 3, 2),      # column count not a multiple of the tile width
])
@pytest.mark.parametrize("p", [VS, NONE, V3])
def test_small_m_long_k_convolutions_exact(cfg, p):
    conv_check(cfg, p, seed=sum(cfg), repeats=2)


@pytest.mark.parametrize("shape", [(256, 256, 65536), (300, 200, 4096), (128, 512, 8192), (1000, 128, 16384)])
@pytest.mark.parametrize("p", [VS, NONE])
def test_long_reduction_gemms_exact(shape, p):
    M, N, K = shape
    A = synth.activations(M + K, (M, K), 0.5)
    B = synth.weights(N + K, (K, N))
    scale, bias = synth.scales(N, N), synth.bias(N, N)
    inv = synth.inv_out_scale(K)
    acc = oracle.gemm(A, B, p.mode, p.window_bits, p.placement_mask, p.rounding)
    f, q = oracle.epilogue(acc, scale, bias, False, inv)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
    for _ in range(3):
        a = torch.full((M, N), -3, dtype=torch.int32, device="cuda")
        f32 = torch.full((M, N), -3.0, dtype=torch.float32, device="cuda")
        u8 = torch.full((M, N), 3, dtype=torch.uint8, device="cuda")
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, inv_out_scale=inv, acc_out=a, f32_out=f32, u8_out=u8)
        sparq.sparq_check()
        assert np.array_equal(a.cpu().numpy(), acc)
        assert np.array_equal(u8.cpu().numpy(), q)
        assert np.allclose(f32.cpu().numpy(), f, rtol=1e-6, atol=1e-6)


def test_accumulator_extremes_on_256_columns():
    K = 65536
    A = np.full((128, K), 255, dtype=np.uint8)
    B = np.full((K, 256), -128, dtype=np.int8)
    B[:, 1] = 127
    acc = torch.zeros((128, 256), dtype=torch.int32, device="cuda")
    sparq.sparq_gemm_s8(torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda(), NONE, acc_out=acc)
    sparq.sparq_check()
    got = acc.cpu().numpy()
    assert (got[:, 0] == K * 255 * -128).all() and (got[:, 1] == K * 255 * 127).all()


def test_launches_on_two_streams():
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for st in (s1, s2, s1):
        with torch.cuda.stream(st):
            conv_check((16, 7, 7, 512, 512, 3, 1), VS, seed=77, stream=st)
    torch.cuda.synchronize()
