"""Residual input of the epilogue: the u8 identity tensor of a residual block, on its own
scale, is added before the ReLU, so the last convolution of a bottleneck writes the block's
output in one pass.  The paper's transform acts on whatever activations a layer receives
(Section 3); this only completes the requantization path between layers."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

VS = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("shape", [(300, 64, 192), (1000, 200, 128), (129, 512, 64), (257, 36, 80)])
@pytest.mark.parametrize("relu", [False, True])
@pytest.mark.parametrize("params", [VS, sparq.SparqParams(sparq.MODE_NONE)])
def test_gemm_residual(shape, relu, params):
    M, N, K = shape
    A = synth.activations(M, (M, K), 0.5)
    B = synth.weights(N, (K, N))
    scale, bias = synth.scales(K, N), synth.bias(K, N)
    res = synth.activations(7 + M, (M, N), 0.3)
    rs = 0.21
    inv = synth.inv_out_scale(K)
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    f32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    sparq.sparq_gemm_s8(dev(A), dev(B.T), params, scale=dev(scale), bias=dev(bias), relu=relu,
                        inv_out_scale=inv, f32_out=f32, u8_out=u8, residual=dev(res), residual_scale=rs)
    sparq.sparq_check()
    acc = oracle.gemm(A, B, params.mode, params.window_bits, params.placement_mask, params.rounding)
    wf, wq = oracle.epilogue(acc, scale, bias, relu, inv, residual=res, residual_scale=rs)
    np.testing.assert_allclose(f32.cpu().numpy(), wf, rtol=1e-6, atol=1e-6)
    assert np.array_equal(u8.cpu().numpy(), wq)
    # u8 alone (the ReLU is then folded into the clamp) must give the same bytes
    u8b = torch.zeros_like(u8)
    sparq.sparq_gemm_s8(dev(A), dev(B.T), params, scale=dev(scale), bias=dev(bias), relu=relu,
                        inv_out_scale=inv, u8_out=u8b, residual=dev(res), residual_scale=rs)
    sparq.sparq_check()
    assert np.array_equal(u8b.cpu().numpy(), wq)


def test_bottleneck_block_with_identity():
    # 1x1 -> 3x3 -> 1x1 (+ identity) -> ReLU, u8 between the layers, vSPARQ in every consumer
    nb, hw, cin, mid = 4, 28, 256, 64
    x = synth.activations(900, (nb, hw, hw, cin), 0.5)
    w1 = synth.weights(901, (mid, 1, 1, cin))
    w2 = synth.weights(902, (mid, 3, 3, mid))
    w3 = synth.weights(903, (cin, 1, 1, mid))
    layers = [(w1, 0, cin), (w2, 1, 9 * mid), (w3, 0, mid)]
    cur_g, cur_o = dev(x), x
    rs = 0.5
    for i, (w, pad, k) in enumerate(layers):
        cout = w.shape[0]
        scale, bias = synth.scales(910 + i, cout), synth.bias(910 + i, cout)
        inv = synth.inv_out_scale(k)
        out = torch.zeros((nb, hw, hw, cout), dtype=torch.uint8, device="cuda")
        last = i == 2
        sparq.sparq_conv2d_nhwc_s8(cur_g, dev(w), (1, 1), (pad, pad), VS, scale=dev(scale), bias=dev(bias),
                                   relu=True, inv_out_scale=inv, u8_out=out,
                                   residual=dev(x) if last else None, residual_scale=rs if last else 0.0)
        acc = oracle.conv2d_nhwc(cur_o, w, (1, 1), (pad, pad), VS.mode, VS.window_bits, VS.placement_mask, VS.rounding)
        _, q = oracle.epilogue(acc, scale, bias, True, inv, residual=x if last else None,
                               residual_scale=rs if last else 0.0)
        sparq.sparq_check()
        assert np.array_equal(out.cpu().numpy(), q), i
        cur_g, cur_o = out, q
    assert (cur_o > 0).mean() > 0.2      # the block's output is not degenerate


def test_window_conv_residual_and_next_transform():
    # stride-1 3x3 (window kernel) with residual, ReLU and the producer-side transform
    nb, hw, c = 2, 56, 64
    x = synth.activations(920, (nb, hw, hw, c), 0.45)
    w = synth.weights(921, (c, 3, 3, c))
    res = synth.activations(922, (nb, hw, hw, c), 0.2)
    scale, bias = synth.scales(923, c), synth.bias(923, c)
    inv = synth.inv_out_scale(9 * c)
    out = torch.zeros((nb, hw, hw, c), dtype=torch.uint8, device="cuda")
    sparq.sparq_conv2d_nhwc_s8(dev(x), dev(w), (1, 1), (1, 1), VS, scale=dev(scale), bias=dev(bias), relu=True,
                               inv_out_scale=inv, u8_out=out, residual=dev(res), residual_scale=0.125,
                               next_transform=VS)
    sparq.sparq_check()
    acc = oracle.conv2d_nhwc(x, w, (1, 1), (1, 1), VS.mode, VS.window_bits, VS.placement_mask, VS.rounding)
    _, q = oracle.epilogue(acc, scale, bias, True, inv, residual=res, residual_scale=0.125)
    want = oracle.transform(q, VS.mode, VS.window_bits, VS.placement_mask, VS.rounding)
    assert np.array_equal(out.cpu().numpy(), want)


def test_host_form_residual():
    M, N, K = 260, 96, 128
    A = synth.activations(930, (M, K), 0.5)
    B = synth.weights(931, (K, N))
    scale = synth.scales(932, N)
    res = synth.activations(933, (M, N), 0.3)
    inv = synth.inv_out_scale(K)
    u8 = torch.zeros((M, N), dtype=torch.uint8).pin_memory()
    sparq.sparq_gemm_s8_host(torch.from_numpy(A).pin_memory(), dev(B.T), VS, scale=dev(scale), relu=True,
                             inv_out_scale=inv, u8_out=u8, residual=torch.from_numpy(res).pin_memory(),
                             residual_scale=0.3)
    acc = oracle.gemm(A, B, VS.mode, VS.window_bits, VS.placement_mask, VS.rounding)
    _, q = oracle.epilogue(acc, scale, None, True, inv, residual=res, residual_scale=0.3)
    assert np.array_equal(u8.numpy(), q)


def test_residual_rejected():
    A = torch.zeros((128, 64), dtype=torch.uint8, device="cuda")
    B = torch.zeros((64, 64), dtype=torch.int8, device="cuda")
    acc = torch.zeros((128, 64), dtype=torch.int32, device="cuda")
    res = torch.zeros((128 * 64 + 16,), dtype=torch.uint8, device="cuda")
    sc = torch.ones(64, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:      # no dequantized output to add it to
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), acc_out=acc, residual=res, residual_scale=1.0)
    assert ei.value.code == -1
    u8 = torch.zeros((128, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:      # misaligned residual
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), scale=sc, u8_out=u8, residual=res[1:], residual_scale=1.0)
    assert ei.value.code == -2
