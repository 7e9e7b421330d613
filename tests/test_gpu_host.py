"""Host-buffer entry points on problems large enough to be cut into chunks (copy in, kernel
and copy out of neighbouring chunks overlap): every output must equal what the device-pointer
entry point writes for the whole problem at once."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

VS = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def pinned(a):
    return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()


def test_conv_host_chunked_equals_device():
    nb, hw, c, cout = 19, 28, 128, 128          # 19 images: chunks of 5, 5, 5, 4
    x = synth.activations(940, (nb, hw, hw, c), 0.45)
    w = synth.weights(941, (cout, 3, 3, c))
    scale, bias = synth.scales(942, cout), synth.bias(942, cout)
    res = synth.activations(943, (nb, hw, hw, cout), 0.3)
    inv = synth.inv_out_scale(9 * c)
    shape = (nb, hw, hw, cout)
    d = {"acc": torch.empty(shape, dtype=torch.int32, device="cuda"),
         "f32": torch.empty(shape, dtype=torch.float32, device="cuda"),
         "u8": torch.empty(shape, dtype=torch.uint8, device="cuda")}
    sparq.sparq_conv2d_nhwc_s8(dev(x), dev(w), (1, 1), (1, 1), VS, scale=dev(scale), bias=dev(bias), relu=True,
                               inv_out_scale=inv, acc_out=d["acc"], f32_out=d["f32"], u8_out=d["u8"],
                               residual=dev(res), residual_scale=0.25)
    sparq.sparq_check()
    h = {"acc": torch.zeros(shape, dtype=torch.int32).pin_memory(),
         "f32": torch.zeros(shape, dtype=torch.float32).pin_memory(),
         "u8": torch.zeros(shape, dtype=torch.uint8).pin_memory()}
    for _ in range(2):                          # the second call reuses streams, events and staging buffers
        for t in h.values():
            t.zero_()
        sparq.sparq_conv2d_nhwc_s8_host(pinned(x), dev(w), (1, 1), (1, 1), VS, scale=dev(scale), bias=dev(bias),
                                        relu=True, inv_out_scale=inv, acc_out=h["acc"], f32_out=h["f32"],
                                        u8_out=h["u8"], residual=pinned(res), residual_scale=0.25)
        for k in h:
            assert torch.equal(h[k], d[k].cpu()), k
    # and against the oracle directly
    acc = oracle.conv2d_nhwc(x, w, (1, 1), (1, 1), VS.mode, 4, 0x1F, 1)
    f, q = oracle.epilogue(acc, scale, bias, True, inv, residual=res, residual_scale=0.25)
    assert np.array_equal(h["acc"].numpy(), acc) and np.array_equal(h["u8"].numpy(), q)
    assert np.allclose(h["f32"].numpy(), f, rtol=1e-6, atol=1e-6)


def test_gemm_host_chunked_equals_device():
    M, N, K = 5003, 192, 256                    # chunks of whole 128-row tiles, ragged last chunk
    A = synth.activations(950, (M, K), 0.5)
    B = synth.weights(951, (K, N))
    scale = synth.scales(952, N)
    inv = synth.inv_out_scale(K)
    d_f = torch.empty((M, N), dtype=torch.float32, device="cuda")
    d_q = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    sparq.sparq_gemm_s8(dev(A), dev(B.T), VS, scale=dev(scale), relu=True, inv_out_scale=inv, f32_out=d_f, u8_out=d_q)
    sparq.sparq_check()
    h_f = torch.zeros((M, N), dtype=torch.float32).pin_memory()
    h_q = torch.zeros((M, N), dtype=torch.uint8).pin_memory()
    sparq.sparq_gemm_s8_host(pinned(A), dev(B.T), VS, scale=dev(scale), relu=True, inv_out_scale=inv,
                             f32_out=h_f, u8_out=h_q)
    assert torch.equal(h_f, d_f.cpu())
    assert torch.equal(h_q, d_q.cpu())
    f, q = oracle.epilogue(oracle.gemm(A, B, VS.mode, 4, 0x1F, 1), scale, None, True, inv)
    assert np.array_equal(h_q.numpy(), q) and np.allclose(h_f.numpy(), f, rtol=1e-6, atol=1e-6)


def test_quantize_host_equals_oracle():
    rows, row_len = 3001, 1000
    x = synth.activations(960, (rows, row_len), 0.5)
    out = torch.zeros((rows, row_len), dtype=torch.uint8).pin_memory()
    sparq.sparq_quantize_host(pinned(x), out, rows, row_len, VS)
    assert np.array_equal(out.numpy(), oracle.transform(x, VS.mode, 4, 0x1F, 1))
