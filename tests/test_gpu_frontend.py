"""Uniform min-max quantization front end (Section 5 of the paper) against the oracle:
the running absmax, the u8 activations and the per-kernel s8 weights, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu


def acts(seed, n, scale=6.0):
    rng = np.random.default_rng(seed)
    x = np.maximum(rng.standard_normal(n) * scale, -1.0).astype(np.float32)   # mostly post-ReLU like, some negatives
    if n > 8:
        x[3] = np.nan
        x[7] = -0.0
    return x


@pytest.mark.parametrize("n", [1, 3, 4, 1024, 4099, (1 << 20) + 5])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_absmax_and_activation_quantize(n, dtype):
    x = acts(n, n)
    if dtype == "bf16":
        xt = torch.from_numpy(x).to(torch.bfloat16)
        xo = xt.view(torch.int16).numpy().view(np.uint16)        # the oracle takes bf16 bit patterns
        xg = xt.cuda()
    else:
        xo, xg = x, torch.from_numpy(x).cuda()
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    sparq.sparq_absmax(xg, mx)
    want_max = oracle.absmax(xo)
    assert float(mx.item()) == want_max
    out = torch.zeros(n, dtype=torch.uint8, device="cuda")
    sparq.sparq_quantize_act_u8(xg, mx, out)
    sparq.sparq_check()
    assert np.array_equal(out.cpu().numpy(), oracle.quantize_act(xo, want_max))


def test_absmax_is_a_running_maximum():
    a = torch.from_numpy(acts(1, 5000, 2.0)).cuda()
    b = torch.from_numpy(acts(2, 7000, 9.0)).cuda()
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    sparq.sparq_absmax(a, mx)
    sparq.sparq_absmax(b, mx)
    sparq.sparq_absmax(a, mx)
    want = max(oracle.absmax(a.cpu().numpy()), oracle.absmax(b.cpu().numpy()))
    assert float(mx.item()) == want
    z = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = torch.full((5000,), 9, dtype=torch.uint8, device="cuda")
    sparq.sparq_quantize_act_u8(a, z, out)                        # max 0: everything maps to 0
    assert not out.any()


@pytest.mark.parametrize("shape", [(64, 3, 3, 64), (10, 1, 1, 7), (3, 4097)])
def test_weights_per_kernel(shape):
    rng = np.random.default_rng(5)
    w = (rng.standard_normal(shape) * rng.random((shape[0],) + (1,) * (len(shape) - 1)) * 3).astype(np.float32)
    w[1] = 0.0
    w.reshape(shape[0], -1)[2, 0] = np.nan
    q = torch.zeros(shape, dtype=torch.int8, device="cuda")
    sc = torch.zeros(shape[0], dtype=torch.float32, device="cuda")
    sparq.sparq_quantize_weight_s8(torch.from_numpy(w).cuda(), q, sc)
    sparq.sparq_check()
    wq, ws = oracle.quantize_weight(w)
    assert np.array_equal(q.cpu().numpy(), wq)
    assert np.array_equal(sc.cpu().numpy(), ws)


def test_float_layer_through_the_whole_path():
    # fp32 activations and weights -> front end -> fused vSPARQ GEMM with the combined scale,
    # against the same chain in the oracle
    rng = np.random.default_rng(6)
    M, N, K = 384, 64, 256
    x = np.maximum(rng.standard_normal((M, K)), 0).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.1).astype(np.float32)
    xg, wg = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    sparq.sparq_absmax(xg, mx)
    xq = torch.zeros((M, K), dtype=torch.uint8, device="cuda")
    sparq.sparq_quantize_act_u8(xg, mx, xq)
    wq = torch.zeros((N, K), dtype=torch.int8, device="cuda")
    ws = torch.zeros(N, dtype=torch.float32, device="cuda")
    sparq.sparq_quantize_weight_s8(wg, wq, ws)
    scale = (mx / 255.0) * ws                                      # one fp32 division, one multiply
    y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    P = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
    sparq.sparq_gemm_s8(xq, wq, P, scale=scale, f32_out=y)
    sparq.sparq_check()
    omax = oracle.absmax(x)
    oxq = oracle.quantize_act(x, omax)
    owq, ows = oracle.quantize_weight(w)
    oscale = (np.float32(omax) / np.float32(255.0)) * ows
    acc = oracle.gemm(oxq, np.ascontiguousarray(owq.T), P.mode, 4, P.placement_mask, P.rounding)
    want, _ = oracle.epilogue(acc, oscale.astype(np.float32), None, False, 1.0)
    np.testing.assert_allclose(y.cpu().numpy(), want, rtol=1e-6, atol=1e-6)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(y.cpu().numpy() - ref).max() < 0.08 * np.abs(ref).max()   # SPARQ + 8-bit noise stays small


def test_rejected():
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_quantize_act_u8(x[1:], mx, out)               # misaligned input
    assert ei.value.code == -2
    L = sparq.load_library()
    assert L.sparq_absmax(x.data_ptr(), 7, 64, mx.data_ptr(), None) == -1      # unknown dtype
    assert L.sparq_absmax(None, 0, 0, mx.data_ptr(), None) == 0                 # empty: no-op
