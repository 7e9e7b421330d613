"""Fused SPARQ GEMM (CUDA, through the C ABI) vs the CPU oracle.

Integer outputs (accumulators, requantized bytes) must match bit for bit; the fp32
dequantized output within rel 1e-6 / abs 1e-6."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-6

VARIANTS = [
    (sparq.MODE_NONE, 4, 0x1F, 1),
    (sparq.MODE_BSPARQ, 4, 0x1F, 1), (sparq.MODE_BSPARQ, 4, 0x15, 0), (sparq.MODE_BSPARQ, 3, 0x3F, 1),
    (sparq.MODE_BSPARQ, 2, 0x7F, 0),
    (sparq.MODE_VSPARQ, 4, 0x1F, 1), (sparq.MODE_VSPARQ, 4, 0x1F, 0), (sparq.MODE_VSPARQ, 4, 0x15, 1),
    (sparq.MODE_VSPARQ, 4, 0x11, 1), (sparq.MODE_VSPARQ, 3, 0x3F, 1), (sparq.MODE_VSPARQ, 3, 0x29, 0),
    (sparq.MODE_VSPARQ, 2, 0x7F, 1), (sparq.MODE_VSPARQ, 2, 0x55, 0),
]


def gpu_gemm(A, B_kn, params, scale=None, bias=None, relu=False, inv=1.0, want=("acc", "f32", "u8")):
    M, K = A.shape
    N = B_kn.shape[1]
    Ad = torch.from_numpy(A).cuda()
    Bd = torch.from_numpy(np.ascontiguousarray(B_kn.T)).cuda()     # the ABI takes B as N x K
    outs = {
        "acc": torch.full((M, N), -7, dtype=torch.int32, device="cuda") if "acc" in want else None,
        "f32": torch.full((M, N), -7.0, dtype=torch.float32, device="cuda") if "f32" in want else None,
        "u8": torch.full((M, N), 7, dtype=torch.uint8, device="cuda") if "u8" in want else None,
    }
    sd = None if scale is None else torch.from_numpy(scale).cuda()
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    sparq.sparq_gemm_s8(Ad, Bd, params, scale=sd, bias=bd, relu=relu, inv_out_scale=inv,
                        acc_out=outs["acc"], f32_out=outs["f32"], u8_out=outs["u8"])
    sparq.sparq_check()
    return {k: (None if v is None else v.cpu().numpy()) for k, v in outs.items()}


def check(A, B_kn, variant, scale, bias, relu, inv):
    mode, n, mask, rnd = variant
    got = gpu_gemm(A, B_kn, sparq.SparqParams(mode, n, mask, rnd), scale, bias, relu, inv)
    acc = oracle.gemm(A, B_kn, mode, n, mask, rnd)
    f, q = oracle.epilogue(acc, scale, bias, relu, inv)
    assert np.array_equal(got["acc"], acc)
    assert np.array_equal(got["u8"], q)
    assert np.allclose(got["f32"], f, rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("variant", VARIANTS)
def test_config1_tiny_gemm(variant):
    # A 256 x 576 with 50% zeros, B 576 x 64, per-column scale from U(0.001, 0.01)
    A = synth.activations(0, (256, 576), 0.5)
    B = synth.weights(0, (576, 64))
    scale = synth.scales(0, 64)
    check(A, B, variant, scale, None, False, synth.inv_out_scale(576))


@pytest.mark.parametrize("shape", [
    (1, 1, 16), (127, 63, 48), (129, 65, 80), (300, 200, 400), (384, 100, 64), (1000, 256, 1024),
    (257, 513, 192), (4096, 320, 128), (130, 24, 1040), (20000, 128, 512),
])
def test_shapes_spanning_tiles_and_ragged_tails(shape):
    M, N, K = shape
    A = synth.activations(M + N, (M, K), 0.4)
    B = synth.weights(K, (K, N))
    scale, bias = synth.scales(N, N), synth.bias(N, N)
    for variant in (VARIANTS[5], VARIANTS[0], VARIANTS[9]):
        check(A, B, variant, scale, bias, True, synth.inv_out_scale(K, 0.4))


def test_accumulator_extremes_and_longest_reduction():
    K = 65536
    A = np.full((128, K), 255, dtype=np.uint8)
    B = np.full((K, 16), -128, dtype=np.int8)
    B[:, 1] = 127
    got = gpu_gemm(A, B, sparq.SparqParams(sparq.MODE_NONE), want=("acc",))
    assert (got["acc"][:, 0] == K * 255 * -128).all() and (got["acc"][:, 1] == K * 255 * 127).all()
    got = gpu_gemm(A, B, sparq.SparqParams(sparq.MODE_BSPARQ, 4, 0x1F, 1), want=("acc",))
    assert (got["acc"][:, 0] == K * 240 * -128).all()          # 255 saturates to the top window 1111 << 4


def test_all_zero_and_single_nonzero_rows():
    A = np.zeros((256, 256), dtype=np.uint8)
    A[5, 7] = 201           # lone non-zero of its pair keeps 8 bits under vSPARQ
    A[9, 10], A[9, 11] = 201, 3
    B = synth.weights(2, (256, 64))
    for variant in (VARIANTS[5], VARIANTS[1]):
        mode, n, mask, rnd = variant
        got = gpu_gemm(A, B, sparq.SparqParams(mode, n, mask, rnd), want=("acc",))
        assert np.array_equal(got["acc"], oracle.gemm(A, B, mode, n, mask, rnd))


def test_only_u8_output_and_strided_operands():
    M, N, K, lda, ldb = 200, 96, 128, 160, 144
    A_full = synth.activations(8, (M, lda), 0.5)
    B_full = synth.weights(8, (N, ldb))
    A, B_nk = A_full[:, :K], B_full[:, :K]
    scale = synth.scales(8, N)
    Ad, Bd = torch.from_numpy(A_full).cuda(), torch.from_numpy(B_full).cuda()
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    import ctypes
    from paper_2105_11010_b200._binding import _CEpilogue, _stream_ptr
    L = sparq.load_library()
    p = sparq.SparqParams()._c()
    sd = torch.from_numpy(scale).cuda()
    e = _CEpilogue(sd.data_ptr(), None, 1, synth.inv_out_scale(K), None, None, u8.data_ptr())
    rc = L.sparq_gemm_s8(Ad.data_ptr(), lda, Bd.data_ptr(), ldb, M, N, K, ctypes.byref(p), ctypes.byref(e), _stream_ptr(None))
    assert rc == 0, sparq.sparq_last_error()
    sparq.sparq_check()
    acc = oracle.gemm(np.ascontiguousarray(A), np.ascontiguousarray(B_nk.T), 2, 4, 0x1F, 1)
    _, q = oracle.epilogue(acc, scale, None, True, synth.inv_out_scale(K))
    assert np.array_equal(u8.cpu().numpy(), q)


def test_rejected_arguments():
    A = torch.zeros((128, 24), dtype=torch.uint8, device="cuda")
    B = torch.zeros((64, 24), dtype=torch.int8, device="cuda")
    acc = torch.zeros((128, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), acc_out=acc)        # K not a multiple of 16
    assert ei.value.code == -2
    A = torch.zeros((128, 32), dtype=torch.uint8, device="cuda")
    B = torch.zeros((64, 32), dtype=torch.int8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams())                     # no output requested
    assert ei.value.code == -1
    with pytest.raises(sparq.SparqError):
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), u8_out=torch.zeros((128, 64), dtype=torch.uint8, device="cuda"))  # no scale
    sparq.sparq_gemm_s8(A[:0], B, sparq.SparqParams(), acc_out=acc)        # M == 0: no-op


@pytest.mark.parametrize("shape", [
    # M, K, N: the requantized-bytes-only form takes its own straight-line epilogue path
    (1000, 64, 256),      # short reduction (add-based int -> float), ragged last row tile
    (777, 128, 96),       # last column group of a warp only partly inside N: general path for it
    (2048, 576, 64),      # long reduction (conversion-based int -> float), 64-wide tiles
    (300, 1024, 512),     # two column tiles of 256
    (20000, 64, 128),     # more tiles than SMs
])
@pytest.mark.parametrize("mode", [sparq.MODE_VSPARQ, sparq.MODE_NONE])
@pytest.mark.parametrize("relu", [True, False])
def test_bytes_only_output_exact(shape, mode, relu):
    M, K, N = shape
    seed = 7000 + M + K + N
    A = synth.activations(seed, (M, K), 0.5)
    B = synth.weights(seed + 1, (K, N))
    scale, bias = synth.scales(seed + 2, N), synth.bias(seed + 3, N)
    inv = synth.inv_out_scale(K)
    got = gpu_gemm(A, B, sparq.SparqParams(mode, 4, 0x1F, 1), scale, bias, relu, inv, want=("u8",))
    acc = oracle.gemm(A, B, mode, 4, 0x1F, 1)
    _, q = oracle.epilogue(acc, scale, bias, relu, inv)
    assert np.array_equal(got["u8"], q)
