"""Pins for the oracle's dot product, convolution and epilogue.

The products are pinned to library routines that are not the oracle's loops:
numpy's int64 matmul and torch's float64 conv2d (exact on these small integers)."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth

P = dict(mode=oracle.MODE_VSPARQ, n=4, mask=0x1F, rnd=1)


def py_transform(A, mode, n, mask, rnd):
    """Row-wise T built from the scalar definitions only."""
    out = np.zeros_like(A)
    for i, row in enumerate(A):
        for k in range(0, len(row), 2):
            a = int(row[k]); b = int(row[k + 1]) if k + 1 < len(row) else 0
            if mode == 0:
                qa, qb = a, b
            elif mode == 1:
                qa, qb = oracle.bsparq(a, n, mask, rnd), oracle.bsparq(b, n, mask, rnd)
            else:
                qa, qb = oracle.vsparq_pair(a, b, n, mask, rnd)
            out[i, k] = qa
            if k + 1 < len(row):
                out[i, k + 1] = qb
    return out


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("shape", [(5, 7, 6), (3, 4, 9), (16, 8, 32), (1, 1, 2)])
def test_gemm_matches_numpy_int64(mode, shape):
    M, N, K = shape
    A = synth.activations(11, (M, K), 0.4)
    B = synth.weights(11, (K, N))
    got = oracle.gemm(A, B, mode, 4, 0x1F, 1)
    TA = py_transform(A, mode, 4, 0x1F, 1).astype(np.int64)
    want = TA @ B.astype(np.int64)
    assert got.dtype == np.int32 and np.array_equal(got.astype(np.int64), want)
    assert np.array_equal(oracle.gemm_i64(A, B, mode, 4, 0x1F, 1), want)


def test_gemm_mode_none_is_plain_integer_matmul_and_extremes():
    A = np.full((4, 64), 255, dtype=np.uint8)
    B = np.full((64, 3), -128, dtype=np.int8)
    got = oracle.gemm(A, B, 0, 4, 0x1F, 1)
    assert (got == 64 * 255 * -128).all()
    A = synth.activations(3, (32, 576), 0.5)
    B = synth.weights(3, (576, 16))
    assert np.array_equal(oracle.gemm(A, B, 0, 8, 1, 0), A.astype(np.int64) @ B.astype(np.int64))


def test_gemm_empty():
    assert oracle.gemm(np.zeros((0, 4), np.uint8), np.zeros((4, 3), np.int8), 2, 4, 0x1F, 1).shape == (0, 3)


def torch_conv(tx, w, stride, pad):
    xt = torch.from_numpy(tx.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(xt, wt, stride=stride, padding=pad)
    return y.permute(0, 2, 3, 1).numpy().astype(np.int64)


@pytest.mark.parametrize("cfg", [
    # nb, h, w, c, cout, r, s, stride, pad
    (2, 6, 5, 8, 4, 3, 3, (1, 1), (1, 1)),
    (1, 7, 7, 6, 5, 3, 3, (2, 2), (1, 1)),
    (2, 8, 6, 4, 3, 1, 1, (2, 2), (0, 0)),
    (1, 5, 9, 10, 2, 3, 1, (1, 2), (1, 0)),
    (3, 4, 4, 16, 8, 1, 1, (1, 1), (0, 0)),
])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_conv_matches_torch_conv_of_transformed_input(cfg, mode):
    nb, h, w, c, cout, r, s, stride, pad = cfg
    x = synth.activations(21, (nb, h, w, c), 0.45)
    wt = synth.weights(21, (cout, r, s, c))
    got = oracle.conv2d_nhwc(x, wt, stride, pad, mode, 4, 0x15, 1)
    tx = py_transform(x.reshape(-1, c), mode, 4, 0x15, 1).reshape(x.shape)
    want = torch_conv(tx, wt, stride, pad)
    assert got.shape == want.shape
    assert np.array_equal(got.astype(np.int64), want)


def test_conv_equals_explicit_im2col_then_gemm():
    # T applied to the NHWC tensor commutes with the im2col gather: pairs are adjacent
    # channels of one pixel and padding zeroes both slots of a pair.
    nb, h, w, c, cout, r, s = 2, 5, 6, 8, 7, 3, 3
    x = synth.activations(5, (nb, h, w, c), 0.5)
    wt = synth.weights(5, (cout, r, s, c))
    for stride, pad in [((1, 1), (1, 1)), ((2, 2), (1, 1))]:
        ho = (h + 2 * pad[0] - r) // stride[0] + 1
        wo = (w + 2 * pad[1] - s) // stride[1] + 1
        xp = np.zeros((nb, h + 2 * pad[0], w + 2 * pad[1], c), np.uint8)
        xp[:, pad[0]:pad[0] + h, pad[1]:pad[1] + w] = x
        rows = []
        for b in range(nb):
            for oy in range(ho):
                for ox in range(wo):
                    patch = xp[b, oy * stride[0]:oy * stride[0] + r, ox * stride[1]:ox * stride[1] + s]
                    rows.append(patch.reshape(-1))
        A = np.stack(rows)
        Bm = wt.reshape(cout, -1).T.copy()
        via_gemm = oracle.gemm(A, Bm, **P)   # T applied to the im2col rows
        direct = oracle.conv2d_nhwc(x, wt, stride, pad, **P)
        assert np.array_equal(direct.reshape(-1, cout), via_gemm)


def test_conv_1x1_is_gemm_and_pixel_subset():
    x = synth.activations(9, (2, 4, 4, 32), 0.5)
    wt = synth.weights(9, (12, 1, 1, 32))
    full = oracle.conv2d_nhwc(x, wt, (1, 1), (0, 0), **P)
    g = oracle.gemm(x.reshape(-1, 32), wt.reshape(12, 32).T.copy(), **P)
    assert np.array_equal(full.reshape(-1, 12), g)
    pix = [0, 5, 31, 17]
    sub = oracle.conv2d_nhwc(x, wt, (1, 1), (0, 0), pixels=pix, **P)
    assert np.array_equal(sub, full.reshape(-1, 12)[pix])


def test_epilogue_against_float64_and_numpy_float32():
    rng = np.random.default_rng(3)
    acc = rng.integers(-3_000_000, 3_000_000, size=(64, 48), dtype=np.int64).astype(np.int32)
    acc[0, :4] = [0, 1, -1, 2**31 - 1]
    scale = synth.scales(1, 48)
    b = synth.bias(1, 48)
    inv = np.float32(1.0 / 37.5)
    for relu in (False, True):
        for bb in (b, None):
            f, q = oracle.epilogue(acc, scale, bb, relu, inv)
            y64 = acc.astype(np.float64) * scale.astype(np.float64) + (0 if bb is None else bb.astype(np.float64))
            if relu:
                y64 = np.maximum(y64, 0)
            err = np.abs(f.astype(np.float64) - y64)
            # one rounding of the int->float conversion and one of the fma, both relative
            # to |acc*scale| (the bias can cancel most of it)
            bound = 1.3e-7 * (np.abs(acc.astype(np.float64) * scale) + np.abs(y64)) + 1e-30
            assert (err <= bound).all()
            z = f * inv                      # numpy float32 multiply, then round-half-even
            want_q = np.clip(np.rint(z), 0, 255).astype(np.uint8)
            assert np.array_equal(q, want_q)
            if relu:
                assert (f >= 0).all()


def test_epilogue_rounding_and_saturation_cases():
    acc = np.array([[1, 3, 5, 1000, -7, 2]], dtype=np.int32)
    scale = np.full(6, 0.5, np.float32)
    f, q = oracle.epilogue(acc, scale, None, False, 1.0)
    assert list(f[0]) == [0.5, 1.5, 2.5, 500.0, -3.5, 1.0]
    assert list(q[0]) == [0, 2, 2, 255, 0, 1]      # ties to even, clamp to [0, 255]


def test_epilogue_residual_against_float64():
    # y = acc*scale + bias + residual*residual_scale, then ReLU: the float64 value bounds the
    # fp32 result (three roundings), the residual is added BEFORE the ReLU, and a NULL
    # residual or a zero residual tensor leaves the plain epilogue.
    rng = np.random.default_rng(5)
    acc = rng.integers(-300_000, 300_000, size=(32, 40), dtype=np.int64).astype(np.int32)
    scale = synth.scales(2, 40)
    b = synth.bias(2, 40)
    res = rng.integers(0, 256, size=(32, 40), dtype=np.uint8)
    rs = np.float32(0.37)
    inv = np.float32(1.0 / 9.0)
    for relu in (False, True):
        f, q = oracle.epilogue(acc, scale, b, relu, inv, residual=res, residual_scale=rs)
        part = acc.astype(np.float64) * scale + b
        y64 = part + res.astype(np.float64) * np.float64(rs)
        if relu:
            y64 = np.maximum(y64, 0)
        bound = 1.3e-7 * (np.abs(acc.astype(np.float64) * scale) + np.abs(part)
                          + np.abs(res * np.float64(rs)) + np.abs(y64)) + 1e-30
        assert (np.abs(f - y64) <= bound).all()
        assert np.array_equal(q, np.clip(np.rint(f * inv), 0, 255).astype(np.uint8))
        f0, q0 = oracle.epilogue(acc, scale, b, relu, inv)
        fz, qz = oracle.epilogue(acc, scale, b, relu, inv, residual=np.zeros_like(res), residual_scale=rs)
        assert np.array_equal(f0, fz) and np.array_equal(q0, qz)
        assert not np.array_equal(f0, f)


def test_epilogue_residual_exact_cases():
    # values exact in fp32: (acc*0.5 + 1) + res*0.25, ReLU after the sum
    acc = np.array([[-10, -10, 4, 0]], dtype=np.int32)
    scale = np.full(4, 0.5, np.float32)
    bias = np.ones(4, np.float32)
    res = np.array([[8, 32, 2, 255]], dtype=np.uint8)
    f, q = oracle.epilogue(acc, scale, bias, True, 1.0, residual=res, residual_scale=0.25)
    assert list(f[0]) == [0.0, 4.0, 3.5, 64.75]       # -4+2 -> ReLU 0 ; -4+8 ; 3+0.5 ; 1+63.75
    assert list(q[0]) == [0, 4, 4, 65]
    f, _ = oracle.epilogue(acc, scale, bias, False, 1.0, residual=res, residual_scale=0.25)
    assert f[0, 0] == -2.0
