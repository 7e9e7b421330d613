"""Pins for the oracle's uniform min-max quantization (Section 5 of the paper: unsigned
symmetric per layer for activations, signed symmetric per kernel for weights).

Closed forms (grid points map to their index), the half-step error bound of a uniform
quantizer evaluated in float64, ties and saturation cases worked by hand, and bf16 widening
checked against a bit-level conversion written here."""
import numpy as np
import pytest

import oracle


def test_absmax_skips_nan_and_takes_magnitudes():
    x = np.array([0.5, -3.25, np.nan, 2.0, -0.0], dtype=np.float32)
    assert oracle.absmax(x) == 3.25
    assert oracle.absmax(np.zeros(7, np.float32)) == 0.0
    assert oracle.absmax(np.array([], np.float32)) == 0.0
    rng = np.random.default_rng(0)
    y = rng.standard_normal(10_001).astype(np.float32)
    assert oracle.absmax(y) == np.abs(y).max()


def test_activation_grid_points_map_to_their_index():
    # max = 255 * step with step a power of two: every grid point k * step is exact in fp32
    for step in (0.5, 0.03125, 4.0):
        x = (np.arange(256, dtype=np.float32) * np.float32(step))
        q = oracle.quantize_act(x, 255 * step)
        assert np.array_equal(q, np.arange(256, dtype=np.uint8))


def test_activation_cases_by_hand():
    # max 255 -> one step is 1.0: ties go to the even neighbour, negatives and NaN give 0,
    # values past the max saturate
    x = np.array([0.5, 1.5, 2.5, 254.5, 255.4, 300.0, -3.0, np.nan, 0.49999, 1e-30], dtype=np.float32)
    assert list(oracle.quantize_act(x, 255.0)) == [0, 2, 2, 254, 255, 255, 0, 0, 0, 0]
    assert list(oracle.quantize_act(x, 0.0)) == [0] * 10          # degenerate layer: all zero


@pytest.mark.parametrize("mx", [1.0, 6.0, 0.731, 117.3])
def test_activation_error_is_at_most_half_a_step(mx):
    rng = np.random.default_rng(1)
    x = (rng.random(50_000) * mx).astype(np.float32)
    x[0] = mx
    q = oracle.quantize_act(x, mx)
    step = np.float64(np.float32(mx)) / 255.0
    err = np.abs(q.astype(np.float64) * step - x.astype(np.float64))
    assert err.max() <= step / 2 * (1 + 1e-5)
    assert q[0] == 255 and q.min() >= 0
    assert np.all(np.diff(q[np.argsort(x, kind="stable")].astype(np.int32)) >= 0)   # monotone


def bf16_bits(x32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns by truncation (any rounding would do for the test)."""
    return (x32.view(np.uint32) >> 16).astype(np.uint16)


def test_bf16_inputs_are_widened_exactly():
    rng = np.random.default_rng(2)
    x32 = (rng.random(4096) * 6.0).astype(np.float32)
    bits = bf16_bits(x32)
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    assert oracle.absmax(bits) == oracle.absmax(widened)
    mx = oracle.absmax(widened)
    assert np.array_equal(oracle.quantize_act(bits, mx), oracle.quantize_act(widened, mx))


def test_weights_per_kernel():
    rng = np.random.default_rng(3)
    w = (rng.standard_normal((12, 3, 3, 16)) * np.arange(1, 13).reshape(12, 1, 1, 1)).astype(np.float32)
    w[5] = 0.0                                             # an all-zero kernel
    q, sc = oracle.quantize_weight(w)
    assert q.dtype == np.int8 and q.shape == w.shape and sc.shape == (12,)
    for j in range(12):
        a = np.abs(w[j]).max()
        assert sc[j] == np.float32(a) / np.float32(127.0)
        if a == 0:
            assert not q[j].any()
            continue
        assert np.abs(q[j]).max() == 127                   # the largest magnitude lands on the grid's end
        assert q[j].min() >= -127
        step = np.float64(a) / 127.0
        err = np.abs(q[j].astype(np.float64) * step - w[j].astype(np.float64))
        assert err.max() <= step / 2 * (1 + 1e-5)
        assert np.array_equal(np.sign(q[j]) * (q[j] != 0), np.sign(w[j]) * (q[j] != 0))
    # exact grid: kernel = {-127..127} * 2^-5 maps to its indices
    g = (np.arange(-127, 128, dtype=np.float32) * np.float32(2.0 ** -5)).reshape(1, -1)
    qg, sg = oracle.quantize_weight(g)
    assert np.array_equal(qg[0], np.arange(-127, 128, dtype=np.int8)) and sg[0] == np.float32(2.0 ** -5)


def test_quantized_layer_reproduces_the_float_layer():
    # end to end through the existing oracle: u8 x s8 GEMM with scale = act step * weight step
    # approximates the float matrix product to within the quantization noise
    rng = np.random.default_rng(4)
    x = np.maximum(rng.standard_normal((64, 128)), 0).astype(np.float32)
    w = (rng.standard_normal((32, 128)) * 0.1).astype(np.float32)
    mx = oracle.absmax(x)
    xq = oracle.quantize_act(x, mx)
    wq, ws = oracle.quantize_weight(w)
    acc = oracle.gemm(xq, np.ascontiguousarray(wq.T), oracle.MODE_NONE, 4, 0x1F, 1)
    y = acc * (np.float32(mx) / np.float32(255.0)) * ws[None, :]
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(y - ref).max() < 0.05 * np.abs(ref).max()
