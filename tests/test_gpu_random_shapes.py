"""Seeded random shapes, variants and epilogue options through the fused GEMM and convolution
(CUDA, through the C ABI) against the CPU oracle.

The other files pick their shapes by hand around known tile and dispatch boundaries; here they
are drawn, so that a boundary nobody thought of (a tile width, a reduction step, the choice
between the window and the im2col kernel, an epilogue path that depends on which outputs are
wanted) still meets a case.  Every case is reproducible from its index."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

RTOL, ATOL = 1e-6, 1e-6

# (mode, n, mask, rounding is drawn)
VARIANTS = [
    (sparq.MODE_NONE, 4, 0x1F),
    (sparq.MODE_BSPARQ, 4, 0x1F), (sparq.MODE_BSPARQ, 4, 0x15), (sparq.MODE_BSPARQ, 3, 0x3F), (sparq.MODE_BSPARQ, 2, 0x7F),
    (sparq.MODE_VSPARQ, 4, 0x1F), (sparq.MODE_VSPARQ, 4, 0x15), (sparq.MODE_VSPARQ, 4, 0x11),
    (sparq.MODE_VSPARQ, 3, 0x3F), (sparq.MODE_VSPARQ, 3, 0x35), (sparq.MODE_VSPARQ, 3, 0x29),
    (sparq.MODE_VSPARQ, 2, 0x7F), (sparq.MODE_VSPARQ, 2, 0x55),
]
WANTS = [("u8",), ("u8",), ("acc", "f32", "u8"), ("f32", "u8"), ("acc", "u8"), ("f32",), ("acc",)]

N_GEMM, N_CONV = 64, 56


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def draw_common(rng, n_cols):
    """Variant, epilogue options and which outputs are wanted."""
    mode, n, mask = VARIANTS[rng.integers(len(VARIANTS))]
    variant = sparq.SparqParams(mode, n, mask, int(rng.integers(2)))
    want = WANTS[rng.integers(len(WANTS))]
    opts = {
        "relu": bool(rng.integers(2)),
        "bias": bool(rng.integers(4)),                          # mostly present
        "zero_frac": float(rng.choice([0.0, 0.3, 0.5, 0.9])),
        "residual": ("u8" in want or "f32" in want) and rng.integers(4) == 0,
        "next": None,
    }
    if "u8" in want and n_cols % 4 == 0 and rng.integers(3) == 0:
        m2, n2, k2 = VARIANTS[1 + rng.integers(len(VARIANTS) - 1)]
        opts["next"] = sparq.SparqParams(m2, n2, k2, int(rng.integers(2)))
    return variant, want, opts


def run_and_compare(launch, acc_want, shape, n_cols, k, seed, variant, want, opts, tag):
    scale = synth.scales(seed, n_cols)
    bias = synth.bias(seed, n_cols) if opts["bias"] else None
    inv = synth.inv_out_scale(k, max(opts["zero_frac"], 0.3))
    res = synth.activations(seed + 5, shape, 0.3, stream=4) if opts["residual"] else None
    rs = 0.37 if opts["residual"] else 0.0
    outs = {
        "acc": torch.full(shape, -7, dtype=torch.int32, device="cuda") if "acc" in want else None,
        "f32": torch.full(shape, -7.0, dtype=torch.float32, device="cuda") if "f32" in want else None,
        "u8": torch.full(shape, 7, dtype=torch.uint8, device="cuda") if "u8" in want else None,
    }
    need_f = "f32" in want or "u8" in want
    launch(variant, dict(scale=dev(scale) if need_f else None, bias=dev(bias) if need_f else None, relu=opts["relu"],
                         inv_out_scale=inv, acc_out=outs["acc"], f32_out=outs["f32"], u8_out=outs["u8"],
                         next_transform=opts["next"], residual=dev(res), residual_scale=rs))
    sparq.sparq_check()
    if "acc" in want:
        assert np.array_equal(outs["acc"].cpu().numpy(), acc_want), tag
    if need_f:
        f, q = oracle.epilogue(acc_want, scale, bias, opts["relu"], inv, residual=res, residual_scale=rs)
        if "f32" in want:
            np.testing.assert_allclose(outs["f32"].cpu().numpy(), f, rtol=RTOL, atol=ATOL, err_msg=tag)
        if "u8" in want:
            nx = opts["next"]
            if nx is not None:
                q = oracle.transform(q, nx.mode, nx.window_bits, nx.placement_mask, nx.rounding)
            assert np.array_equal(outs["u8"].cpu().numpy(), q), tag


def gemm_case(i):
    rng = np.random.default_rng([2105, 11010, 1, i])
    kind = rng.integers(4)
    if kind == 0:        # small everything
        M, N, K = int(rng.integers(1, 140)), int(rng.integers(1, 70)), 16 * int(rng.integers(1, 12))
    elif kind == 1:      # several row tiles, ragged columns
        M, N, K = int(rng.integers(129, 900)), int(rng.integers(1, 300)), 16 * int(rng.integers(1, 40))
    elif kind == 2:      # wide: several column tiles
        M, N, K = int(rng.integers(1, 300)), int(rng.integers(257, 700)), 16 * int(rng.integers(1, 24))
    else:                # long reduction
        M, N, K = int(rng.integers(1, 260)), int(rng.integers(1, 200)), 16 * int(rng.integers(60, 400))
    if rng.integers(2):
        N = (N + 3) // 4 * 4
    variant, want, opts = draw_common(rng, N)
    return M, N, K, variant, want, opts


@pytest.mark.gpu
@pytest.mark.parametrize("i", range(N_GEMM))
def test_random_gemm(i):
    M, N, K, variant, want, opts = gemm_case(i)
    tag = f"gemm case {i}: M={M} N={N} K={K} {variant} want={want} {opts}"
    A = synth.activations(1000 + i, (M, K), opts["zero_frac"])
    B = synth.weights(1000 + i, (K, N))
    acc = oracle.gemm(A, B, variant.mode, variant.window_bits, variant.placement_mask, variant.rounding)
    Ad, Bd = dev(A), dev(B.T)

    def launch(v, kw):
        sparq.sparq_gemm_s8(Ad, Bd, v, **kw)

    run_and_compare(launch, acc, (M, N), N, K, 1000 + i, variant, want, opts, tag)


def conv_case(i):
    rng = np.random.default_rng([2105, 11010, 2, i])
    r, s = [(1, 1), (3, 3), (3, 3), (3, 3), (5, 5), (1, 3), (3, 1), (7, 7)][rng.integers(8)]
    stride = int(rng.choice([1, 1, 1, 2]))
    pad = int(rng.integers(0, min(max(r, s) // 2, min(r, s) - 1) + 1))      # the library wants pad < filter extent
    h = int(rng.integers(max(r, 4), 34))
    w = int(rng.integers(max(s, 4), 34))
    # channel counts the window kernel takes (64, multiples of 128) and ones it does not
    c = int(rng.choice([16, 32, 48, 64, 64, 96, 128, 128, 160, 256, 384]))
    if r * s >= 25:
        c = min(c, 64)
    cout = int(rng.choice([8, 24, 64, 64, 72, 128, 128, 192, 256, 320]))
    nb = int(rng.integers(1, 5))
    variant, want, opts = draw_common(rng, cout)
    return nb, h, w, c, cout, r, s, stride, pad, variant, want, opts


@pytest.mark.gpu
@pytest.mark.parametrize("i", range(N_CONV))
def test_random_conv(i):
    nb, h, w, c, cout, r, s, stride, pad, variant, want, opts = conv_case(i)
    tag = f"conv case {i}: {nb}x{h}x{w}x{c} -> {cout} {r}x{s}/s{stride} p{pad} {variant} want={want} {opts}"
    ho, wo = synth.conv_out_hw(h, w, r, s, stride, pad)
    assert ho > 0 and wo > 0, tag
    x = synth.activations(2000 + i, (nb, h, w, c), opts["zero_frac"])
    wt = synth.weights(2000 + i, (cout, r, s, c))
    acc = oracle.conv2d_nhwc(x, wt, (stride, stride), (pad, pad), variant.mode, variant.window_bits,
                             variant.placement_mask, variant.rounding)
    xd, wd = dev(x), dev(wt)

    def launch(v, kw):
        sparq.sparq_conv2d_nhwc_s8(xd, wd, (stride, stride), (pad, pad), v, **kw)

    run_and_compare(launch, acc, (nb, ho, wo, cout), cout, r * s * c, 2000 + i, variant, want, opts, tag)


def test_the_draws_cover_the_dispatch():
    """Runs without a GPU: the drawn cases reach every variant, both kernels' shapes and every option."""
    g = [gemm_case(i) for i in range(N_GEMM)]
    c = [conv_case(i) for i in range(N_CONV)]
    seen = {(v.mode, v.window_bits, v.placement_mask) for *_, v, _, _ in g} | {(cc[9].mode, cc[9].window_bits, cc[9].placement_mask) for cc in c}
    assert len(seen) == len(VARIANTS)
    assert any(o["residual"] for *_, o in g) and any(o["next"] is not None for *_, o in g)
    assert any(cc[11]["residual"] for cc in c) and any(cc[11]["next"] is not None for cc in c)
    # window-kernel shapes (stride 1, 64 or a multiple of 128 channels, 3x3) and im2col shapes
    assert any(cc[7] == 1 and cc[3] in (64, 128, 256, 384) and cc[5] == 3 for cc in c)
    assert any(cc[7] == 2 or cc[3] in (16, 32, 48, 96, 160) for cc in c)
    assert any(k >= 16 * 60 for _, _, k, *_ in g) and any(n > 256 for _, n, *_ in g)
