"""Fused SPARQ convolution (CUDA, through the C ABI) vs the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-6
V5 = (sparq.MODE_VSPARQ, 4, 0x1F, 1)


def gpu_conv(x, w, stride, pad, variant, scale=None, bias=None, relu=False, inv=1.0, want=("acc", "f32", "u8")):
    mode, n, mask, rnd = variant
    nb, h, wd, c = x.shape
    cout, r, s, _ = w.shape
    ho, wo = synth.conv_out_hw(h, wd, r, s, stride, pad)
    shape = (nb, ho, wo, cout)
    xd, wdv = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    outs = {
        "acc": torch.full(shape, -7, dtype=torch.int32, device="cuda") if "acc" in want else None,
        "f32": torch.full(shape, -7.0, dtype=torch.float32, device="cuda") if "f32" in want else None,
        "u8": torch.full(shape, 7, dtype=torch.uint8, device="cuda") if "u8" in want else None,
    }
    sd = None if scale is None else torch.from_numpy(scale).cuda()
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    sparq.sparq_conv2d_nhwc_s8(xd, wdv, (stride, stride), (pad, pad), sparq.SparqParams(mode, n, mask, rnd),
                               scale=sd, bias=bd, relu=relu, inv_out_scale=inv,
                               acc_out=outs["acc"], f32_out=outs["f32"], u8_out=outs["u8"])
    sparq.sparq_check()
    return {k: (None if v is None else v.cpu().numpy()) for k, v in outs.items()}


def check_full(x, w, stride, pad, variant, seed):
    mode, n, mask, rnd = variant
    cout, r, s, c = w.shape
    scale, bias = synth.scales(seed, cout), synth.bias(seed, cout)
    inv = synth.inv_out_scale(r * s * c)
    got = gpu_conv(x, w, stride, pad, variant, scale, bias, True, inv)
    acc = oracle.conv2d_nhwc(x, w, (stride, stride), (pad, pad), mode, n, mask, rnd)
    f, q = oracle.epilogue(acc, scale, bias, True, inv)
    assert np.array_equal(got["acc"], acc)
    assert np.array_equal(got["u8"], q)
    assert np.allclose(got["f32"], f, rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("cfg", [
    # nb, h, w, c, cout, r, s, stride, pad
    (2, 8, 8, 64, 64, 3, 3, 1, 1),
    (3, 14, 14, 128, 128, 3, 3, 2, 1),
    (3, 14, 14, 256, 512, 1, 1, 2, 0),
    (5, 7, 7, 64, 96, 3, 3, 1, 1),
    (2, 9, 11, 192, 40, 3, 3, 2, 1),
    (1, 13, 13, 128, 72, 5, 5, 1, 2),
    (2, 12, 10, 64, 64, 1, 3, 1, 0),
    (3, 10, 10, 48, 80, 1, 1, 1, 0),
    (2, 28, 28, 256, 256, 3, 3, 1, 1),
])
@pytest.mark.parametrize("variant", [V5, (sparq.MODE_NONE, 4, 0x1F, 1), (sparq.MODE_BSPARQ, 3, 0x3F, 0)])
def test_small_convolutions_exact(cfg, variant):
    nb, h, w, c, cout, r, s, stride, pad = cfg
    x = synth.activations(sum(cfg), (nb, h, w, c), 0.45)
    wt = synth.weights(sum(cfg), (cout, r, s, c))
    check_full(x, wt, stride, pad, variant, seed=sum(cfg))


@pytest.mark.parametrize("cfg", [
    # shapes chosen to walk the stride-1 window kernel's paths and its fall-backs
    (2, 30, 30, 384, 128, 3, 3, 1, 1),    # three channel blocks: 27 (tap, block) pairs, streamed weights
    (3, 17, 23, 128, 200, 3, 3, 1, 1),    # cout not a tile multiple, rows not a multiple of the tile height
    (1, 40, 20, 64, 64, 3, 3, 1, 1),      # tall image, 64-channel resident weights
    (2, 14, 14, 256, 256, 3, 3, 1, 1),    # two channel blocks, partial last tile per image
    (1, 8, 140, 64, 64, 3, 3, 1, 1),      # padded width above 128: im2col kernel
    (1, 20, 20, 64, 64, 7, 7, 1, 3),      # 49 taps do not fit resident: im2col kernel
    (2, 9, 9, 128, 128, 3, 3, 1, 0),      # no padding: output smaller than input
    (2, 16, 16, 128, 128, 2, 2, 1, 1),    # even filter size
    (4, 7, 7, 512, 512, 3, 3, 1, 1),      # 7x7 maps (too small for the window tiling)
])
def test_stride1_filter_shapes_exact(cfg):
    nb, h, w, c, cout, r, s, stride, pad = cfg
    x = synth.activations(sum(cfg) + 1, (nb, h, w, c), 0.5)
    wt = synth.weights(sum(cfg) + 1, (cout, r, s, c))
    for variant in (V5, (sparq.MODE_VSPARQ, 3, 0x29, 0)):
        check_full(x, wt, stride, pad, variant, seed=sum(cfg))


@pytest.mark.parametrize("cfg", [
    # more tiles than SMs, so that a CTA's share of the tile sequence holds several tiles: groups
    # of tiles sharing one window, shares that cross image boundaries, short last groups
    (12, 56, 56, 64, 64, 3, 3, 1, 1),     # 336 tiles of two rows: groups of three, 64-channel resident weights
    (40, 28, 28, 128, 128, 3, 3, 1, 1),   # 280 tiles of four rows: groups of two beside 144 KB of weights
    (30, 27, 28, 128, 128, 3, 3, 1, 1),   # last tile of every image has three rows
    (80, 14, 14, 256, 256, 3, 3, 1, 1),   # two channel blocks, streamed weights, 256-wide tiles
    (23, 28, 28, 128, 256, 3, 3, 1, 1),   # 161 tiles, two column tiles or one 256-wide
])
@pytest.mark.parametrize("variant", [V5, (sparq.MODE_NONE, 4, 0x1F, 1)])
def test_grouped_windows_exact(cfg, variant):
    nb, h, w, c, cout, r, s, stride, pad = cfg
    x = synth.activations(sum(cfg) + 2, (nb, h, w, c), 0.45)
    wt = synth.weights(sum(cfg) + 2, (cout, r, s, c))
    check_full(x, wt, stride, pad, variant, seed=sum(cfg))


def test_config2_resnet18_conv_full():
    # 32 x 56 x 56 x 64, 45% zeros, 3x3 stride 1 pad 1, 64 filters; scale, bias, ReLU, requant
    x = synth.activations(1, (32, 56, 56, 64), 0.45)
    wt = synth.weights(1, (64, 3, 3, 64))
    check_full(x, wt, 1, 1, V5, seed=1)


def sampled_pixels(total, seed, count=192):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, total - 129, total - 128, total - 1]
    pix = sorted(set(int(p) for p in fixed if 0 <= p < total) | set(int(p) for p in rng.integers(0, total, count)))
    return np.array(pix, dtype=np.int64)


@pytest.mark.parametrize("layer", list(range(22)))
def test_config3_resnet50_layers_batch64_sampled(layer):
    """Every conv shape of the ResNet-50 stack at batch 64, launched as the benchmark
    launches it; the oracle computes a sample of output pixels one by one."""
    L = synth.resnet50_conv_layers()[layer]
    seed = 100 + layer
    zf = float(np.random.default_rng(seed).uniform(0.3, 0.7))
    x = synth.activations(seed, (64, L.h, L.w, L.cin), zf)
    wt = synth.weights(seed, (L.cout, L.r, L.s, L.cin))
    scale, bias = synth.scales(seed, L.cout), synth.bias(seed, L.cout)
    inv = synth.inv_out_scale(L.r * L.s * L.cin, zf)
    got = gpu_conv(x, wt, L.stride, L.pad, V5, scale, bias, True, inv, want=("u8", "acc"))
    ho, wo = L.out_hw()
    pix = sampled_pixels(64 * ho * wo, seed)
    acc = oracle.conv2d_nhwc(x, wt, (L.stride, L.stride), (L.pad, L.pad), *V5, pixels=pix)
    _, q = oracle.epilogue(acc, scale, bias, True, inv)
    assert np.array_equal(got["acc"].reshape(-1, L.cout)[pix], acc)
    assert np.array_equal(got["u8"].reshape(-1, L.cout)[pix], q)
    # size-independent property: requantized outputs are a function of the accumulators
    f_all, q_all = oracle.epilogue(got["acc"], scale, bias, True, inv)
    assert np.array_equal(got["u8"], q_all)


def test_config3_chained_bottleneck_u8_feeds_u8():
    # 1x1 -> 3x3 -> 1x1, each layer's requantized output is the next layer's input
    nb, hw, cin, mid = 4, 28, 512, 128
    x = synth.activations(7, (nb, hw, hw, cin), 0.5)
    shapes = [(mid, 1, 1, cin, 0), (mid, 3, 3, mid, 1), (cin, 1, 1, mid, 0)]
    cur_gpu, cur_cpu = x, x
    for i, (cout, r, s, c, pad) in enumerate(shapes):
        wt = synth.weights(70 + i, (cout, r, s, c))
        scale, bias = synth.scales(70 + i, cout), synth.bias(70 + i, cout)
        inv = synth.inv_out_scale(r * s * c)
        cur_gpu = gpu_conv(cur_gpu, wt, 1, pad, V5, scale, bias, True, inv, want=("u8",))["u8"]
        acc = oracle.conv2d_nhwc(cur_cpu, wt, (1, 1), (pad, pad), *V5)
        _, cur_cpu = oracle.epilogue(acc, scale, bias, True, inv)
        assert np.array_equal(cur_gpu, cur_cpu), i
    assert 0.2 < (cur_cpu == 0).mean() < 0.8      # the chain keeps a realistic zero fraction


ABLATION = [
    (sparq.MODE_VSPARQ, 4, 0x1F, 1), (sparq.MODE_VSPARQ, 4, 0x1F, 0), (sparq.MODE_VSPARQ, 4, 0x15, 1),
    (sparq.MODE_VSPARQ, 4, 0x11, 1), (sparq.MODE_VSPARQ, 3, 0x3F, 1), (sparq.MODE_VSPARQ, 3, 0x35, 1),
    (sparq.MODE_VSPARQ, 3, 0x29, 0), (sparq.MODE_VSPARQ, 2, 0x7F, 1), (sparq.MODE_VSPARQ, 2, 0x55, 1),
    (sparq.MODE_BSPARQ, 4, 0x1F, 1), (sparq.MODE_BSPARQ, 2, 0x7F, 0),
]


@pytest.mark.parametrize("zero_frac", [0.0, 0.25, 0.5, 0.75, 0.9])
def test_config5_ablation_fused_and_unfused(zero_frac):
    """3x3 conv 128 x 28 x 28 x 128 -> 128: window width, placement set, rounding and
    zero fraction; fused kernel vs transform kernel followed by the plain kernel."""
    nb, hw, c, cout = 128, 28, 128, 128
    seed = 500 + int(zero_frac * 100)
    x = synth.activations(seed, (nb, hw, hw, c), zero_frac)
    wt = synth.weights(seed, (cout, 3, 3, c))
    xd, wd = torch.from_numpy(x).cuda(), torch.from_numpy(wt).cuda()
    pix = sampled_pixels(nb * hw * hw, seed, 96)
    for variant in ABLATION:
        mode, n, mask, rnd = variant
        p = sparq.SparqParams(mode, n, mask, rnd)
        fused = torch.empty((nb, hw, hw, cout), dtype=torch.int32, device="cuda")
        sparq.sparq_conv2d_nhwc_s8(xd, wd, (1, 1), (1, 1), p, acc_out=fused)
        tx = torch.empty_like(xd)
        sparq.sparq_quantize(xd, tx, nb * hw * hw, c, p)
        unfused = torch.empty_like(fused)
        sparq.sparq_conv2d_nhwc_s8(tx, wd, (1, 1), (1, 1), sparq.SparqParams(sparq.MODE_NONE), acc_out=unfused)
        sparq.sparq_check()
        assert torch.equal(fused, unfused), variant
        want = oracle.conv2d_nhwc(x, wt, (1, 1), (1, 1), mode, n, mask, rnd, pixels=pix)
        assert np.array_equal(fused.cpu().numpy().reshape(-1, cout)[pix], want), variant


@pytest.mark.parametrize("cfg", [
    # nb, h, w, c, cout, r, s, stride, pad: channel counts that are multiples of 16 but not of 64
    (2, 9, 9, 16, 40, 3, 3, 1, 1),
    (1, 12, 12, 48, 64, 3, 3, 2, 1),
    (2, 10, 10, 160, 72, 5, 5, 1, 2),
    (1, 8, 8, 96, 128, 7, 7, 1, 3),
    (3, 11, 7, 32, 24, 1, 3, 1, 0),
])
@pytest.mark.parametrize("variant", [V5, (sparq.MODE_NONE, 4, 0x1F, 1), (sparq.MODE_VSPARQ, 2, 0x7F, 0)])
def test_channel_counts_with_a_zero_filled_last_block(cfg, variant):
    # the last 64-channel block of every tap reaches past c: those channels must count as zeros
    # whatever the weights of the next tap are (dense random here)
    nb, h, w, c, cout, r, s, stride, pad = cfg
    x = synth.activations(sum(cfg), (nb, h, w, c), 0.2)
    wt = synth.weights(sum(cfg), (cout, r, s, c))
    check_full(x, wt, stride, pad, variant, seed=sum(cfg))


def test_rejected_arguments():
    x = torch.zeros((1, 8, 8, 32), dtype=torch.uint8, device="cuda")
    w = torch.zeros((16, 3, 3, 32), dtype=torch.int8, device="cuda")
    acc = torch.zeros((1, 8, 8, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_conv2d_nhwc_s8(torch.zeros((1, 8, 8, 24), dtype=torch.uint8, device="cuda"),
                                   torch.zeros((16, 3, 3, 24), dtype=torch.int8, device="cuda"),
                                   (1, 1), (1, 1), sparq.SparqParams(), acc_out=acc)   # c % 16
    assert ei.value.code == -2
    big = torch.zeros((1, 12, 12, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError):
        sparq.sparq_conv2d_nhwc_s8(x, w, (1, 1), (3, 3), sparq.SparqParams(), acc_out=big)   # pad >= filter


def test_weights_written_by_the_previous_launch_are_not_fetched_early():
    """Back-to-back fused launches overlap: a launch may fetch its weights while its predecessor
    is still running -- unless the predecessor writes them.  Here the first convolution's
    requantized output IS the second convolution's weight tensor (same bytes read as int8);
    the second launch must see the finished values."""
    c = 128
    x1 = synth.activations(31, (1, 36, 32, c), 0.4)
    w1 = synth.weights(31, (c, 3, 3, c))
    scale1, bias1 = synth.scales(31, c), synth.bias(31, c)
    inv1 = synth.inv_out_scale(9 * c, 0.4) * 2.0
    x2 = synth.activations(32, (3, 28, 28, c), 0.5)
    acc1 = oracle.conv2d_nhwc(x1, w1, (1, 1), (1, 1), *V5)
    _, q1 = oracle.epilogue(acc1, scale1, bias1, True, inv1)
    w2 = q1.reshape(-1).view(np.int8).reshape(c, 3, 3, c)             # 1152 pixels x 128 channels = 128 x 3 x 3 x 128 bytes
    want = oracle.conv2d_nhwc(x2, w2, (1, 1), (1, 1), *V5)
    p = sparq.SparqParams(*V5)
    x1d, w1d, x2d = torch.from_numpy(x1).cuda(), torch.from_numpy(w1).cuda(), torch.from_numpy(x2).cuda()
    s1, b1 = torch.from_numpy(scale1).cuda(), torch.from_numpy(bias1).cuda()
    wbuf = torch.zeros(c * 9 * c, dtype=torch.uint8, device="cuda")
    acc2 = torch.zeros((3, 28, 28, c), dtype=torch.int32, device="cuda")
    for _ in range(20):
        wbuf.zero_()
        sparq.sparq_conv2d_nhwc_s8(x1d, w1d, (1, 1), (1, 1), p, scale=s1, bias=b1, relu=True, inv_out_scale=inv1,
                                   u8_out=wbuf.view(1, 36, 32, c))
        sparq.sparq_conv2d_nhwc_s8(x2d, wbuf.view(torch.int8).view(c, 3, 3, c), (1, 1), (1, 1), p, acc_out=acc2)
        sparq.sparq_check()
        assert np.array_equal(acc2.cpu().numpy(), want)
