"""The method's edge cases pushed through the FUSED kernels (through the C ABI) vs the CPU oracle.

The standalone transform kernel is checked on all 65,536 byte pairs elsewhere; the fused GEMM,
the window convolution, the im2col convolution and the producer-side transform of the epilogue
instantiate the packed transform differently (run-time window width for everything but
n = 4 / five placements), so the same exhaustive input goes through each of them here:

  * every (a, b) pair laid out along the reduction axis of a GEMM / the channel axis of an NHWC
    tensor, with one-hot weights, so that the int32 accumulators read back T(x) itself
    (Section 3.1: rounding carry into the next window, saturation at the top of the range;
    Section 3.2 Eq. 2: the pair rule; Section 5.1: the 6- and 4-bit lone windows for n = 3, 2);
  * the same bytes produced BY an epilogue (identity weights, unit scales) with the next
    layer's transform applied to them before the store;
  * an epilogue whose accumulators, scales, biases and output scale land on exact .5 ties, on
    both sides of 0 and 255, far outside the byte range and on NaN / +-inf.
Integer outputs are compared bit for bit, fp32 outputs bit for bit where they are numbers.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

COMBOS = [
    (4, 0x1F), (4, 0x15), (4, 0x11), (4, 0x1B), (4, 0x13),
    (3, 0x3F), (3, 0x35), (3, 0x29), (2, 0x7F), (2, 0x55), (2, 0x6B),
]
MODES = [sparq.MODE_BSPARQ, sparq.MODE_VSPARQ]


def all_pairs() -> np.ndarray:
    """131,072 bytes: (a, b) for a, b in 0..255, pairs adjacent."""
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    return np.stack([a.ravel(), b.ravel()], axis=1).reshape(-1).copy()


def gemm_acc(A, B_nk, params):
    M, N = A.shape[0], B_nk.shape[0]
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    sparq.sparq_gemm_s8(torch.from_numpy(A).cuda(), torch.from_numpy(B_nk).cuda(), params, acc_out=acc)
    sparq.sparq_check()
    return acc.cpu().numpy()


# ---- (a) consumer-side transform inside the fused kernels ---------------------------------------

@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("layout", [(1024, 128, 1), (2048, 64, 1), (16384, 128, 2), (512, 256, 1), (1365, 96, 1)])
def test_all_pairs_through_fused_gemm(n, mask, rnd, mode, layout):
    """B = `reps` stacked identities, so acc[m][j] = T(A)[m][j mod K].  1024 x 128 takes 128-byte
    reduction steps, 2048 x 64 and 1365 x 96 64-byte steps (the latter with a ragged last row tile
    and a zero-filled half step), 512 x 256 two steps per tile, and 16384 rows with 256 columns
    the 256-wide tiles."""
    M, K, reps = layout
    flat = all_pairs()
    need = M * K
    A = np.resize(flat, need).reshape(M, K)              # whole pairs stay adjacent: K is even
    B = np.concatenate([np.eye(K, dtype=np.int8)] * reps, axis=0)
    got = gemm_acc(A, B, sparq.SparqParams(mode, n, mask, rnd))
    want = oracle.transform(A, mode, n, mask, rnd).astype(np.int32)
    assert np.array_equal(got, np.concatenate([want] * reps, axis=1))


def conv_acc(x, w, stride, pad, params):
    nb, h, wd, _ = x.shape
    cout, r, s, _ = w.shape
    ho = (h + 2 * pad - r) // stride + 1
    wo = (wd + 2 * pad - s) // stride + 1
    acc = torch.full((nb, ho, wo, cout), -7, dtype=torch.int32, device="cuda")
    sparq.sparq_conv2d_nhwc_s8(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), (stride, stride), (pad, pad),
                               params, acc_out=acc)
    sparq.sparq_check()
    return acc.cpu().numpy()


def centre_tap_identity(c: int, r: int = 3, s: int = 3) -> np.ndarray:
    w = np.zeros((c, r, s, c), dtype=np.int8)
    w[np.arange(c), r // 2, s // 2, np.arange(c)] = 1
    return w


@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("c", [64, 128, 256])
def test_all_pairs_through_window_convolution(n, mask, rnd, mode, c):
    """3x3, stride 1, one-hot at the centre tap: output pixel = T(input pixel).  64 channels take
    the 64-wide resident-weight window kernel, 128 the 128-wide one, 256 two channel blocks."""
    hw = 32 if c <= 128 else 16
    nb = 131072 // (hw * hw * c)
    x = all_pairs().reshape(nb, hw, hw, c)
    got = conv_acc(x, centre_tap_identity(c), 1, 1, sparq.SparqParams(mode, n, mask, rnd))
    assert np.array_equal(got, oracle.transform(x, mode, n, mask, rnd).astype(np.int32))
    assert np.array_equal(got, oracle.conv2d_nhwc(x, centre_tap_identity(c), (1, 1), (1, 1), mode, n, mask, rnd))


@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("c", [64, 128])
def test_all_pairs_through_strided_convolution(n, mask, rnd, mode, c):
    """3x3, stride 2 (the im2col kernel): output (i, j) reads input (2i, 2j) through the centre tap,
    so the pairs sit on the even pixels and the odd pixels hold other bytes."""
    hw = 32
    nb = 131072 // (hw * hw * c)
    pairs = all_pairs().reshape(nb, hw, hw, c)
    x = np.resize(np.roll(all_pairs(), 12346), nb * 2 * hw * 2 * hw * c).reshape(nb, 2 * hw, 2 * hw, c).copy()
    x[:, ::2, ::2, :] = pairs
    w = centre_tap_identity(c)
    got = conv_acc(x, w, 2, 1, sparq.SparqParams(mode, n, mask, rnd))
    assert np.array_equal(got, oracle.transform(pairs, mode, n, mask, rnd).astype(np.int32))
    assert np.array_equal(got, oracle.conv2d_nhwc(x, w, (2, 2), (1, 1), mode, n, mask, rnd))


# ---- (b) producer-side transform of the epilogue --------------------------------------------------

@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("layout", [(1024, 128), (2048, 64), (512, 256), (4096, 32)])
def test_all_pairs_emitted_by_gemm_epilogue(n, mask, rnd, mode, layout):
    """mode NONE, identity weights, scale 1, no bias: the requantized bytes are A itself, and the
    epilogue applies the next layer's transform to them (pairs along N)."""
    M, K = layout
    A = all_pairs().reshape(M, K)
    B = np.eye(K, dtype=np.int8)
    u8 = torch.full((M, K), 9, dtype=torch.uint8, device="cuda")
    nxt = sparq.SparqParams(mode, n, mask, rnd)
    sparq.sparq_gemm_s8(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), sparq.SparqParams(sparq.MODE_NONE),
                        scale=torch.ones(K, device="cuda"), inv_out_scale=1.0, u8_out=u8, next_transform=nxt)
    sparq.sparq_check()
    assert np.array_equal(u8.cpu().numpy(), oracle.transform(A, mode, n, mask, rnd))


@pytest.mark.parametrize("n,mask", COMBOS)
@pytest.mark.parametrize("rnd", [0, 1])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("c", [64, 128])
def test_all_pairs_emitted_by_window_convolution_epilogue(n, mask, rnd, mode, c):
    hw = 32
    nb = 131072 // (hw * hw * c)
    x = all_pairs().reshape(nb, hw, hw, c)
    u8 = torch.full((nb, hw, hw, c), 9, dtype=torch.uint8, device="cuda")
    nxt = sparq.SparqParams(mode, n, mask, rnd)
    sparq.sparq_conv2d_nhwc_s8(torch.from_numpy(x).cuda(), torch.from_numpy(centre_tap_identity(c)).cuda(), (1, 1), (1, 1),
                               sparq.SparqParams(sparq.MODE_NONE), scale=torch.ones(c, device="cuda"),
                               inv_out_scale=1.0, relu=True, u8_out=u8, next_transform=nxt)
    sparq.sparq_check()
    assert np.array_equal(u8.cpu().numpy(), oracle.transform(x, mode, n, mask, rnd))


# ---- (c) epilogue: ties, clamps, NaN and infinities ---------------------------------------------

F = np.float32
SCALES = np.array([0.5, 1.0, 0.25, 1.5, 1e30, -0.5, np.nan, np.inf, -np.inf, 0.0, 2.0 ** -20, 0.125, -1.0], dtype=F)
BIASES = np.array([0.0, 0.5, -0.5, 254.5, 255.5, 1e9, np.nan, np.inf, -np.inf, -0.25, 127.5, 255.0, 1.5, -254.5, 2.5,
                   256.0, 0.49999997], dtype=F)
INVS = [1.0, 0.5, 2.0, 0.37, -1.0, float("inf"), float("nan"), 0.0]


def tie_problem(K: int, N: int, seed: int):
    """acc[m][j] = m * b_j for the first 256 rows (b_j sweeps -128..127, so every product of a byte
    and a weight occurs, odd and even), then 64 dense rows whose sums reach the accumulator's
    range for this K.  Returns A (M x K), B in the oracle's K x N orientation."""
    rng = np.random.default_rng(seed)
    M = 320
    A = np.zeros((M, K), dtype=np.uint8)
    A[:256, 0] = np.arange(256)
    A[256:300] = rng.integers(0, 256, (44, K), dtype=np.uint8)
    A[300:] = 255
    B = rng.integers(-128, 128, (K, N)).astype(np.int8)
    B[0, :] = (np.arange(N) % 256 - 128).astype(np.int8)
    B[:, N - 1] = 127            # the largest accumulators: rows of 255 times a column of 127
    B[:, N - 2] = -128
    return A, B


def same_floats(got: np.ndarray, want: np.ndarray) -> bool:
    nan_g, nan_w = np.isnan(got), np.isnan(want)
    return bool(np.array_equal(nan_g, nan_w) and np.array_equal(got[~nan_g].view(np.uint32), want[~nan_w].view(np.uint32)))


@pytest.mark.parametrize("K", [16, 128, 144, 1024])       # K <= 128: the add-based exact int -> float step
@pytest.mark.parametrize("N", [64, 256, 96])               # 64: epilogue teams; 96: a ragged last group
@pytest.mark.parametrize("mode", [sparq.MODE_NONE, sparq.MODE_VSPARQ])
@pytest.mark.parametrize("relu", [False, True])
def test_gemm_epilogue_ties_clamps_and_non_finite(K, N, mode, relu):
    A, B = tie_problem(K, N, seed=K + N)
    acc = oracle.gemm(A, B, mode, 4, 0x1F, 1)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    p = sparq.SparqParams(mode, 4, 0x1F, 1)
    for si, inv in enumerate(INVS):
        scale = np.resize(np.roll(SCALES, si), N).astype(F)
        bias = np.resize(np.roll(BIASES, 2 * si), N).astype(F)
        f_want, q_want = oracle.epilogue(acc, scale, bias, relu, inv)
        sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
        # bytes only: the straight-line path (and the teams when N <= 64)
        u8 = torch.full(acc.shape, 7, dtype=torch.uint8, device="cuda")
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (inv, "bytes only")
        # bytes and fp32: the general path
        u8.fill_(7)
        f32 = torch.full(acc.shape, -7.0, dtype=torch.float32, device="cuda")
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8, f32_out=f32)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (inv, "with fp32")
        assert same_floats(f32.cpu().numpy(), f_want), (inv, "fp32")
        # no bias
        f_nb, q_nb = oracle.epilogue(acc, scale, None, relu, inv)
        u8.fill_(7)
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, relu=relu, inv_out_scale=inv, u8_out=u8)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_nb), (inv, "no bias")


def float_bit_patterns(rng, n: int) -> np.ndarray:
    """Floats drawn over the whole format: any sign, any exponent (subnormals, infinities and NaNs
    included), plus a share near the output grid, where the rounding and the clamp decide."""
    bits = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
    f = bits.view(F).copy()
    near = rng.random(n) < 0.5
    f[near] = (rng.integers(-600, 600, n)[near] / 2.0 + rng.choice([0.0, 1e-3, -1e-3, 2.0 ** -24], n)[near]).astype(F)
    return f


@pytest.mark.parametrize("K", [16, 144])                 # add-based and converted int -> float step
@pytest.mark.parametrize("N", [64, 128, 256])
@pytest.mark.parametrize("relu", [False, True])
def test_requantization_over_arbitrary_float_bit_patterns(K, N, relu):
    # the float -> byte step is a conversion followed by a saturating pack: every float the
    # arithmetic before it can produce must come out as the oracle's clamp(rint(z), 0, 255)
    rng = np.random.default_rng([K, N, int(relu)])
    A, B = tie_problem(K, N, seed=3 * K + N)
    acc = oracle.gemm(A, B, sparq.MODE_NONE, 4, 0x1F, 1)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    p = sparq.SparqParams(sparq.MODE_NONE)
    for rep in range(6):
        scale, bias = float_bit_patterns(rng, N), float_bit_patterns(rng, N)
        inv = float(float_bit_patterns(rng, 1)[0]) if rep else 1.0
        f_want, q_want = oracle.epilogue(acc, scale, bias, relu, inv)
        u8 = torch.full(acc.shape, 7, dtype=torch.uint8, device="cuda")
        f32 = torch.full(acc.shape, -7.0, dtype=torch.float32, device="cuda")
        sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (rep, inv, "bytes only")
        u8.fill_(7)
        sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8, f32_out=f32)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (rep, inv, "with fp32")
        assert same_floats(f32.cpu().numpy(), f_want), (rep, inv, "fp32")


@pytest.mark.parametrize("K", [16, 144])
@pytest.mark.parametrize("mode", [sparq.MODE_NONE, sparq.MODE_VSPARQ])
def test_gemm_epilogue_edge_values_on_256_wide_tiles(K, mode):
    """The same accumulators repeated over 20,480 rows, so that the 256-wide tiles are chosen."""
    N = 256
    A, B = tie_problem(K, N, seed=K)
    A = np.tile(A, (64, 1))
    acc = oracle.gemm(A, B, mode, 4, 0x1F, 1)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    p = sparq.SparqParams(mode, 4, 0x1F, 1)
    for si, inv in ((0, 1.0), (3, 0.5), (5, float("nan"))):
        scale = np.resize(np.roll(SCALES, si), N).astype(F)
        bias = np.resize(np.roll(BIASES, 2 * si), N).astype(F)
        for relu in (False, True):
            f_want, q_want = oracle.epilogue(acc, scale, bias, relu, inv)
            sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
            u8 = torch.full(acc.shape, 7, dtype=torch.uint8, device="cuda")
            sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8)
            sparq.sparq_check()
            assert np.array_equal(u8.cpu().numpy(), q_want), (inv, relu, "bytes only")
            f32 = torch.full(acc.shape, -7.0, dtype=torch.float32, device="cuda")
            sparq.sparq_gemm_s8(Ad, Bd, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8, f32_out=f32)
            sparq.sparq_check()
            assert np.array_equal(u8.cpu().numpy(), q_want), (inv, relu, "with fp32")
            assert same_floats(f32.cpu().numpy(), f_want), (inv, relu, "fp32")


@pytest.mark.parametrize("cfg", [
    # c, cout, r, s: 64 -> 64 takes the 64-wide window kernel (1x2: K = 128, the add-based step),
    # 128 -> 128 and 128 -> 256 the wide ones
    (64, 64, 1, 2), (64, 64, 3, 3), (128, 128, 3, 3), (128, 256, 3, 3),
])
@pytest.mark.parametrize("relu", [False, True])
def test_window_convolution_epilogue_ties_clamps_and_non_finite(cfg, relu):
    c, cout, r, s = cfg
    rng = np.random.default_rng(c + cout + r)
    nb, h, wd = 2, 16, 32
    x = rng.integers(0, 256, (nb, h, wd, c), dtype=np.uint8)
    x[0, :8, :, 0] = np.arange(256, dtype=np.uint8).reshape(8, 32)
    x[0, :8, :, 1:] = 0
    w = np.zeros((cout, r, s, c), dtype=np.int8)
    w[:, r // 2, s // 2, 0] = (np.arange(cout) % 256 - 128).astype(np.int8)     # acc = x[p][0] * b_co on the sparse pixels
    w[:, :, :, 1:] = rng.integers(-128, 128, (cout, r, s, c - 1)).astype(np.int8)
    pad = (r // 2, s // 2)
    p = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
    acc = oracle.conv2d_nhwc(x, w, (1, 1), pad, p.mode, 4, 0x1F, 1)
    xd, wdv = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    for si, inv in enumerate(INVS):
        scale = np.resize(np.roll(SCALES, si), cout).astype(F)
        bias = np.resize(np.roll(BIASES, 2 * si), cout).astype(F)
        f_want, q_want = oracle.epilogue(acc, scale, bias, relu, inv)
        sd, bd = torch.from_numpy(scale).cuda(), torch.from_numpy(bias).cuda()
        u8 = torch.full(acc.shape, 7, dtype=torch.uint8, device="cuda")
        sparq.sparq_conv2d_nhwc_s8(xd, wdv, (1, 1), pad, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv, u8_out=u8)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (inv, "bytes only")
        u8.fill_(7)
        f32 = torch.full(acc.shape, -7.0, dtype=torch.float32, device="cuda")
        sparq.sparq_conv2d_nhwc_s8(xd, wdv, (1, 1), pad, p, scale=sd, bias=bd, relu=relu, inv_out_scale=inv,
                                   u8_out=u8, f32_out=f32)
        sparq.sparq_check()
        assert np.array_equal(u8.cpu().numpy(), q_want), (inv, "with fp32")
        assert same_floats(f32.cpu().numpy(), f_want), (inv, "fp32")


def test_tie_cases_really_occur():
    """The construction above must produce what it claims: exact .5 ties next to even and odd
    integers, values on both sides of 0 and 255, and non-finite values (checked on the oracle's
    fp32 output, so a change of the generators cannot silently empty the test)."""
    A, B = tie_problem(16, 64, seed=80)
    acc = oracle.gemm(A, B, sparq.MODE_NONE, 4, 0x1F, 1)
    scale = np.resize(SCALES, 64).astype(F)
    bias = np.resize(BIASES, 64).astype(F)
    f, q = oracle.epilogue(acc, scale, bias, False, 1.0)
    fin = f[np.isfinite(f)]
    frac = fin - np.floor(fin)
    ties = fin[(frac == 0.5) & (fin > 0) & (fin < 255)]
    assert (np.floor(ties) % 2 == 0).any() and (np.floor(ties) % 2 == 1).any()
    assert ((fin > -1) & (fin < 0)).any() and ((fin > 255) & (fin < 256)).any() and (fin > 1e6).any()
    assert np.isnan(f).any() and np.isposinf(f).any() and np.isneginf(f).any()
    assert q.min() == 0 and q.max() == 255
