"""Producer-side SPARQ: the epilogue of one layer emits T(activations) for the next layer.

T depends on the activations only (Section 3 of the paper), so applying it where the
activations are produced and running the consumer with mode NONE must give exactly what
the consumer computes when it applies T itself.  The oracle side is a composition of the
existing oracle functions: epilogue, then transform along the channel axis."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

NEXT = [
    sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1),
    sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x15, 0),
    sparq.SparqParams(sparq.MODE_VSPARQ, 3, 0x3F, 1),
    sparq.SparqParams(sparq.MODE_BSPARQ, 2, 0x7F, 1),
]


@pytest.mark.parametrize("nxt", NEXT)
@pytest.mark.parametrize("shape", [(300, 64, 192), (1000, 200, 128), (129, 512, 64)])
def test_gemm_epilogue_emits_transformed_activations(nxt, shape):
    M, N, K = shape
    A = synth.activations(M, (M, K), 0.5)
    B = synth.weights(N, (K, N))
    scale, bias = synth.scales(K, N), synth.bias(K, N)
    inv = synth.inv_out_scale(K)
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    sparq.sparq_gemm_s8(torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(B.T)).cuda(),
                        sparq.SparqParams(), scale=torch.from_numpy(scale).cuda(), bias=torch.from_numpy(bias).cuda(),
                        relu=True, inv_out_scale=inv, acc_out=acc, u8_out=u8, next_transform=nxt)
    sparq.sparq_check()
    want_acc = oracle.gemm(A, B, 2, 4, 0x1F, 1)
    _, q = oracle.epilogue(want_acc, scale, bias, True, inv)
    want = oracle.transform(q, nxt.mode, nxt.window_bits, nxt.placement_mask, nxt.rounding)
    assert np.array_equal(acc.cpu().numpy(), want_acc)        # raw accumulators are unaffected
    assert np.array_equal(u8.cpu().numpy(), want)


def conv(x, w, pad, params, scale, bias, inv, nxt=None):
    nb, h, wd, _ = x.shape
    cout = w.shape[0]
    out = torch.zeros((nb, h, wd, cout), dtype=torch.uint8, device="cuda")
    sparq.sparq_conv2d_nhwc_s8(x, w, (1, 1), (pad, pad), params, scale=scale, bias=bias, relu=True,
                               inv_out_scale=inv, u8_out=out, next_transform=nxt)
    return out


def test_chain_producer_side_equals_consumer_side():
    # 1x1 -> 3x3 -> 1x1; variant A: every consumer applies vSPARQ itself;
    # variant B: each producer emits T(output) and the consumers run with mode NONE.
    P = sparq.SparqParams(sparq.MODE_VSPARQ, 4, 0x1F, 1)
    none = sparq.SparqParams(sparq.MODE_NONE)
    nb, hw, cin, mid = 4, 28, 256, 64
    x = torch.from_numpy(synth.activations(9, (nb, hw, hw, cin), 0.5)).cuda()
    layers = []
    for i, (cout, r, c, pad) in enumerate([(mid, 1, cin, 0), (mid, 3, mid, 1), (cin, 1, mid, 0)]):
        w = torch.from_numpy(synth.weights(90 + i, (cout, r, r, c))).cuda()
        sc = torch.from_numpy(synth.scales(90 + i, cout)).cuda()
        bi = torch.from_numpy(synth.bias(90 + i, cout)).cuda()
        layers.append((w, pad, sc, bi, synth.inv_out_scale(r * r * c)))
    a = x
    for w, pad, sc, bi, inv in layers:
        a = conv(a, w, pad, P, sc, bi, inv)
    tx = torch.empty_like(x)
    sparq.sparq_quantize(x, tx, nb * hw * hw, cin, P)              # the chain's input is transformed once
    b = tx
    for i, (w, pad, sc, bi, inv) in enumerate(layers):
        last = i == len(layers) - 1
        b = conv(b, w, pad, none, sc, bi, inv, nxt=None if last else P)
    sparq.sparq_check()
    assert torch.equal(a, b)


def test_rejected_next_transform():
    A = torch.zeros((128, 64), dtype=torch.uint8, device="cuda")
    B = torch.zeros((18, 64), dtype=torch.int8, device="cuda")
    sc = torch.ones(18, device="cuda")
    u8 = torch.zeros((128, 18), dtype=torch.uint8, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:                    # N not a multiple of 4
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), scale=sc, u8_out=u8, next_transform=NEXT[0])
    assert ei.value.code == -2
    B = torch.zeros((16, 64), dtype=torch.int8, device="cuda")
    acc = torch.zeros((128, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError):                          # no u8 output to transform
        sparq.sparq_gemm_s8(A, B, sparq.SparqParams(), acc_out=acc, next_transform=NEXT[0])
