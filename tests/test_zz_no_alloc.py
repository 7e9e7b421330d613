"""sparq_gemm_s8_static: the entry point for hosts that must not allocate device memory.

A serving process that has already handed all free device memory to its framework's pool,
or a loop that cannot afford the device-wide synchronization of an allocation, cannot use
the entry points that allocate lazily.  This one keeps its scratch (the transformed
activations and the status word) in a fixed array inside the library.  The test calls it
through the C ABI twice in a row -- the second call finds the first call's leftovers in the
shared array -- and compares every output with the existing fused entry point's.

Collected last on purpose (file name), so that a run that stops at the first failure has
already run every other test; it passes alone in a fresh process as well.
"""
import ctypes

import numpy as np
import pytest
import torch

import sparq_synth as synth
import paper_2105_11010_b200 as sparq
from paper_2105_11010_b200._binding import _CEpilogue, _stream_ptr

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-6


def run_both(M, N, K, params, seed, relu):
    A = torch.from_numpy(synth.activations(seed, (M, K), 0.5)).cuda()
    B = torch.from_numpy(synth.weights(seed, (N, K))).cuda()
    scale = torch.from_numpy(synth.scales(seed, N)).cuda()
    bias = torch.from_numpy(synth.bias(seed, N)).cuda()
    inv = synth.inv_out_scale(K)
    outs = []
    for which in ("fused", "static"):
        acc = torch.full((M, N), -5, dtype=torch.int32, device="cuda")
        f32 = torch.full((M, N), -5.0, dtype=torch.float32, device="cuda")
        u8 = torch.full((M, N), 5, dtype=torch.uint8, device="cuda")
        p = params._c()
        e = _CEpilogue(scale.data_ptr(), bias.data_ptr(), int(relu), inv, acc.data_ptr(), f32.data_ptr(), u8.data_ptr())
        L = sparq.load_library()
        fn = L.sparq_gemm_s8 if which == "fused" else L.sparq_gemm_s8_static
        rc = fn(A.data_ptr(), K, B.data_ptr(), K, M, N, K, ctypes.byref(p), ctypes.byref(e), _stream_ptr(None))
        assert rc == 0, sparq.sparq_last_error()
        if which == "fused":
            sparq.sparq_check()
        # the static entry point is synchronous: its outputs are complete on return
        outs.append((acc.cpu().numpy(), f32.cpu().numpy(), u8.cpu().numpy()))
    return outs


def test_two_calls_in_a_row_match_the_fused_entry_point():
    calls = [
        (1000, 192, 1024, sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST), 11, True),
        (300, 100, 400, sparq.SparqParams(sparq.MODE_BSPARQ, 3, sparq.SET_6OPT, sparq.ROUND_TRUNCATE), 12, False),
    ]
    for M, N, K, params, seed, relu in calls:      # the second call reuses the shared scratch
        (acc_f, f32_f, u8_f), (acc_s, f32_s, u8_s) = run_both(M, N, K, params, seed, relu)
        assert np.array_equal(acc_s, acc_f)
        assert np.array_equal(u8_s, u8_f)
        assert np.allclose(f32_s, f32_f, rtol=RTOL, atol=ATOL)


def test_sizes_beyond_the_static_scratch_are_rejected():
    K = 4096
    M = sparq.STATIC_SCRATCH_BYTES // K + 1
    A = torch.zeros((M, K), dtype=torch.uint8, device="cuda")
    B = torch.zeros((16, K), dtype=torch.int8, device="cuda")
    acc = torch.zeros((M, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_gemm_s8_static(A, B, sparq.SparqParams(), acc_out=acc)
    assert ei.value.code == -2 and "static scratch" in str(ei.value)
    # exactly at the limit is accepted
    M = sparq.STATIC_SCRATCH_BYTES // K
    sparq.sparq_gemm_s8_static(A[:M], B, sparq.SparqParams(), acc_out=acc[:M])
    assert int(acc[:M].abs().sum()) == 0
