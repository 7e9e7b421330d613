"""sparq_gemm_s8_static: the entry point for hosts that must not allocate device memory.

A serving process that has already handed all free device memory to its framework's pool,
or a loop that cannot afford the device-wide synchronization of an allocation, cannot use
the entry points that allocate lazily.  This one keeps its scratch (the transformed
activations and the status word) in a fixed array inside the library.  The test calls it
through the C ABI twice in a row -- the second call finds the first call's leftovers in the
shared array -- and compares every output with the existing fused entry point's and with the
CPU oracle.  A second test, in a process of its own that never touches the allocating entry
points, shows the entry point's one promise: the device's free memory is the same after a
series of calls as before it.

Collected last on purpose (file name), so that a run that stops at the first failure has
already run every other test; it passes alone in a fresh process as well.
"""
import ctypes
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq
from paper_2105_11010_b200._binding import _CEpilogue, _stream_ptr

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-6


def run_both(M, N, K, params, seed, relu):
    A_h, B_h = synth.activations(seed, (M, K), 0.5), synth.weights(seed, (N, K))
    scale_h, bias_h = synth.scales(seed, N), synth.bias(seed, N)
    A, B = torch.from_numpy(A_h).cuda(), torch.from_numpy(B_h).cuda()
    scale, bias = torch.from_numpy(scale_h).cuda(), torch.from_numpy(bias_h).cuda()
    inv = synth.inv_out_scale(K)
    acc_o = oracle.gemm(A_h, np.ascontiguousarray(B_h.T), params.mode, params.window_bits, params.placement_mask,
                        params.rounding)
    f32_o, u8_o = oracle.epilogue(acc_o, scale_h, bias_h, relu, inv)
    outs = [(acc_o, f32_o, u8_o)]
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
        (acc_o, f32_o, u8_o), (acc_f, f32_f, u8_f), (acc_s, f32_s, u8_s) = run_both(M, N, K, params, seed, relu)
        assert np.array_equal(acc_s, acc_f) and np.array_equal(acc_s, acc_o)
        assert np.array_equal(u8_s, u8_f) and np.array_equal(u8_s, u8_o)
        assert np.allclose(f32_s, f32_f, rtol=RTOL, atol=ATOL) and np.allclose(f32_s, f32_o, rtol=RTOL, atol=ATOL)


def test_epilogue_options_and_strided_weights_through_the_static_entry_point():
    """Producer-side transform, residual input and ldb > K, against the oracle."""
    M, N, K, ldb = 640, 128, 256, 320
    A_h = synth.activations(21, (M, K), 0.5)
    B_full = synth.weights(21, (N, ldb))
    B_h = np.ascontiguousarray(B_full[:, :K])
    scale_h, bias_h = synth.scales(21, N), synth.bias(21, N)
    res_h = synth.activations(22, (M, N), 0.3)
    inv = synth.inv_out_scale(K)
    P = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_3OPT, sparq.ROUND_NEAREST)
    nxt = sparq.SparqParams(sparq.MODE_VSPARQ, 3, sparq.SET_6OPT, sparq.ROUND_TRUNCATE)
    acc_o = oracle.gemm(A_h, np.ascontiguousarray(B_h.T), P.mode, P.window_bits, P.placement_mask, P.rounding)
    f_o, q_o = oracle.epilogue(acc_o, scale_h, bias_h, True, inv, residual=res_h, residual_scale=0.125)
    q_o = oracle.transform(q_o, nxt.mode, nxt.window_bits, nxt.placement_mask, nxt.rounding)
    A, Bd = torch.from_numpy(A_h).cuda(), torch.from_numpy(B_full).cuda()
    scale, bias, res = torch.from_numpy(scale_h).cuda(), torch.from_numpy(bias_h).cuda(), torch.from_numpy(res_h).cuda()
    f32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    p, n = P._c(), nxt._c()
    e = _CEpilogue(scale.data_ptr(), bias.data_ptr(), 1, inv, None, f32.data_ptr(), u8.data_ptr(), ctypes.pointer(n),
                   res.data_ptr(), 0.125)
    rc = sparq.load_library().sparq_gemm_s8_static(A.data_ptr(), K, Bd.data_ptr(), ldb, M, N, K, ctypes.byref(p),
                                                   ctypes.byref(e), _stream_ptr(None))
    assert rc == 0, sparq.sparq_last_error()
    assert np.array_equal(u8.cpu().numpy(), q_o)
    assert np.allclose(f32.cpu().numpy(), f_o, rtol=RTOL, atol=ATOL)


_NO_ALLOC_CHILD = r"""
import sys
import numpy as np, torch
sys.path.insert(0, sys.argv[1])
import sparq_synth as synth
import paper_2105_11010_b200 as sparq
torch.cuda.set_device(0)
M, N, K = 2048, 256, 512
A = torch.from_numpy(synth.activations(31, (M, K), 0.5)).cuda()
B = torch.from_numpy(synth.weights(31, (N, K))).cuda()
scale = torch.from_numpy(synth.scales(31, N)).cuda()
u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
P = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)
def call():
    sparq.sparq_gemm_s8_static(A, B, P, scale=scale, relu=True, inv_out_scale=synth.inv_out_scale(K), u8_out=u8, acc_out=acc)
call()                                   # set-up call: address look-up, device code loaded
torch.cuda.synchronize()
first = acc.clone().cpu()                # torch's own allocation, made before the snapshot
free0, _ = torch.cuda.mem_get_info()
alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
for _ in range(25):
    call()
torch.cuda.synchronize()
free1, _ = torch.cuda.mem_get_info()
assert free1 == free0, (free0, free1)
assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
assert torch.equal(acc.cpu(), first)
print("NO_ALLOC_OK", free0, free1)
"""


def test_static_calls_leave_free_device_memory_unchanged():
    """A fresh process that only ever calls the static entry point (so neither the lazily
    allocated status word nor a staging buffer of the other entry points exists): after the
    set-up call, 25 more calls leave cudaMemGetInfo's free bytes and torch's allocator counters
    exactly where they were."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _NO_ALLOC_CHILD, root], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "NO_ALLOC_OK" in r.stdout, r.stdout + r.stderr


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
