"""The give-up path of the bounded device-side waits, exercised without endangering the GPU.

Every wait inside the fused kernels has a limit (about a second); their barriers always
complete, so that path cannot be reached on demand.  `sparq_selftest_wait_timeout` launches a
one-CTA kernel built from the same wait / abort-flag / tensor-memory code that waits, with a
limit of a few microseconds, on a barrier nothing arrives on.  The kernel returns normally;
nothing traps, faults or spins without a limit."""
import numpy as np
import pytest
import torch

import oracle
import sparq_synth as synth
import paper_2105_11010_b200 as sparq

pytestmark = pytest.mark.gpu

VS = sparq.SparqParams(sparq.MODE_VSPARQ, 4, sparq.SET_5OPT, sparq.ROUND_NEAREST)


def small_gemm_matches_oracle(entry):
    M, N, K = 500, 128, 256
    A, B = synth.activations(70, (M, K), 0.5), synth.weights(70, (N, K))
    scale = synth.scales(70, N)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    u8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    entry(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), VS, scale=torch.from_numpy(scale).cuda(), relu=True,
          inv_out_scale=synth.inv_out_scale(K), acc_out=acc, u8_out=u8)
    want = oracle.gemm(A, np.ascontiguousarray(B.T), VS.mode, 4, 0x1F, 1)
    return np.array_equal(acc.cpu().numpy(), want) and \
        np.array_equal(u8.cpu().numpy(), oracle.epilogue(want, scale, None, True, synth.inv_out_scale(K))[1])


def test_expired_wait_is_reported_once_and_the_library_keeps_working():
    sparq.sparq_check()                                   # start from a clean status word
    report = torch.zeros(4, dtype=torch.int32, device="cuda")
    limit = 200000
    sparq.sparq_selftest_wait_timeout(limit, report)
    with pytest.raises(sparq.SparqError) as ei:
        sparq.sparq_check()
    assert ei.value.code == -4 and "wait expired" in str(ei.value)
    gave_up, left_by_abort, waited, finished = report.cpu().tolist()
    assert finished == 1                                  # the kernel ran to its normal end (and freed its tensor memory)
    assert gave_up == 1 and left_by_abort == 1
    # the second waiter's own limit was 1000 x longer: it left because the CTA's abort flag was raised
    assert waited < 500 * limit
    sparq.sparq_check()                                   # reported once; the word is clean again
    # ordinary work on the same stream still passes its parity check (tensor memory was given back)
    assert small_gemm_matches_oracle(sparq.sparq_gemm_s8)
    sparq.sparq_check()


def test_static_entry_point_reports_and_clears_its_own_status_word():
    assert small_gemm_matches_oracle(sparq.sparq_gemm_s8_static)     # also the set-up call
    report = torch.zeros(4, dtype=torch.int32, device="cuda")
    sparq.sparq_selftest_wait_timeout(5000, report, use_static_word=True)
    torch.cuda.synchronize()
    assert report.cpu().tolist()[3] == 1
    sparq.sparq_check()                                   # the library-wide word is untouched
    # the static entry point reads its own word after its kernels: it finds the bit, reports it ...
    with pytest.raises(sparq.SparqError) as ei:
        small_gemm_matches_oracle(sparq.sparq_gemm_s8_static)
    assert ei.value.code == -4
    # ... and has cleared it: the next call is clean and correct
    assert small_gemm_matches_oracle(sparq.sparq_gemm_s8_static)


def test_limits_outside_the_allowed_range_are_refused():
    report = torch.zeros(4, dtype=torch.int32, device="cuda")
    for bad in (0, 999, 10**9):
        with pytest.raises(sparq.SparqError) as ei:
            sparq.sparq_selftest_wait_timeout(bad, report)
        assert ei.value.code == -1
    sparq.sparq_check()
