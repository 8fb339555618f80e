"""The allocation-free campaign entry point against the ordinary one.

mpgemmfi_campaign_static serves callers that may not allocate device memory (plugins running
inside another program's pipeline, services whose memory pools are frozen after start-up):
its trial schedule sits in an array built into the library instead of a caller-provided
workspace. Every call on a device reuses that one array, so the test makes two calls in a row
with different trial tables -- the second smaller than the first -- and checks that each gives
exactly the records and the clean product that mpgemmfi_campaign gives for the same inputs.
Both entry points run the same kernels, so records agree bit for bit; the clean product is
compared within the tolerance of the other parity tests.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test. It also passes on its own in a fresh process.
"""
import numpy as np
import pytest
import torch

import paper_2311_05782_b200 as mpg
import synth

pytestmark = pytest.mark.gpu


def _run_both(w, sites):
    M, N, K = w.M, w.N, w.K
    n = len(sites)
    view = np.int32 if w.dtype == synth.DTYPE_TF32 else np.int16
    a = torch.from_numpy(w.A.view(view)).cuda()
    b = torch.from_numpy(w.Bt.view(view)).cuda()
    s = torch.from_numpy(np.ascontiguousarray(sites).view(np.int32).reshape(n, 8)).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    # every buffer is allocated here, before the call under test, which itself must allocate nothing
    c_ref = torch.empty((M, N), dtype=torch.float32, device="cuda")
    c_new = torch.empty((M, N), dtype=torch.float32, device="cuda")
    r_ref = torch.zeros((n, 12), dtype=torch.int32, device="cuda")
    r_new = torch.full((n, 12), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(mpg.mpgemmfi_campaign_workspace_bytes(w.dtype, M, N, K, n), dtype=torch.uint8, device="cuda")
    rc = mpg.mpgemmfi_campaign(w.dtype, M, N, K, a.data_ptr(), b.data_ptr(), c_ref.data_ptr(), s.data_ptr(), n,
                               w.detect_mode, r_ref.data_ptr(), ws.data_ptr(), ws.numel(), stream)
    assert rc == 0
    torch.cuda.synchronize()

    def call_static():
        rc = mpg.mpgemmfi_campaign_static(w.dtype, M, N, K, a.data_ptr(), b.data_ptr(), c_new.data_ptr(), s.data_ptr(), n,
                                          w.detect_mode, r_new.data_ptr(), stream)
        assert rc == 0
        torch.cuda.synchronize()

    # A first call does the one-time set-up (address look-up, kernel attributes, lazy loading of the kernels by the
    # driver). The call after it is the one measured: the device's free memory as the driver reports it
    # (cudaMemGetInfo) must not move, which would show a cudaMalloc inside the library; torch's own counter, which
    # only sees torch's allocator, is checked beside it.
    call_static()
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    call_static()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, f"device free memory moved by {free_before - free_after} bytes during the call"
    assert torch.cuda.memory_allocated() == torch_before
    return c_ref.cpu().numpy(), r_ref.cpu().numpy(), c_new.cpu().numpy(), r_new.cpu().numpy()


def test_static_campaign_matches_campaign_on_two_calls_in_a_row():
    # first call: a mixed table (operand, accumulator and output sites) that fills all three lists
    w1 = synth.make_workload("c5", 2048, 64, 576, trials=500)
    # second call: fewer trials of another mix on another shape, so leftovers of call one would show
    w2 = synth.make_workload("c2", 384, 512, 256, trials=90)
    for w in (w1, w2):
        c_ref, r_ref, c_new, r_new = _run_both(w, w.sites)
        assert np.array_equal(r_new, r_ref), "records differ from mpgemmfi_campaign"
        scale = np.abs(c_ref).max()
        assert np.all(np.abs(c_new - c_ref) <= 1e-3 * scale)
        rec = r_new.view(np.uint32).reshape(-1).view(mpg.RECORD_DTYPE)
        assert np.array_equal(rec["kind"], w.sites["kind"]) and (rec["n_affected"] > 0).all()


def test_static_campaign_refuses_more_trials_than_its_array_holds():
    w = synth.make_workload("c1", 128, 128, 64, trials=4)
    a = torch.from_numpy(w.A.view(np.int16)).cuda()
    b = torch.from_numpy(w.Bt.view(np.int16)).cuda()
    c = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    s = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    r = torch.zeros((4, 12), dtype=torch.int32, device="cuda")
    too_many = mpg.STATIC_MAX_TRIALS + 1
    rc = mpg.mpgemmfi_campaign_static(w.dtype, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), s.data_ptr(),
                                      too_many, w.detect_mode, r.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == -5 and "workspace" in mpg.mpgemmfi_strerror(rc)
    torch.cuda.synchronize()
