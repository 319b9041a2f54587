"""GPU test of mofq_tensor_error_noalloc, the entry point for callers that cannot allocate.

A host program that has given all device memory to its own pool, or a plug-in that must not grow
its process, cannot hand the library a workspace.  The variant under test keeps its scratch in a
fixed array inside the library, so it must (a) give the same numbers as mofq_tensor_error and
(b) not be confused by what the previous call left in that shared array.  This file is named so
that pytest collects it last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import binding as B
from paper_2305_12356_b200 import inputs

pytestmark = pytest.mark.gpu

MSE_RTOL = 1e-5


def _weights(dev, rows, cols, kind, seed, layer):
    w = torch.empty((rows, cols), dtype=torch.float16, device=dev)
    return inputs.device_weight(w, kind, seed, layer)


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row():
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    cands = ["INT4", "FP4_E2M1"]
    a = _weights(dev, 300, 1152, "student_t", 41, 0)
    b = _weights(dev, 77, 6656, "laplace", 42, 1)          # different shape, kernel and granularities
    b[5, 9] = float("inf")                                  # second call must report its own status ...
    cases = [(a, "group", None), (b, "channel", "group")]
    # preallocated outputs: nothing is allocated between the two calls under test
    outs = [torch.empty(2, dtype=torch.float32, device=dev), torch.empty((2, 2), dtype=torch.float32, device=dev)]
    stats = [torch.full((1,), -1, dtype=torch.int32, device=dev) for _ in cases]
    for (x, g1, g2), o, s in zip(cases, outs, stats):       # two calls in a row through the C ABI
        mofq.tensor_error_noalloc(x, cands, g1, gran2=g2, group=128, mse_out=o, status_out=s)
    torch.cuda.synchronize()
    for (x, g1, g2), o, s in zip(cases, outs, stats):
        want, want_status = mofq.tensor_error(x, cands, g1, gran2=g2, group=128)
        torch.cuda.synchronize()
        assert int(s.item()) == int(want_status.item())
        if int(s.item()) == 0:
            assert torch.allclose(o, want, rtol=MSE_RTOL, atol=0.0)
    assert int(stats[0].item()) == 0                        # ... and the first call's status stays clean
    assert int(stats[1].item()) & B.STATUS_NONFINITE_INPUT
    # a third call after the flagged one starts from a clean status again
    o3, s3 = mofq.tensor_error_noalloc(a, cands, "channel")
    want3, _ = mofq.tensor_error(a, cands, "channel")
    torch.cuda.synchronize()
    assert int(s3.item()) == 0 and torch.allclose(o3, want3, rtol=MSE_RTOL, atol=0.0)


def test_noalloc_matches_the_oracle_and_takes_the_large_tensor_route(orc):
    """The numbers are checked against the CPU oracle directly (not only against the sibling entry point), and a dense
    tensor of more than 32 Mi elements with group scales goes through the persistent multi-tensor kernel, whose work
    table, partial sums and status words then all live inside the built-in scratch; a small call right after it
    must not see what that left behind."""
    dev = torch.device("cuda:0")
    cands = ["INT4", "FP4_E2M1"]
    fm = [orc.INT4, orc.FP4_E2M1]
    small = _weights(dev, 96, 1152, "laplace", 44, 0)
    big = _weights(dev, 8192, 8192, "student_t", 45, 1)      # 64 Mi elements = 128 MiB of fp16
    o_big = torch.empty(2, dtype=torch.float32, device=dev)
    o_small = torch.empty((2, 2), dtype=torch.float32, device=dev)
    s_big = torch.full((1,), -1, dtype=torch.int32, device=dev)
    s_small = torch.full((1,), -1, dtype=torch.int32, device=dev)
    mofq.tensor_error_noalloc(big, cands, "group", group=128, mse_out=o_big, status_out=s_big)
    mofq.tensor_error_noalloc(small, cands, "channel", gran2="group", group=128, mse_out=o_small, status_out=s_small)
    torch.cuda.synchronize()
    assert int(s_big.item()) == 0 and int(s_small.item()) == 0
    rows = torch.arange(0, 8192, 37)                          # the oracle scores a row sample of the large tensor ...
    sample = big[rows.to(dev)].contiguous()
    got_sample, _ = mofq.tensor_error(sample, cands, "group", group=128)
    want_sample = [orc.tensor_mse(sample.cpu(), f, orc.PER_GROUP, 128) for f in fm]
    assert np.allclose(got_sample.cpu().numpy(), want_sample, rtol=MSE_RTOL, atol=0)
    want_big, _ = mofq.tensor_error(big, cands, "group", group=128)      # ... and the whole of it must agree with the workspace path
    assert torch.allclose(o_big, want_big, rtol=MSE_RTOL, atol=0.0)
    want_small = [[orc.tensor_mse(small.cpu(), f, g, 128) for f in fm] for g in (orc.PER_CHANNEL, orc.PER_GROUP)]
    assert np.allclose(o_small.cpu().numpy(), want_small, rtol=MSE_RTOL, atol=0)


def test_noalloc_rejects_tensors_beyond_its_limit():
    L = mofq.lib()
    assert L.mofq_noalloc_scratch_bytes() >= L.mofq_tensor_workspace_bytes(None)
    too_big = B.MofqTensor(0x10000, B.F16, 0, 1 << 16, 1 << 16, 1 << 16)      # 2^32 elements; never dereferenced
    fm = (C.c_int32 * 2)(B.INT4, B.FP4_E2M1)
    rc = L.mofq_tensor_error_noalloc(C.byref(too_big), fm, 2, B.PER_CHANNEL, B.GRAN_NONE, 0, 0x20000, None, None)
    assert rc == -6 and b"scratch" in L.mofq_status_string(rc)
