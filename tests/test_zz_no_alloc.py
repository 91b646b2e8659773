"""The no-allocation entry point against the workspace-based one and the oracle (GPU).

compass_gemm_rs_sequential_noalloc exists for callers that cannot give the
library a workspace because all device memory is already spoken for, or that
cannot afford cudaMalloc's device-wide synchronisation.  Its scratch is a
built-in device array shared by all calls, which keeps the previous call's
contents.  The checks: calls in a row (each sees the previous one's leftovers,
and uses a different shape) must each reproduce, bit for bit, what
compass_decomp with d = 1 computes with a caller-provided workspace, and match
the CPU oracle within the acceptance rule of the other parity tests; the
device's free memory (as the driver reports it) and torch's allocator
statistics must not change across the call; the status left in the built-in
array must read back as OK; a problem beyond the array's size must be refused.

This file is collected last on purpose: a failure here cannot hide another.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import compare
from oracle import operators as ops
from paper_2609_10549_b200 import api
from paper_2609_10549_b200 import workloads as wl
from tests import gpu_util as gu


def _run_pair(w):
    A_bits, B_bits = wl.make_inputs(w)
    A, B = gu.device_inputs(A_bits, B_bits)
    # reference: the existing entry point with a caller-provided workspace
    ref, status, guards = gu.run_decomp(w, A_bits, B_bits, d=1, two_streams=False)
    assert status == (api.OK, 0) and guards
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    pr = gu.problem_of(w)
    # The first use on a device resolves the array's address; with CUDA's lazy module loading that is also
    # when the driver reserves the array's memory.  That one-time set-up is not the call's own doing, so it
    # is triggered here, before free memory is compared.
    api.compass_noalloc_read_status()
    torch.cuda.synchronize()
    before = torch.cuda.memory_stats()["allocation.all.allocated"]
    free_before = torch.cuda.mem_get_info()[0]          # the driver's own count: sees a cudaMalloc inside the library
    api.compass_gemm_rs_sequential_noalloc(pr, A, B, [o.view for o in outs])
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    after = torch.cuda.memory_stats()["allocation.all.allocated"]
    assert after == before, "the call went through torch's allocator"
    assert free_after == free_before, "the device's free memory changed across the call"
    assert api.compass_noalloc_read_status() == (api.OK, 0)
    assert all(o.guards_intact() for o in outs)
    oracle = ops.gemm_rs(A_bits, B_bits)
    for r in range(w.P):
        # same kernels, same order of additions: identical bits
        assert np.array_equal(outs[r].bits(), ref[r]), f"rank {r} differs from compass_decomp(d=1)"
        # and the oracle, within the tolerance of the other parity tests (1e-2*max|ref| + 1e-3 per element)
        rep = compare.check(outs[r].bits(), oracle[r])
        assert rep.ok, f"rank {r} against the oracle: {rep}"


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_point():
    first = wl.Workload("noalloc-1", wl.OP_GEMM_RS, P=4, M=2048, N=520, K=344, b_dist=("normal", 0.05), seed=11)
    second = wl.Workload("noalloc-2", wl.OP_GEMM_RS, P=2, M=512, N=264, K=200, b_dist=("normal", 0.05), seed=12)
    _run_pair(first)
    _run_pair(second)      # starts from the first call's leftovers in the shared array
    _run_pair(first)


@pytest.mark.gpu
def test_refuses_problems_beyond_the_builtin_array():
    lib = api.lib()
    big = api.make_problem(api.OP_GEMM_RS, 8, 8192, 4096, 1376)       # 8 partials of 64 MiB
    ptrs = (C.c_void_p * 8)(*[0x1000 * (i + 1) for i in range(8)])
    assert lib.compass_gemm_rs_sequential_noalloc(C.byref(big), ptrs, ptrs, ptrs, None) == api.ERR_SCRATCH_LIMIT
    assert "built-in scratch" in api.status_string(api.ERR_SCRATCH_LIMIT)
    ag = api.make_problem(api.OP_AG_GEMM, 2, 512, 256, 128)
    assert lib.compass_gemm_rs_sequential_noalloc(C.byref(ag), ptrs, ptrs, ptrs, None) == api.ERR_INVALID_ARG
    bad = api.make_problem(api.OP_GEMM_RS, 2, 514, 256, 128)
    assert lib.compass_gemm_rs_sequential_noalloc(C.byref(bad), ptrs, ptrs, ptrs, None) == api.ERR_SHAPE
