"""adloco_norm_test_noalloc: the norm test for callers that cannot allocate
device memory where the test runs (a frozen allocator pool inside a training
step, a spent device-memory budget).  Its reduction scratch is a device array
built into the library, so the call needs no context and no cudaMalloc.

Checked here against the fp64 oracle and against adloco_norm_test on the same
inputs, twice in a row (the second call finds the first call's leftovers in the
shared array); also on a side stream, on rows that do not start on a 16-byte
boundary, and for what the entry point is for: device memory in use does not
move across its calls.  The file
name sorts last on purpose: a failure here cannot hide any other test from a
run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_F32, assert_test_result, rel_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _same(a, b):
    assert a.device_status == 0 and b.device_status == 0
    assert a.batch_count == b.batch_count
    for f in ("sum_sqnorm", "mean_sqnorm", "variance", "stat"):
        assert rel_close(getattr(a, f), getattr(b, f), TOL_F32), (f, getattr(a, f), getattr(b, f))
    # same kernel, same reduction order: the decisions agree exactly unless the grid differs,
    # in which case the statistic may move in the last bits across an integer
    if abs(b.stat - round(b.stat)) > 2 * TOL_F32 * abs(b.stat):
        assert (a.b_req, a.flags, a.accum_steps, a.b_micro) == (b.b_req, b.flags, b.accum_steps, b.b_micro)


def test_noalloc_matches_the_context_entry_point_twice_in_a_row():
    torch.cuda.set_device(0)
    ctx = A.Context(0)
    res_dev = torch.zeros(A.TestResult_size(), dtype=torch.uint8, device=DEV)
    res_host = torch.zeros(A.TestResult_size(), dtype=torch.uint8).pin_memory()
    cases = [(16, 300001, 0.5), (64, (1 << 18) + 8, 0.25), (3, 4099, 1.0), (1, 1000, 0.5)]
    for rep in range(2):                                  # two full passes: every call after the first
        for B, P, eta in cases:                           # starts from a used scratch array
            G = W.per_sample_grads(B, P, sigma=0.5, seed=40 + B + rep, device=DEV)
            p = A.make_params(eta, b_cur=B, b_max=32)
            n_ref = torch.zeros(B, device=DEV)
            ref = ctx.norm_test(G, p, per_sample_sqnorm=n_ref)
            n = torch.full((B,), -1.0, device=DEV)
            got = A.norm_test_noalloc(G, p, res_dev, res_host, per_sample_sqnorm=n)
            _same(got, ref)
            assert torch.allclose(n, n_ref, rtol=TOL_F32, atol=0)
            ora = O.norm_test(W.to_numpy(G), eta=eta, b_cur=B, b_max=32)
            assert_test_result(got, ora, p, TOL_F32, what=f"noalloc B={B} P={P}")
            assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32, atol=0)
            again = A.norm_test_noalloc(G, p, res_dev, res_host, per_sample_sqnorm=n)
            assert (again.stat, again.sum_sqnorm, again.b_req) == (got.stat, got.sum_sqnorm, got.b_req)
    ctx.close()


def test_noalloc_side_stream_unaligned_rows_and_no_growth_of_device_memory():
    torch.cuda.set_device(0)
    res_dev = torch.zeros(A.TestResult_size(), dtype=torch.uint8, device=DEV)
    res_host = torch.zeros(A.TestResult_size(), dtype=torch.uint8).pin_memory()
    wide = W.per_sample_grads(12, 50003, sigma=0.5, seed=9, device=DEV)
    G = wide[:, 1:]                                       # rows start 4 bytes past a 16-byte boundary, odd pitch
    n = torch.zeros(12, device=DEV)
    p = A.make_params(0.5, b_cur=12, b_max=32)
    ora = O.norm_test(W.to_numpy(G), eta=0.5, b_cur=12, b_max=32)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    A.norm_test_noalloc(G, p, res_dev, res_host, per_sample_sqnorm=n, stream=side)     # first call: set-up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        got = A.norm_test_noalloc(G, p, res_dev, res_host, per_sample_sqnorm=n, stream=side)
        assert_test_result(got, ora, p, TOL_F32, what="noalloc on a side stream, unaligned rows")
        assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32, atol=0)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0          # nothing was allocated on the device
    with pytest.raises(A.AdlocoError) as e:
        A.norm_test_noalloc(G.double(), p, res_dev, res_host)
    assert e.value.status == A.ERR_UNSUPPORTED


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    torch.cuda.set_device(0)
    res_dev = torch.zeros(A.TestResult_size(), dtype=torch.uint8, device=DEV)
    res_host = torch.zeros(A.TestResult_size(), dtype=torch.uint8).pin_memory()
    G = torch.zeros(65, 128, device=DEV)
    with pytest.raises(A.AdlocoError) as e:
        A.norm_test_noalloc(G, A.make_params(0.5), res_dev, res_host)
    assert e.value.status == A.ERR_UNSUPPORTED
    with pytest.raises(A.AdlocoError) as e:
        A.norm_test_noalloc(G[:4], A.make_params(-1.0), res_dev, res_host)
    assert e.value.status == A.ERR_INVALID_ARG
