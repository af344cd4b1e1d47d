"""The library enqueues on the caller's stream and keeps contexts independent:
calls on a non-default stream, two contexts side by side, and results that are
only read after the stream has been synchronised."""
import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_BF16, TOL_F32, assert_test_result

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_non_default_stream_and_two_contexts():
    c1, c2 = A.Context(0), A.Context(0)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    G1 = W.per_sample_grads(16, 1 << 18, seed=1, device=DEV)
    G2 = W.per_sample_grads(32, 1 << 17, sigma=1.0, mean_scale="raw", seed=2, device=DEV)
    X, D = W.linear_layer(4, 256, 128, 256, seed=3, device=DEV)
    n = torch.zeros(4, device=DEV)
    S = torch.zeros(256, 128, device=DEV)
    torch.cuda.synchronize()
    p1, p2 = A.make_params(0.5, b_cur=16, b_max=32), A.make_params(0.5, b_cur=32, b_max=32)
    with torch.cuda.stream(s1):
        c1.norm_test(G1, p1, stream=s1, sync=False)
        c1.linear_sqnorm(X, D, n, grad_sum=S, method="direct", stream=s1)
    with torch.cuda.stream(s2):
        c2.norm_test(G2, p2, stream=s2, sync=False)
    r1, r2 = c1._read_result(s1), c2._read_result(s2)
    assert_test_result(r1, O.norm_test(W.to_numpy(G1), eta=0.5, b_cur=16, b_max=32), p1, TOL_F32, what="stream 1")
    assert_test_result(r2, O.norm_test(W.to_numpy(G2), eta=0.5, b_cur=32, b_max=32), p2, TOL_F32, what="stream 2")
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    c1.close()
    c2.close()


def test_layers_of_one_micro_batch_on_two_streams_add_into_the_same_norms():
    """The per-layer entry points use no context workspace: layers issued alternately on two streams
    (every route, an embedding and a bias among them) add into one n vector atomically and each into
    its own sum buffer; every launch that draws work from a counter gets a counter of its own."""
    c = A.Context(0)
    s = [torch.cuda.Stream(), torch.cuda.Stream()]
    B, T = 6, 384
    shapes = [(128, 256), (256, 128), (64, 512), (512, 64), (128, 128), (256, 256), (72, 264), (264, 72)]
    methods = ["pair", "gram_pair", "direct", "gram", "auto", "pair", "gram_pair", "direct"]
    data = [W.linear_layer(B, T, di, do, seed=40 + l, device=DEV) for l, (di, do) in enumerate(shapes)]
    sums = [torch.full((do, di), 9.0, device=DEV) for di, do in shapes]
    g = torch.Generator(device=DEV)
    g.manual_seed(7)
    ids = torch.randint(0, 50, (B, T), generator=g, device=DEV, dtype=torch.int32)
    n = torch.zeros(B, device=DEV)
    Sb = torch.full((256,), 9.0, device=DEV)
    torch.cuda.synchronize()
    for l, ((X, D), S, m) in enumerate(zip(data, sums, methods)):
        with torch.cuda.stream(s[l & 1]):
            c.linear_sqnorm(X, D, n, accumulate_norms=True, grad_sum=S, method=m, stream=s[l & 1])
    with torch.cuda.stream(s[0]):
        c.embedding_sqnorm(ids, data[0][1], 50, n, accumulate_norms=True, stream=s[0])
    with torch.cuda.stream(s[1]):
        c.vector_param_sqnorm(data[0][1], n, accumulate_norms=True, grad_sum=Sb, stream=s[1])
    torch.cuda.synchronize()
    assert c.device_status() == 0
    n_ref = np.zeros(B)
    for (X, D), S in zip(data, sums):
        n_l, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
        n_ref += n_l
        assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    n_ref += O.embedding_terms(ids.cpu().numpy(), W.to_numpy(data[0][1]), 50)[0]
    nb, Sb_ref = O.vector_param_terms(W.to_numpy(data[0][1]))
    n_ref += nb
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16), n.cpu().numpy() / n_ref
    assert np.allclose(Sb.cpu().numpy(), Sb_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(Sb_ref).max() * 0.05)
    c.close()


def test_bad_device_index_is_an_error_not_a_crash():
    with pytest.raises(A.AdlocoError) as e:
        A.Context(4096)
    assert e.value.status == A.ERR_CUDA


def test_empty_inputs_are_argument_errors_and_launch_nothing():
    """Zero-sized problems (no samples, no parameters, no tokens, no instances) are
    rejected on the host; nothing is enqueued."""
    import ctypes as C
    c = A.Context(0)
    lib, h = c.lib, c.h
    buf = torch.zeros(1024, device=DEV)
    bfb = torch.zeros(1024, device=DEV, dtype=torch.bfloat16)
    p = A.make_params(0.5)
    before = c.launch_count
    vp = C.c_void_p
    d, b = vp(buf.data_ptr()), vp(bfb.data_ptr())
    res = vp(c._res_dev.data_ptr())
    assert lib.adloco_norm_test(h, d, A.F32, 0, 16, 16, C.byref(p), None, None, None, res, None, None) == A.ERR_INVALID_ARG
    assert lib.adloco_norm_test(h, d, A.F32, 4, 0, 0, C.byref(p), None, None, None, res, None, None) == A.ERR_INVALID_ARG
    assert lib.adloco_norm_test(h, d, A.F32, 4, 16, 8, C.byref(p), None, None, None, res, None, None) == A.ERR_INVALID_ARG  # pitch < P
    assert lib.adloco_norm_test(h, None, A.F32, 4, 16, 16, C.byref(p), None, None, None, res, None, None) == A.ERR_INVALID_ARG
    assert lib.adloco_gram_sqnorm(h, b, b, 0, 8, 8, 8, d, 0, None, 0, None) == A.ERR_INVALID_ARG
    assert lib.adloco_gram_sqnorm(h, b, b, 2, 0, 8, 8, d, 0, None, 0, None) == A.ERR_INVALID_ARG
    assert lib.adloco_linear_sqnorm(h, b, b, 2, 8, 0, 8, d, 0, None, 0, 0, None) == A.ERR_INVALID_ARG
    assert lib.adloco_vector_param_sqnorm(h, b, None, 2, 0, 8, d, 0, None, 0, None) == A.ERR_INVALID_ARG
    arr = (vp * 1)(buf.data_ptr())
    assert lib.adloco_outer_step(h, arr, A.F32, 0, 16, d, d, d, d, 0.7, 0.9, 1, None, None) == A.ERR_INVALID_ARG
    assert lib.adloco_outer_step(h, arr, A.F32, 1, 0, d, d, d, d, 0.7, 0.9, 1, None, None) == A.ERR_INVALID_ARG
    w = (C.c_int64 * 1)(0)
    assert lib.adloco_merge(h, arr, w, A.F32, 1, 16, d, None, None) == A.ERR_INVALID_ARG      # weight 0
    assert c.launch_count == before
    c.close()


def test_host_copy_of_the_result_in_page_locked_and_in_pageable_memory():
    """result_host in page-locked memory is written by the kernel itself; in pageable memory it is
    filled by a copy on the stream.  Both hold the decision once the stream is synchronised, for
    the norm test, the re-decision from stored sums and the accumulator's final test."""
    import ctypes as C
    import oracle.adloco_oracle as O
    from parity import TOL_F32, assert_test_result
    c = A.Context(0)
    G = W.per_sample_grads(16, (1 << 16) + 4, sigma=0.5, seed=1, device=DEV)
    p = A.make_params(0.5, b_cur=16, b_max=32)
    ora = O.norm_test(W.to_numpy(G), eta=0.5, b_cur=16, b_max=32)
    pinned = c.norm_test(G, p)                                       # the binding's page-locked buffer
    pageable = A.TestResult()
    vp = C.c_void_p
    rc = c.lib.adloco_norm_test(c.h, vp(G.data_ptr()), A.F32, 16, G.shape[1], G.stride(0), C.byref(p), None, None,
                                vp(c._sums_dev.data_ptr()), vp(c._res_dev.data_ptr()), C.cast(C.byref(pageable), vp), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert_test_result(pinned, ora, p, TOL_F32, what="page-locked result")
    assert (pageable.stat, pageable.b_req, pageable.flags, pageable.sum_sqnorm) == (pinned.stat, pinned.b_req, pinned.flags, pinned.sum_sqnorm)
    p2 = A.make_params(1.0, b_cur=16, b_max=32)
    again = c.test_decide(p2)
    pageable2 = A.TestResult()
    rc = c.lib.adloco_test_decide(c.h, vp(c._sums_dev.data_ptr()), C.byref(p2), vp(c._res_dev.data_ptr()), C.cast(C.byref(pageable2), vp), None)
    assert rc == 0
    torch.cuda.synchronize()
    o2 = O.decide(ora.sum_sqnorm, ora.mean_sqnorm, ora.variance, 16, eta=1.0, b_cur=16, b_max=32)
    assert_test_result(again, o2, p2, TOL_F32, what="re-decision")
    assert (pageable2.stat, pageable2.b_req) == (again.stat, again.b_req)
    c.close()
