"""GPU parity: adloco_norm_test / adloco_test_decide / adloco_norm_test_host /
adloco_accumulate against the fp64 oracle, through the C ABI."""
import math

import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_F32, assert_test_result, rel_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _run(ctx, G, params, want_S=True):
    B, P = G.shape
    n = torch.full((B,), -1.0, device=DEV)
    S = torch.full((P,), -1.0, device=DEV) if want_S else None
    r = ctx.norm_test(G, params, per_sample_sqnorm=n, grad_sum=S)
    return r, n.cpu().numpy(), (S.cpu().numpy() if want_S else None)


def _check(ctx, G, params, what, want_S=True):
    r, n, S = _run(ctx, G, params, want_S)
    ora = O.norm_test(W.to_numpy(G), eta=params.eta, ddof=params.ddof, b_cur=params.b_cur, b_max=params.b_max,
                      b_cap=params.b_cap, switch_n=params.switch_n, want_sum=True)
    info = assert_test_result(r, ora, params, TOL_F32, what=what)
    assert np.allclose(n, ora.per_sample_sqnorm, rtol=TOL_F32, atol=0), what
    if want_S:
        scale = np.sqrt(ora.per_sample_sqnorm.max()) / math.sqrt(G.shape[1])  # typical |g_ij|
        assert np.allclose(S, ora.grad_sum, rtol=1e-5, atol=1e-5 * scale * G.shape[0]), what
    return r, ora, info


# sizes chosen to span several 1024-column block tiles, ragged tails (P % 4 != 0),
# row tiles (B > 64) and the small-B register tiles
@pytest.mark.parametrize("B,P", [(16, 1 << 20), (1, 1000), (2, 4099), (3, 77), (5, 1 << 16), (16, 300001),
                                 (17, 65536 + 4), (32, 99999), (33, 40000), (64, 1 << 18), (65, 30001),
                                 (130, 20002), (257, 5003)])
def test_norm_test_matches_oracle(ctx, B, P):
    G = W.per_sample_grads(B, P, sigma=0.5, seed=100 + B, device=DEV)
    p = A.make_params(0.5, b_cur=B, b_max=32)
    _check(ctx, G, p, f"B={B} P={P}")


@pytest.mark.parametrize("sigma,scale", [(0.1, "raw"), (1.0, "raw"), (10.0, "raw"), (0.1, "unit")])
def test_signal_dominated_variance_has_no_cancellation(ctx, sigma, scale):
    G = W.per_sample_grads(32, 1 << 18, sigma=sigma, mean_scale=scale, seed=5, device=DEV)
    _check(ctx, G, A.make_params(0.5, b_cur=32, b_max=32), f"sigma={sigma} {scale}")


def test_strided_rows_and_optional_outputs(ctx):
    G = W.per_sample_grads(9, 5000, seed=2, device=DEV, row_stride=5008)
    assert G.stride(0) == 5008
    _check(ctx, G, A.make_params(0.8, b_cur=9, b_max=4), "strided")
    _check(ctx, G, A.make_params(0.8, b_cur=9, b_max=4), "strided, no S", want_S=False)
    r = ctx.norm_test(G, A.make_params(0.8, b_cur=9, b_max=4))      # no per-sample output either
    ora = O.norm_test(W.to_numpy(G), eta=0.8, b_cur=9, b_max=4)
    assert_test_result(r, ora, A.make_params(0.8, b_cur=9, b_max=4), TOL_F32)


def test_eta_sweep_reuses_the_sums(ctx):
    G = W.per_sample_grads(16, 1 << 17, seed=8, device=DEV)
    Gn = W.to_numpy(G)
    first = ctx.norm_test(G, A.make_params(0.5, b_cur=16, b_max=32))
    launches = ctx.launch_count
    for eta in (0.1, 0.5, 1.0, 0.8):
        p = A.make_params(eta, b_cur=16, b_max=32)
        r = ctx.test_decide(p)
        assert_test_result(r, O.norm_test(Gn, eta=eta, b_cur=16, b_max=32), p, TOL_F32, what=f"eta={eta}")
        if eta == 0.5:
            assert r.stat == first.stat and r.b_req == first.b_req
    assert ctx.launch_count == launches + 4


def test_closed_forms_and_degenerate_cases(ctx):
    # orthonormal rows: stat = B / eta^2 exactly (ddof = 1)
    for B, P, eta in [(2, 4, 0.5), (4, 8, 0.5), (8, 1028, 0.25)]:
        G = torch.eye(P, device=DEV)[:B].contiguous()
        r = ctx.norm_test(G, A.make_params(eta, b_cur=1, b_max=1 << 20))
        assert r.stat == B / eta ** 2 and r.b_req == int(B / eta ** 2)
    # identical gradients: zero variance, batch of one requested
    g = torch.arange(1, 4097, device=DEV, dtype=torch.float32) / 64
    r = ctx.norm_test(g.repeat(6, 1), A.make_params(0.5, b_cur=6, b_max=32))
    assert r.variance == 0.0 and r.stat == 0.0 and r.b_req == 1 and not (r.flags & A.FLAG_GROW)
    # zero mean gradient
    G = torch.tensor([[1.0, -2.0, 0, 0], [-1.0, 2.0, 0, 0]], device=DEV)
    r = ctx.norm_test(G, A.make_params(0.5, b_cur=2, b_max=4))
    assert r.flags & A.FLAG_ZERO_MEAN and math.isinf(r.stat) and r.b_req == O.INT64_MAX
    r = ctx.norm_test(G, A.make_params(0.5, b_cur=2, b_max=4, b_cap=100))
    assert r.b_req == 100 and r.flags & A.FLAG_ACCUMULATE and (r.accum_steps, r.b_micro) == (25, 4)
    # one sample: the variance is undefined
    r = ctx.norm_test(G[:1], A.make_params(0.5, b_cur=3, b_max=4))
    assert r.flags & A.FLAG_UNDEFINED and r.b_req == 3 and r.stat == 0.0
    # scale invariance is exact for a power of two
    G = W.per_sample_grads(8, 4096, seed=1, device=DEV)
    p = A.make_params(0.5, b_cur=8, b_max=32)
    assert ctx.norm_test(G, p).stat == ctx.norm_test(G * 4.0, p).stat
    # run-to-run determinism
    a, c = ctx.norm_test(G, p), ctx.norm_test(G, p)
    assert (a.stat, a.sum_sqnorm, a.mean_sqnorm) == (c.stat, c.sum_sqnorm, c.mean_sqnorm)


def test_switch_plan_cases_through_the_kernel(ctx):
    # 64 orthonormal rows give stat = 64 / eta^2 exactly; eta is chosen to put the
    # statistic half-way between two integers, so that ceil() yields b_req robustly
    G = torch.eye(256, device=DEV)[:64].contiguous()
    for b_req, b_max, n, acc, steps, micro in [(65, 32, 2, 1, 3, 32), (64, 32, 2, 0, 1, 32), (20, 32, 2, 0, 1, 20),
                                               (128, 32, 2, 1, 4, 32), (97, 32, 3, 1, 4, 32), (96, 32, 3, 0, 1, 32)]:
        eta = math.sqrt(64.0 / (b_req - 0.5))
        r = ctx.norm_test(G, A.make_params(eta, b_cur=32, b_max=b_max, switch_n=n))
        assert abs(r.stat - (b_req - 0.5)) < 1e-3
        assert (r.b_req, bool(r.flags & A.FLAG_ACCUMULATE), r.accum_steps, r.b_micro) == (b_req, bool(acc), steps, micro)


def test_argument_errors_never_launch(ctx):
    G = torch.zeros(4, 64, device=DEV)
    before = ctx.launch_count
    for bad in (A.make_params(0.0), A.make_params(-1.0), A.make_params(float("nan")), A.make_params(float("inf")),
                A.make_params(0.5, b_max=0), A.make_params(0.5, switch_n=0), A.make_params(0.5, ddof=-1)):
        with pytest.raises(A.AdlocoError) as e:
            ctx.norm_test(G, bad)
        assert e.value.status == A.ERR_INVALID_ARG
    import ctypes as C
    rc = ctx.lib.adloco_norm_test(ctx.h, C.c_void_p(G.data_ptr()), 7, 4, 64, 64, C.byref(A.make_params(0.5)), None, None,
                                  None, C.c_void_p(ctx._res_dev.data_ptr()), None, None)       # no such dtype
    assert rc == A.ERR_UNSUPPORTED
    with pytest.raises(A.AdlocoError) as e:
        ctx.norm_test(torch.zeros(4097, 8, device=DEV), A.make_params(0.5))
    assert e.value.status == A.ERR_UNSUPPORTED
    assert ctx.launch_count == before


def test_unaligned_rows_take_the_scalar_path(ctx):
    buf = W.per_sample_grads(1, 3 * 6007 + 8, seed=6, device=DEV).view(-1)
    G = buf[1:1 + 3 * 6007].view(3, 6007)                 # base 4 bytes past a 16-byte boundary, odd pitch
    assert G.data_ptr() % 16 == 4
    _check(ctx, G, A.make_params(0.5, b_cur=3, b_max=32), "unaligned")
    G2 = W.per_sample_grads(70, 4103, seed=7, device=DEV, row_stride=4105)
    _check(ctx, G2, A.make_params(0.5, b_cur=70, b_max=32), "odd pitch")


@pytest.mark.parametrize("B,P,stride", [(16, 1 << 18, None), (3, 4099, None), (64, 70001, 70004), (65, 9001, None),
                                        (33, 12345, 12348)])
def test_bf16_gradients(ctx, B, P, stride):
    """Per-sample gradients stored as bfloat16 are widened exactly; the oracle reads the same bits."""
    G32 = W.per_sample_grads(B, P, sigma=0.5, seed=B, device=DEV, row_stride=stride)
    buf = torch.zeros((B, stride or P), dtype=torch.bfloat16, device=DEV)
    G = buf[:, :P]
    G.copy_(G32)
    p = A.make_params(0.5, b_cur=B, b_max=32)
    n = torch.zeros(B, device=DEV)
    S = torch.zeros(P, device=DEV)
    r = ctx.norm_test(G, p, per_sample_sqnorm=n, grad_sum=S)
    ora = O.norm_test(W.to_numpy(G.contiguous()), eta=0.5, b_cur=B, b_max=32, want_sum=True)
    assert_test_result(r, ora, p, TOL_F32, what=f"bf16 B={B} P={P}")
    assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32)
    assert np.allclose(S.cpu().numpy(), ora.grad_sum, rtol=1e-5, atol=1e-5 * B)
    # switch-mode accumulation of the same rows in two micro-batches
    if B >= 2 and stride is None:
        h = B // 2
        Sacc = torch.empty(P, device=DEV)
        acc = A.Accumulator(ctx, [Sacc])
        acc.reset()
        acc.accumulate(G[:h].contiguous())
        acc.accumulate(G[h:].contiguous())
        ra = acc.finalize(p)
        assert_test_result(ra, ora, p, TOL_F32, what="bf16 accumulated")
        acc.close()
    # inner-product tests on the bf16 rows
    ri = ctx.inner_product_test(G, S, theta=0.01, nu=0.3, b_cur=B)
    oi = O.inner_product_tests(W.to_numpy(G.contiguous()), theta=0.01, nu=0.3, b_cur=B)
    assert rel_close(ri.stat_ip, oi.stat_ip, 4 * TOL_F32) and rel_close(ri.stat_orth, oi.stat_orth, 4 * TOL_F32)


def test_largest_supported_batch(ctx):
    G = W.per_sample_grads(4096, 2052, seed=4, device=DEV)
    _check(ctx, G, A.make_params(0.5, b_cur=4096, b_max=32), "B=4096")


# ------------------------------------------------------------------ switch-mode accumulation
@pytest.mark.parametrize("n_micro,b,P,sigma,scale", [(4, 3, 1001, 1.0, "raw"), (8, 32, 1 << 16, 0.1, "raw"),
                                                      (8, 32, 1 << 16, 10.0, "raw"), (3, 16, 70001, 0.5, "unit"),
                                                      (2, 65, 9001, 1.0, "raw")])
def test_accumulated_test_matches_one_shot_oracle(ctx, n_micro, b, P, sigma, scale):
    mbs = W.micro_batches(n_micro, b, P, sigma=sigma, mean_scale=scale, seed=21, device=DEV)
    S = torch.full((P,), 7.0, device=DEV)
    acc = A.Accumulator(ctx, [S])
    acc.reset()
    n_all = torch.zeros(n_micro * b, device=DEV)
    for j, m in enumerate(mbs):
        acc.accumulate(m, per_sample_sqnorm=n_all[j * b:(j + 1) * b])
    p = A.make_params(0.5, b_cur=n_micro * b, b_max=b)
    r = acc.finalize(p)
    ora = O.accumulated_norm_test([W.to_numpy(m) for m in mbs], eta=0.5, b_cur=n_micro * b, b_max=b, want_sum=True)
    assert_test_result(r, ora, p, TOL_F32, what="accumulated")
    assert np.allclose(n_all.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32)
    assert np.allclose(S.cpu().numpy(), ora.grad_sum, rtol=1e-5, atol=1e-5 * np.abs(ora.grad_sum).max())
    # same answer as the GPU one-shot test on the concatenation
    one = ctx.norm_test(torch.cat(mbs), p)
    assert rel_close(one.stat, r.stat, 2e-5)
    # reset really clears
    acc.reset()
    acc.accumulate(mbs[0])
    r1 = acc.finalize(A.make_params(0.5, b_cur=b, b_max=b))
    o1 = O.norm_test(W.to_numpy(mbs[0]), eta=0.5, b_cur=b, b_max=b)
    assert_test_result(r1, o1, A.make_params(0.5, b_cur=b, b_max=b), TOL_F32, what="after reset")
    acc.close()


@pytest.mark.parametrize("sigma", [1e-3, 3e-5])
def test_accumulated_variance_keeps_its_digits_when_the_mean_dominates(ctx, sigma):
    """Mean far above the noise: Q - b N would cancel 6 to 9 digits (sum_i n_i / ((b-1) V) ~ 1e6 .. 1e9).
    The materialised accumulation keeps the column-centred sum of squares across micro-batches, so
    the accumulated variance must match the one-shot test and the oracle as if nothing cancelled."""
    n_micro, b, P = 6, 16, 40000
    mbs = W.micro_batches(n_micro, b, P, sigma=sigma, mean_scale="raw", seed=77, device=DEV)
    S = torch.empty(P, device=DEV)
    acc = A.Accumulator(ctx, [S])
    acc.reset()
    for m in mbs:
        acc.accumulate(m)
    p = A.make_params(0.5, b_cur=n_micro * b, b_max=b)
    r = acc.finalize(p)
    sums = ctx.read_sums()
    assert sums.has_centred == 1 and sums.batch_count == n_micro * b
    ora = O.accumulated_norm_test([W.to_numpy(m) for m in mbs], eta=0.5, b_cur=n_micro * b, b_max=b)
    assert ora.sum_sqnorm / (ora.variance * (n_micro * b - 1)) > 1e5
    assert_test_result(r, ora, p, TOL_F32, what="signal-dominated accumulation")
    one = ctx.norm_test(torch.cat(mbs), p)
    assert rel_close(one.variance, r.variance, TOL_F32) and rel_close(one.stat, r.stat, TOL_F32)
    # a form-(b) call in between drops the centred sum for good: the identity takes over
    acc.reset()
    acc.accumulate(mbs[0])
    n1 = torch.zeros(b, device=DEV)
    ctx.norm_test(mbs[1], p, per_sample_sqnorm=n1)
    S += mbs[1].sum(0)
    acc.accumulate(per_sample_sqnorm=n1)
    acc.finalize(p)
    assert ctx.read_sums().has_centred == 0
    acc.close()


@pytest.mark.parametrize("bad", [float("inf"), float("nan"), 3e38])
def test_nonfinite_gradients_raise_the_flag_and_keep_the_batch(ctx, bad):
    """One Inf / NaN entry (or one whose square overflows fp32) poisons the sums: the result carries
    NONFINITE, the batch stays at b_cur and the switch plan is that of b_cur -- no huge request."""
    G = W.per_sample_grads(8, 5000, seed=6, device=DEV)
    G[3, 1234] = bad
    p = A.make_params(0.5, b_cur=8, b_max=32)
    r = ctx.norm_test(G, p)
    assert r.flags == A.FLAG_NONFINITE and r.b_req == 8 and r.stat == 0.0 and r.variance == 0.0
    assert (r.accum_steps, r.b_micro) == (1, 8)
    if bad != 3e38:
        Gn = W.to_numpy(G)
        assert_test_result(r, O.norm_test(Gn, eta=0.5, b_cur=8, b_max=32), p, TOL_F32, what="non-finite")
        S = torch.empty(5000, device=DEV)
        ctx.norm_test(G, p, grad_sum=S)
        ri = ctx.inner_product_test(G, S, theta=0.1, nu=0.3, b_cur=8)
        assert ri.flags == A.FLAG_NONFINITE and ri.b_ip == ri.b_aug == 8
    # the accumulator reports it too
    S = torch.empty(5000, device=DEV)
    acc = A.Accumulator(ctx, [S])
    acc.reset()
    acc.accumulate(G)
    ra = acc.finalize(p)
    assert ra.flags == A.FLAG_NONFINITE and ra.b_req == 8
    acc.close()
    G[3, 1234] = 0.0
    assert ctx.norm_test(G, p).flags & A.FLAG_NONFINITE == 0


def test_accumulate_from_given_norms_uses_the_identity(ctx):
    # form (b): the caller adds the gradient sums itself and hands over n_i
    mbs = W.micro_batches(3, 8, 5000, sigma=1.0, seed=3, device=DEV)
    S = torch.zeros(5000, device=DEV)
    S2 = torch.zeros(12, device=DEV)         # a second, empty parameter buffer
    acc = A.Accumulator(ctx, [S, S2])
    acc.reset()
    for m in mbs:
        S += m.sum(0)
        acc.accumulate(per_sample_sqnorm=(m.double() ** 2).sum(1).float())
    p = A.make_params(0.5, b_cur=24, b_max=8)
    r = acc.finalize(p)
    ora = O.accumulated_norm_test_by_sums([W.to_numpy(m) for m in mbs], eta=0.5, b_cur=24, b_max=8)
    assert_test_result(r, ora, p, TOL_F32, what="from norms")
    acc.close()


# ------------------------------------------------------------------ host-memory entry point
@pytest.mark.parametrize("B,P", [(16, 1 << 20), (3, 5001), (64, (1 << 19) + 12)])
def test_host_entry_point_matches_oracle(ctx, B, P):
    G = W.per_sample_grads(B, P, seed=31, device="cpu").pin_memory()
    p = A.make_params(0.5, b_cur=B, b_max=32)
    n = torch.zeros(B).pin_memory()
    r = ctx.norm_test_host(G, p, per_sample_sqnorm_host=n)
    ora = O.norm_test(G.numpy(), eta=0.5, b_cur=B, b_max=32)
    assert_test_result(r, ora, p, TOL_F32, what="host")
    assert np.allclose(n.numpy(), ora.per_sample_sqnorm, rtol=TOL_F32)
