"""GPU parity at the full sizes of the five workload configurations, in the
launch configuration the benchmark times.  Where the oracle cannot finish the
whole problem in seconds it checks sampled outputs it can compute one by one
(the outer step is elementwise; a gradient-sum row is one matrix-vector
product) and properties that hold at any size (the Gaussian closed form of the
statistic)."""
import math

import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_BF16, TOL_F32, assert_outer_step, assert_test_result, rel_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _outer_sampled(ctx, K, P, dtype, seed, n_slices=48, width=4096):
    """Full-size outer step on the GPU (two steps, in place), oracle on sampled slices."""
    theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=seed, device=DEV)
    rng = np.random.default_rng(seed)
    starts = sorted(set([0, max(P - width, 0)] + [int(x) for x in rng.integers(0, max(P - width, 1), n_slices)]))
    lr, mu = float(np.float32(0.7)), float(np.float32(0.9))
    worst = (0.0, 0.0)
    for step in range(2):
        before = [(theta[s:s + width].cpu().numpy(), mom[s:s + width].cpu().numpy(),
                   [W.to_numpy(t[s:s + width]) for t in inst]) for s in starts]
        ctx.outer_step(inst, theta, mom, lr=0.7, momentum=0.9, nesterov=True)
        torch.cuda.synchronize()
        for s, (th0, v0, ins) in zip(starts, before):
            th_ref, v_ref = O.outer_step(th0, ins, v0, lr=lr, momentum=mu, nesterov=True)
            d = np.mean([th0.astype(np.float64) - O.widen(x) for x in ins], axis=0)
            e = assert_outer_step(theta[s:s + width].cpu().numpy(), mom[s:s + width].cpu().numpy(), th_ref, v_ref,
                                  th0.astype(np.float64), v0.astype(np.float64), d, lr, mu,
                                  what=f"K={K} P={P} step={step} slice={s}")
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
    return worst


# ---------------------------------------------------------------- config 1 (small; the oracle runs it whole)
def test_config1_norm_test_and_outer_step(ctx):
    G = W.per_sample_grads(16, 1 << 20, sigma=0.5, seed=1, device=DEV)
    p = A.make_params(0.5, b_cur=16, b_max=32)
    r = ctx.norm_test(G, p)
    ora = O.norm_test(W.to_numpy(G), eta=0.5, b_cur=16, b_max=32)
    assert_test_result(r, ora, p, TOL_F32, what="config 1")
    # Gaussian closed form: stat -> s^2 P / (eta^2 (|m|^2 + s^2 P / B)) ~ 64
    assert abs(r.stat - 64.0) < 0.5
    worst = _outer_sampled(ctx, 4, 1 << 20, torch.float32, seed=11, n_slices=256)
    assert worst[0] <= 2.0


# ---------------------------------------------------------------- config 2
def test_config2_norm_test_eta_sweep_full_size(ctx):
    B, P = 64, 1 << 24
    G = W.per_sample_grads(B, P, sigma=0.5, seed=2, device=DEV)
    n = torch.zeros(B, device=DEV)
    p0 = A.make_params(0.1, b_cur=B, b_max=32)
    r0 = ctx.norm_test(G, p0, per_sample_sqnorm=n)
    Gh = W.to_numpy(G)
    ora = O.norm_test(Gh, eta=0.1, b_cur=B, b_max=32)
    assert_test_result(r0, ora, p0, TOL_F32, what="config 2 eta=0.1")
    assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32)
    for eta, expect in ((0.5, 256.0), (1.0, 64.0)):
        p = A.make_params(eta, b_cur=B, b_max=32)
        r = ctx.test_decide(p)
        o = O.decide(ora.sum_sqnorm, ora.mean_sqnorm, ora.variance, B, eta=eta, b_cur=B, b_max=32)
        assert_test_result(r, o, p, TOL_F32, what=f"config 2 eta={eta}")
        assert abs(r.stat - expect) < 0.02 * expect
    assert abs(r0.stat - 6400.0) < 0.02 * 6400.0


def test_config2_outer_step_full_size(ctx):
    _outer_sampled(ctx, 8, W.GPT2_SMALL_P, torch.bfloat16, seed=22)


# ---------------------------------------------------------------- config 3
def test_config3_gram_layer_full_size(ctx):
    B, T, d_in, d_out = 32, 1024, 768, 3072
    X, D = W.linear_layer(B, T, d_in, d_out, seed=3, device=DEV)
    n = torch.zeros(B, device=DEV)
    S = torch.zeros(d_out, d_in, device=DEV)
    acc = A.Accumulator(ctx, [S])
    acc.reset()
    ctx.gram_sqnorm(X, D, n, grad_sum=S, accumulate_sum=True)
    acc.accumulate(per_sample_sqnorm=n)
    p = A.make_params(0.5, b_cur=B, b_max=32)
    r = acc.finalize(p)
    ora = O.linear_layers_norm_test([(W.to_numpy(X), W.to_numpy(D))], eta=0.5, b_cur=B, b_max=32, two_pass=False)
    assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_BF16)
    S_ref = ora.grad_sum[0]
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    kappa = ora.sum_sqnorm / (ora.variance * (B - 1))
    assert_test_result(r, ora, p, TOL_BF16, stat_tol=TOL_BF16 * max(1.0, kappa), what="config 3")
    assert abs(r.stat - 128.0) < 2.0          # pure-noise layers: stat ~ B / eta^2
    acc.close()


# ---------------------------------------------------------------- config 4
def test_config4_whole_model_switch_mode_full_size(ctx):
    """12 blocks x 4 linear layers, batch 128 as 4 accumulated micro-batches of 32, three ways: the
    Gram identity layer by layer, the automatic route layer by layer (the direct kernel over CTA pairs
    for these shapes), and the grouped call that takes the 48 layers of a micro-batch in ONE launch --
    the launch configuration the benchmark times.  The oracle
    runs the whole model once, streamed layer by layer and micro-batch by micro-batch (explicit
    per-sample gradients in fp64; about a minute of host BLAS), and every output is compared: the
    128 per-sample norms, each layer's gradient sum element by element, ||S_l||^2 per layer, and the
    statistic, decision and switch plan."""
    shapes = list(W.GPT2_SMALL_BLOCK_LINEARS) * 12
    n_micro, b, T = 4, 32, 1024
    routes = ("gram", "auto", "group")
    sums = {m: [torch.empty(do, di, device=DEV) for di, do in shapes] for m in routes}
    accs = {m: A.Accumulator(ctx, sums[m]) for m in routes}
    n_mb = {m: torch.zeros(b, device=DEV) for m in routes}
    n_all = {m: torch.zeros(n_micro * b, device=DEV) for m in routes}
    for m in routes:
        accs[m].reset()
    n_ref = np.zeros(n_micro * b)
    S_ref = [np.zeros((do, di)) for di, do in shapes]
    for j in range(n_micro):
        # the grouped launch needs every layer of the micro-batch resident at once (9.7 GB)
        data = [W.linear_layer(b, T, di, do, seed=100000 + 100 * l + j, device=DEV) for l, (di, do) in enumerate(shapes)]
        ctx.linear_sqnorm_group([(X, D, S) for (X, D), S in zip(data, sums["group"])], n_mb["group"], method="auto",
                                accumulate_sum=True)
        for l, (X, D) in enumerate(data):
            for m in ("gram", "auto"):
                ctx.linear_sqnorm(X, D, n_mb[m], accumulate_norms=(l > 0), grad_sum=sums[m][l], accumulate_sum=True,
                                  method=m)
            n_l, S_l = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))     # overlaps the GPU work
            n_ref[j * b:(j + 1) * b] += n_l
            S_ref[l] += S_l
        del data
        for m in routes:
            accs[m].accumulate(per_sample_sqnorm=n_mb[m])
            n_all[m][j * b:(j + 1) * b] = n_mb[m]
    p = A.make_params(0.5, b_cur=128, b_max=32)
    ora = O.norm_test_from_sums(n_ref, S_ref, n_micro * b, eta=0.5, b_cur=128, b_max=32)
    kappa = ora.sum_sqnorm / (ora.variance * (n_micro * b - 1))
    for m in routes:
        r = accs[m].finalize(p)
        assert ctx.device_status() == 0
        assert np.allclose(n_all[m].cpu().numpy(), n_ref, rtol=TOL_BF16, atol=0), m
        for l in range(len(shapes)):
            got = sums[m][l].cpu().numpy().astype(np.float64)
            assert np.allclose(got, S_ref[l], rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref[l]).max() * 0.05), (m, l)
            assert rel_close(float((got ** 2).sum()), float((S_ref[l] ** 2).sum()), TOL_BF16), (m, l)
        assert_test_result(r, ora, p, TOL_BF16, stat_tol=TOL_BF16 * max(1.0, kappa), what=f"config 4 {m}")
        assert r.batch_count == 128 and r.flags & A.FLAG_ACCUMULATE and r.flags & A.FLAG_GROW and r.b_micro == 32
        # pure-noise gradients: stat ~ B / eta^2 = 512
        assert abs(r.stat - 512.0) < 0.01 * 512.0, r.stat
        accs[m].close()


# ---------------------------------------------------------------- config 5
def test_config5_large_outer_merge(ctx):
    _outer_sampled(ctx, 4, W.LARGE_P, torch.bfloat16, seed=55)


@pytest.mark.parametrize("scale", ["unit", "raw"])
@pytest.mark.parametrize("sigma", [0.1, 1.0, 10.0])
def test_config5_accumulated_test(ctx, sigma, scale):
    n_micro, b, P = 8, 32, 1 << 22
    mbs = W.micro_batches(n_micro, b, P, sigma=sigma, mean_scale=scale, seed=5, device=DEV)
    S = torch.empty(P, device=DEV)
    acc = A.Accumulator(ctx, [S])
    acc.reset()
    for m in mbs:
        acc.accumulate(m)
    p = A.make_params(0.5, b_cur=256, b_max=32)
    r = acc.finalize(p)
    ora = O.accumulated_norm_test([W.to_numpy(m) for m in mbs], eta=0.5, b_cur=256, b_max=32)
    info = assert_test_result(r, ora, p, TOL_F32, what=f"config 5 sigma={sigma} {scale}")
    if scale == "raw":
        # signal-dominated: stat ~ sigma^2 / (eta^2 (1 + sigma^2 / B)); the decision flips with sigma
        expect = sigma ** 2 / (0.25 * (1.0 + sigma ** 2 / 256))
        assert abs(r.stat - expect) < 0.01 * expect
        assert bool(r.flags & A.FLAG_GROW) == (sigma == 10.0)
        assert bool(r.flags & A.FLAG_ACCUMULATE) == (sigma == 10.0)
    acc.close()
