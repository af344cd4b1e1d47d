"""GPU parity: adloco_inner_product_test (inner-product test and its augmented
form, a second pass over the gradients after the norm test) against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_F32, rel_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _run(ctx, G, theta, nu, **kw):
    B, P = G.shape
    S = torch.empty(P, device=DEV)
    n = torch.empty(B, device=DEV)
    ctx.norm_test(G, A.make_params(0.5, b_cur=B, b_max=32), per_sample_sqnorm=n, grad_sum=S)
    p = torch.full((B,), -1.0, device=DEV)
    r = ctx.inner_product_test(G, S, theta=theta, nu=nu, inner_products=p, **kw)
    return r, p.cpu().numpy()


def _check(ctx, G, theta, nu, what, **kw):
    r, p = _run(ctx, G, theta, nu, **kw)
    o = O.inner_product_tests(W.to_numpy(G), theta=theta, nu=nu, **kw)
    assert r.device_status == 0 and r.batch_count == o.batch_count and r.flags == o.flags, what
    assert rel_close(r.mean_sqnorm, o.mean_sqnorm, TOL_F32), what
    assert np.allclose(p, o.inner_products, rtol=TOL_F32), what
    assert rel_close(r.var_ip, o.var_ip, 2 * TOL_F32), (what, r.var_ip, o.var_ip)
    assert rel_close(r.stat_ip, o.stat_ip, 4 * TOL_F32), (what, r.stat_ip, o.stat_ip)
    assert rel_close(r.var_orth, o.var_orth, 2 * TOL_F32), (what, r.var_orth, o.var_orth)
    assert rel_close(r.stat_orth, o.stat_orth, 4 * TOL_F32), (what, r.stat_orth, o.stat_orth)
    for got, ref, stat in ((r.b_ip, o.b_ip, o.stat_ip), (r.b_aug, o.b_aug, max(o.stat_ip, o.stat_orth))):
        if abs(stat - round(stat)) > 8 * TOL_F32 * abs(stat):      # decisive: away from an integer boundary
            assert got == ref, (what, got, ref, stat)
        else:
            assert abs(got - ref) <= 1, (what, got, ref, stat)
    return r, o


@pytest.mark.parametrize("B,P,sigma,scale", [(16, 1 << 20, 0.5, "unit"), (2, 4099, 0.5, "unit"), (5, 77, 1.0, "raw"),
                                             (32, 99999, 0.1, "raw"), (33, 40000, 10.0, "raw"), (64, 1 << 18, 0.5, "unit"),
                                             (130, 20002, 1.0, "raw"), (64, 300001, 1.0, "unit")])
def test_inner_product_tests_match_oracle(ctx, B, P, sigma, scale):
    G = W.per_sample_grads(B, P, sigma=sigma, mean_scale=scale, seed=B + 7, device=DEV)
    # theta = 0.01 and nu = 0.3 are the paper's hyper-parameters
    _check(ctx, G, 0.01, 0.3, f"B={B} P={P} sigma={sigma} {scale}", b_cur=B)


def test_closed_forms_and_degenerate_cases(ctx):
    # orthonormal gradients: no spread of the inner products; orthogonal parts give b / nu^2
    G = torch.eye(1024, device=DEV)[:8].contiguous()
    r, _ = _run(ctx, G, 0.01, 0.5)
    assert r.stat_ip < 1e-9 and r.b_ip == 1 and abs(r.stat_orth - 32.0) < 1e-4 and r.b_aug == 32
    # collinear gradients: no orthogonal part
    a = torch.tensor([1.0, 2.0, 3.0, 6.0], device=DEV)
    u = torch.zeros(4096, device=DEV)
    u[5] = 1.0
    r, p = _run(ctx, (a[:, None] * u[None, :]).contiguous(), 0.5, 0.3)
    assert abs(r.stat_ip - (14.0 / 3) / (0.25 * 9.0)) < 1e-5 and r.var_orth < 1e-9 and r.b_aug == r.b_ip == 3
    assert np.allclose(p, [3.0, 6.0, 9.0, 18.0])
    # one sample / zero mean / cap
    G = W.per_sample_grads(6, 3000, seed=1, device=DEV)
    r, _ = _run(ctx, G[:1], 0.01, 0.3, b_cur=5)
    assert r.flags & A.FLAG_UNDEFINED and r.b_ip == r.b_aug == 5
    Z = torch.tensor([[1.0, -1.0, 0, 0], [-1.0, 1.0, 0, 0]], device=DEV)
    r, _ = _run(ctx, Z, 0.01, 0.3)
    assert r.flags & A.FLAG_ZERO_MEAN and math.isinf(r.stat_ip) and r.b_aug == O.INT64_MAX
    _check(ctx, G, 0.01, 0.3, "cap", b_cur=6, b_cap=50)
    before = ctx.launch_count
    S = torch.zeros(3000, device=DEV)
    with pytest.raises(A.AdlocoError) as e:
        ctx.inner_product_test(G, S, theta=0.0, nu=0.3)
    assert e.value.status == A.ERR_INVALID_ARG and ctx.launch_count == before


def test_unaligned_and_strided_rows(ctx):
    G = W.per_sample_grads(9, 5003, seed=2, device=DEV, row_stride=5005)
    _check(ctx, G, 0.01, 0.3, "odd pitch", b_cur=9)
