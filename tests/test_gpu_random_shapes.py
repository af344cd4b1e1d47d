"""Randomised shapes (fixed seed): every entry point against the oracle on many
small, ragged problems -- row counts around the register-tile sizes, column counts
off every vector width, token counts off the tile sizes, feature widths that are
only multiples of 8."""
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


def test_norm_test_and_inner_product_random_shapes(ctx):
    rng = np.random.default_rng(2024)
    for case in range(40):
        B = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 129]))
        P = int(rng.integers(1, 20000))
        pad = int(rng.choice([0, 0, 1, 3, 4, 8]))
        bf16 = bool(rng.integers(0, 2))
        sigma = float(rng.choice([0.1, 0.5, 2.0]))
        scale = str(rng.choice(["unit", "raw"]))
        G32 = W.per_sample_grads(B, P, sigma=sigma, mean_scale=scale, seed=case, device=DEV, row_stride=P + pad)
        if bf16:
            buf = torch.zeros((B, P + pad), dtype=torch.bfloat16, device=DEV)
            G = buf[:, :P]
            G.copy_(G32)
        else:
            G = G32
        eta = float(rng.choice([0.1, 0.5, 0.8, 1.0]))
        p = A.make_params(eta, b_cur=B, b_max=int(rng.choice([1, 4, 32])), switch_n=int(rng.choice([1, 2, 3])))
        n = torch.zeros(B, device=DEV)
        S = torch.zeros(P, device=DEV)
        r = ctx.norm_test(G, p, per_sample_sqnorm=n, grad_sum=S)
        Gn = W.to_numpy(G.contiguous())
        ora = O.norm_test(Gn, eta=eta, b_cur=B, b_max=p.b_max, switch_n=p.switch_n, want_sum=True)
        what = f"case {case}: B={B} P={P} pad={pad} bf16={bf16}"
        assert_test_result(r, ora, p, TOL_F32, what=what)
        assert np.allclose(n.cpu().numpy(), ora.per_sample_sqnorm, rtol=TOL_F32), what
        assert np.allclose(S.cpu().numpy(), ora.grad_sum, rtol=1e-5, atol=1e-5 * np.abs(ora.grad_sum).max() + 1e-30), what
        if B >= 2 and ora.mean_sqnorm > 0:
            ri = ctx.inner_product_test(G, S, theta=0.05, nu=0.3, b_cur=B)
            oi = O.inner_product_tests(Gn, theta=0.05, nu=0.3, b_cur=B)
            for got, ref in ((ri.var_ip, oi.var_ip), (ri.var_orth, oi.var_orth)):
                assert rel_close(got, ref, 4 * TOL_F32) or abs(got - ref) < 1e-7 * ora.sum_sqnorm, (what, got, ref)


def test_outer_step_random_shapes(ctx):
    rng = np.random.default_rng(7)
    for case in range(30):
        K = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 12, 16, 17, 33]))
        P = int(rng.integers(1, 50000))
        dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
        nesterov = bool(rng.integers(0, 2))
        lr, mu = float(rng.choice([0.1, 0.5, 0.7, 1.0])), float(rng.choice([0.0, 0.5, 0.9]))
        theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=case, device=DEV, zero_momentum=bool(rng.integers(0, 2)))
        th0, v0 = W.to_numpy(theta).astype(np.float64), W.to_numpy(mom).astype(np.float64)
        ins = [W.to_numpy(t) for t in inst]
        lrf, muf = float(np.float32(lr)), float(np.float32(mu))
        th_ref, v_ref = O.outer_step(W.to_numpy(theta), ins, W.to_numpy(mom), lr=lrf, momentum=muf, nesterov=nesterov)
        d = np.mean([th0 - O.widen(x) for x in ins], axis=0)
        th, v = ctx.outer_step(inst, theta, mom, lr=lr, momentum=mu, nesterov=nesterov)
        assert_outer_step(th.cpu().numpy(), v.cpu().numpy(), th_ref, v_ref, th0, v0, d, lrf, muf,
                          what=f"case {case}: K={K} P={P} {dtype} nesterov={nesterov}")


def test_linear_layer_random_shapes(ctx):
    rng = np.random.default_rng(99)
    for case in range(24):
        B = int(rng.integers(1, 9))
        T = int(rng.integers(1, 400)) if case % 4 else int(rng.integers(400, 1300))
        d_in = 8 * int(rng.integers(1, 50))
        d_out = 8 * int(rng.integers(1, 70))
        X, D = W.linear_layer(B, T, d_in, d_out, seed=case, delta_std=0.1, device=DEV)
        n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
        for method in ("gram", "gram_pair", "direct", "pair"):
            n = torch.zeros(B, device=DEV)
            S = torch.zeros(d_out, d_in, device=DEV)
            ctx.linear_sqnorm(X, D, n, grad_sum=S, method=method)
            torch.cuda.synchronize()
            what = f"case {case} {method}: B={B} T={T} {d_in}->{d_out}"
            assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16), what
            assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05), what
        d = min(d_in, d_out)
        nb = torch.zeros(B, device=DEV)
        Sb = torch.zeros(d, device=DEV)
        Xg, Dg = X[:, :, :d].contiguous(), D[:, :, :d].contiguous()
        ctx.vector_param_sqnorm(Dg, nb, X=Xg, grad_sum=Sb)
        torch.cuda.synchronize()
        nb_ref, Sb_ref = O.vector_param_terms(W.to_numpy(Dg), W.to_numpy(Xg))
        assert np.allclose(nb.cpu().numpy(), nb_ref, rtol=TOL_BF16) and np.allclose(Sb.cpu().numpy(), Sb_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(Sb_ref).max() * 0.05)
        # the same output gradients as those of an embedding table: few ids (long groups), many ids, ids outside the table
        V = int(rng.choice([2, 17, 5000]))
        ids = torch.from_numpy(rng.integers(-2, V + 3, size=(B, T)).astype(np.int32)).to(DEV)
        ne = torch.zeros(B, device=DEV)
        ctx.embedding_sqnorm(ids, D, V, ne)
        torch.cuda.synchronize()
        ne_ref, _ = O.embedding_terms(ids.cpu().numpy(), W.to_numpy(D), V)
        assert np.allclose(ne.cpu().numpy(), ne_ref, rtol=TOL_BF16, atol=1e-30), f"embedding case {case}: B={B} T={T} d={d_out} V={V}"
    assert ctx.device_status() == 0
