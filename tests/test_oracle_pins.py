"""Pins for the fp64 oracle: each check ties the oracle to something other than
itself -- exact rational arithmetic written out from the paper's definitions,
closed forms, hand-worked fixtures, a library optimiser, brute force.

Every pin is a function of the oracle module, so that the same pins can be run
against deliberately broken copies of the oracle (test_mutants_are_caught): a
dropped term, a flipped sign, a transposed operand or a wrong normaliser must
fail at least one pin.
"""
import importlib.util
import math
import os
import sys
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle.adloco_oracle as ORACLE
from paper_2508_18182_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


# ---------------------------------------------------------------- exact helpers
def exact_norm_test(G, eta, ddof):
    """Definitions of Eq. 1 and of the norm-test section in exact rationals."""
    b, P = len(G), len(G[0])
    gbar = [sum(Fraction(G[i][j]) for i in range(b)) / b for j in range(P)]
    n = [sum(Fraction(G[i][j]) ** 2 for j in range(P)) for i in range(b)]
    N = sum(x * x for x in gbar)
    dev = sum((Fraction(G[i][j]) - gbar[j]) ** 2 for i in range(b) for j in range(P))
    V = dev / (b - ddof)
    stat = V / (Fraction(eta) ** 2 * N)
    return n, N, V, stat, math.ceil(stat)


def int_matrix(rng, b, P, lo=-4, hi=5):
    return rng.integers(lo, hi, size=(b, P)).astype(np.float32)


# ------------------------------------------------------------------------ pins
def pin_exact_rational_norm_test(O):
    rng = np.random.default_rng(7)
    for b, P, eta, ddof in [(3, 4, 0.5, 1), (5, 7, 0.25, 1), (4, 6, 2.0, 0), (2, 9, 0.5, 1)]:
        G = int_matrix(rng, b, P)
        G[0, 0] += 1.0  # keep the mean away from zero
        n, N, V, stat, b_req = exact_norm_test(G.tolist(), eta, ddof)
        r = O.norm_test(G, eta=eta, ddof=ddof, b_cur=1, b_max=1 << 40, want_sum=True)
        assert np.allclose(r.per_sample_sqnorm, [float(x) for x in n], rtol=1e-14)
        assert math.isclose(r.sum_sqnorm, float(sum(n)), rel_tol=1e-14)
        assert math.isclose(r.mean_sqnorm, float(N), rel_tol=1e-13)
        assert math.isclose(r.variance, float(V), rel_tol=1e-13)
        assert math.isclose(r.stat, float(stat), rel_tol=1e-13)
        assert r.b_req == max(1, b_req)
        assert r.batch_count == b
        assert np.array_equal(r.grad_sum, G.astype(np.float64).sum(axis=0))


def pin_orthonormal_closed_form(O):
    for line in _rows("norm_test_closed_forms.txt"):
        lhs, rhs = line.split("|")
        b, P, eta, ddof = lhs.split()
        Q, N, V, stat, b_req = (float(x) for x in rhs.split())
        G = np.eye(int(P), dtype=np.float32)[: int(b)]
        r = O.norm_test(G, eta=float(eta), ddof=int(ddof), b_cur=1, b_max=1 << 40)
        assert math.isclose(r.sum_sqnorm, Q, rel_tol=1e-15)
        assert math.isclose(r.mean_sqnorm, N, rel_tol=1e-15)
        assert math.isclose(r.variance, V, rel_tol=1e-14)
        assert math.isclose(r.stat, stat, rel_tol=1e-14)
        assert r.b_req == int(b_req)


def pin_identical_gradients_zero_variance(O):
    g = np.arange(1, 33, dtype=np.float32) / 8
    G = np.tile(g, (6, 1))
    r = O.norm_test(G, eta=0.5, b_cur=6, b_max=32)
    assert r.variance == 0.0 and r.stat == 0.0 and r.b_req == 1
    assert not (r.flags & O.FLAG_GROW)
    assert math.isclose(r.mean_sqnorm, float(np.dot(g.astype(np.float64), g)), rel_tol=1e-15)


def pin_scale_invariance_and_identity(O):
    G = W.to_numpy(W.per_sample_grads(8, 257, sigma=0.5, seed=3))
    a = O.norm_test(G, eta=0.5, b_cur=8, b_max=64)
    c = O.norm_test(G * np.float32(4.0), eta=0.5, b_cur=8, b_max=64)
    assert a.stat == c.stat and c.variance == 16.0 * a.variance   # power-of-two scale: exact
    # sum_i ||g_i - gbar||^2 == sum_i n_i - b ||gbar||^2
    b = G.shape[0]
    assert math.isclose(a.variance * (b - 1), a.sum_sqnorm - b * a.mean_sqnorm, rel_tol=1e-10)
    # Cauchy-Schwarz sanity
    assert a.variance >= 0 and a.mean_sqnorm <= a.sum_sqnorm / b
    # eta enters as 1/eta^2
    d = O.norm_test(G, eta=1.0, b_cur=8, b_max=64)
    assert math.isclose(d.stat * 4.0, a.stat, rel_tol=1e-15)
    # sample permutation changes nothing beyond rounding
    p = O.norm_test(G[::-1].copy(), eta=0.5, b_cur=8, b_max=64)
    assert math.isclose(p.stat, a.stat, rel_tol=1e-12)
    assert np.allclose(p.per_sample_sqnorm[::-1], a.per_sample_sqnorm, rtol=1e-15)


def pin_gaussian_concentration(O):
    # g_i = m + s z_i: E[V] = s^2 P, E[N] = ||m||^2 + s^2 P / b  =>  stat -> s^2 P / (eta^2 (||m||^2 + s^2 P / b))
    b, P, s, eta = 16, 1 << 16, 0.5, 0.5
    G = W.per_sample_grads(b, P, sigma=s, seed=11)
    r = O.norm_test(W.to_numpy(G), eta=eta, b_cur=b, b_max=32)
    expect = s * s * P / (eta * eta * (1.0 + s * s * P / b))
    assert abs(r.stat - expect) < 8 * expect * math.sqrt(2.0 / P) + 0.05 * expect / (s * s * P / b)


def pin_decision_branches(O):
    # zero mean gradient
    G = np.array([[1.0, -2.0], [-1.0, 2.0]], dtype=np.float32)
    r = O.norm_test(G, eta=0.5, b_cur=2, b_max=4)
    assert r.flags & O.FLAG_ZERO_MEAN and math.isinf(r.stat) and r.b_req == O.INT64_MAX
    r = O.norm_test(G, eta=0.5, b_cur=2, b_max=4, b_cap=100)
    assert r.b_req == 100 and r.flags & O.FLAG_ACCUMULATE and r.accum_steps == 25 and r.b_micro == 4
    # a single sample: variance undefined with ddof = 1
    r = O.norm_test(G[:1], eta=0.5, b_cur=1, b_max=4)
    assert r.flags & O.FLAG_UNDEFINED and r.b_req == 1 and r.stat == 0.0
    # b_cap clamps, GROW compares with b_cur
    G = np.eye(8, dtype=np.float32)[:4]            # stat = 16 at eta = 0.5
    r = O.norm_test(G, eta=0.5, b_cur=16, b_max=32)
    assert r.b_req == 16 and not (r.flags & O.FLAG_GROW)
    r = O.norm_test(G, eta=0.5, b_cur=15, b_max=32)
    assert r.flags & O.FLAG_GROW
    r = O.norm_test(G, eta=0.5, b_cur=4, b_max=32, b_cap=10)
    assert r.b_req == 10
    with pytest.raises(ValueError):
        O.norm_test(G, eta=0.0)


def pin_switch_plan(O):
    for line in _rows("switch_plan_cases.txt"):
        lhs, rhs = line.split("|")
        b_req, b_max, n = (int(x) for x in lhs.split())
        acc, steps, micro = (int(x) for x in rhs.split())
        assert O.switch_plan(b_req, b_max, n) == (bool(acc), steps, micro)
        # through the batch rule: orthonormal rows give stat = b / eta^2 exactly (eta = 1 => b_req = b)
    G = np.eye(128, dtype=np.float32)[:65]
    r = O.norm_test(G, eta=1.0, b_cur=32, b_max=32, switch_n=2)
    assert (r.b_req, bool(r.flags & O.FLAG_ACCUMULATE), r.accum_steps, r.b_micro) == (65, True, 3, 32)
    r = O.norm_test(G[:64], eta=1.0, b_cur=32, b_max=32, switch_n=2)
    assert (r.b_req, bool(r.flags & O.FLAG_ACCUMULATE), r.accum_steps, r.b_micro) == (64, False, 1, 32)


def pin_accumulated_equals_one_shot(O):
    mbs = [W.to_numpy(m) for m in W.micro_batches(4, 3, 101, sigma=1.0, mean_scale="raw", seed=5)]
    one = O.norm_test(np.concatenate(mbs), eta=0.5, b_cur=12, b_max=3)
    acc = O.accumulated_norm_test(mbs, eta=0.5, b_cur=12, b_max=3)
    byS = O.accumulated_norm_test_by_sums(mbs, eta=0.5, b_cur=12, b_max=3)
    assert acc.stat == one.stat and acc.b_req == one.b_req and acc.batch_count == 12
    assert math.isclose(byS.stat, one.stat, rel_tol=1e-10)
    assert math.isclose(byS.mean_sqnorm, one.mean_sqnorm, rel_tol=1e-13)
    assert math.isclose(byS.sum_sqnorm, one.sum_sqnorm, rel_tol=1e-13)
    assert byS.b_req == one.b_req and byS.flags == one.flags
    # exact: integer micro-batches against the rational definition on the union
    rng = np.random.default_rng(2)
    ms = [int_matrix(rng, 2, 5) for _ in range(3)]
    ms[0][0, 0] += 1
    n, N, V, stat, b_req = exact_norm_test(np.concatenate(ms).tolist(), 0.5, 1)
    r = O.accumulated_norm_test_by_sums(ms, eta=0.5, b_cur=1, b_max=1 << 30)
    assert math.isclose(r.stat, float(stat), rel_tol=1e-13) and r.b_req == max(1, b_req)


def _explicit_weight_grad(X_i, D_i):
    """G_i[o][j] = sum_t delta_t[o] * x_t[j] in Python integers."""
    T, d_in, d_out = len(X_i), len(X_i[0]), len(D_i[0])
    return [[sum(int(D_i[t][o]) * int(X_i[t][j]) for t in range(T)) for j in range(d_in)]
            for o in range(d_out)]


def pin_linear_layer_brute_force(O):
    X, D = W.small_integer_layer(3, 5, 4, 6, seed=9)
    Xn, Dn = W.to_numpy(X), W.to_numpy(D)
    Xi, Di = X.float().numpy(), D.float().numpy()
    n, S = O.linear_layer_terms(Xn, Dn)
    assert S.shape == (6, 4)
    S_ref = np.zeros((6, 4))
    for i in range(3):
        G_i = np.array(_explicit_weight_grad(Xi[i].tolist(), Di[i].tolist()), dtype=np.float64)
        assert np.array_equal(O.per_sample_weight_grad(Xn[i], Dn[i]), G_i)
        # Gram identity: ||sum_t delta_t x_t^T||_F^2 = sum_{t,s} (x_t . x_s)(delta_t . delta_s)
        gram = sum(int(np.dot(Xi[i][t], Xi[i][s])) * int(np.dot(Di[i][t], Di[i][s]))
                   for t in range(5) for s in range(5))
        assert n[i] == float(gram) == float((G_i ** 2).sum())
        S_ref += G_i
    assert np.array_equal(S, S_ref)
    # rank one: a single token gives ||delta x^T||^2 = ||x||^2 ||delta||^2
    X1, D1 = W.small_integer_layer(2, 1, 7, 3, seed=4)
    n1, _ = O.linear_layer_terms(W.to_numpy(X1), W.to_numpy(D1))
    for i in range(2):
        assert n1[i] == float((X1[i].float() ** 2).sum() * (D1[i].float() ** 2).sum())


def pin_vector_param_terms(O):
    X, D = W.small_integer_layer(3, 5, 6, 6, seed=13)
    Xi, Di = X.float().numpy(), D.float().numpy()
    n, S = O.vector_param_terms(W.to_numpy(D))
    n2, S2 = O.vector_param_terms(W.to_numpy(D), W.to_numpy(X))
    S_ref, S2_ref = [0] * 6, [0] * 6
    for i in range(3):
        g = [sum(int(Di[i][t][j]) for t in range(5)) for j in range(6)]
        g2 = [sum(int(Di[i][t][j]) * int(Xi[i][t][j]) for t in range(5)) for j in range(6)]
        assert n[i] == float(sum(x * x for x in g)) and n2[i] == float(sum(x * x for x in g2))
        S_ref = [a + c for a, c in zip(S_ref, g)]
        S2_ref = [a + c for a, c in zip(S2_ref, g2)]
    assert S.tolist() == [float(x) for x in S_ref] and S2.tolist() == [float(x) for x in S2_ref]
    # a bias is the weight of a constant input 1: same norms as the linear layer with X = ones [T, 1]
    ones = torch.ones(3, 5, 1, dtype=torch.bfloat16)
    n_lin, S_lin = O.linear_layer_terms(W.to_numpy(ones), W.to_numpy(D))
    assert np.array_equal(n_lin, n) and np.array_equal(S_lin[:, 0], S)


def pin_embedding_terms(O):
    rng = np.random.default_rng(23)
    _, D = W.small_integer_layer(3, 7, 8, 8, seed=31)
    Dn, Di = W.to_numpy(D), D.float().numpy()
    V = 5
    ids = rng.integers(0, V, size=(3, 7))
    n, S = O.embedding_terms(ids, Dn, V)
    S_ref = [[0] * 8 for _ in range(V)]
    for i in range(3):
        G = [[0] * 8 for _ in range(V)]
        for t in range(7):
            for j in range(8):
                G[int(ids[i, t])][j] += int(Di[i][t][j])
        assert n[i] == float(sum(x * x for row in G for x in row))
        for v in range(V):
            for j in range(8):
                S_ref[v][j] += G[v][j]
    assert S.tolist() == [[float(x) for x in row] for row in S_ref]
    # a lookup is a linear layer on one-hot inputs: same per-sample norms, transposed sum
    onehot = torch.zeros(3, 7, V, dtype=torch.bfloat16)
    for i in range(3):
        for t in range(7):
            onehot[i, t, int(ids[i, t])] = 1.0
    n_lin, S_lin = O.linear_layer_terms(W.to_numpy(onehot), Dn)
    assert np.array_equal(n_lin, n) and np.array_equal(S_lin.T, S)
    # all tokens distinct: n_i = sum_t ||delta_t||^2; all equal: the bias case
    n_d, _ = O.embedding_terms(np.tile(np.arange(7), (3, 1)), Dn, 7)
    assert np.array_equal(n_d, (Di.astype(np.float64) ** 2).sum(axis=(1, 2)))
    n_e, S_e = O.embedding_terms(np.full((3, 7), 2), Dn, 4)
    n_b, S_b = O.vector_param_terms(Dn)
    assert np.array_equal(n_e, n_b) and np.array_equal(S_e[2], S_b) and not S_e[[0, 1, 3]].any()
    # tokens whose id names no row of the table (padding such as -100, ids >= V) have no gradient:
    # brute force over the tokens that remain; two padding tokens must not pair up with each other
    pad = ids.copy()
    pad[0, 1] = pad[0, 4] = -100
    pad[1, 0] = pad[1, 6] = V
    pad[2, 3] = V + 7
    n_p, S_p = O.embedding_terms(pad, Dn, V)
    S_ref = [[0] * 8 for _ in range(V)]
    for i in range(3):
        G = [[0] * 8 for _ in range(V)]
        for t in range(7):
            if 0 <= int(pad[i, t]) < V:
                for j in range(8):
                    G[int(pad[i, t])][j] += int(Di[i][t][j])
        assert n_p[i] == float(sum(x * x for row in G for x in row))
        for v in range(V):
            for j in range(8):
                S_ref[v][j] += G[v][j]
    assert S_p.tolist() == [[float(x) for x in row] for row in S_ref]
    n_none, S_none = O.embedding_terms(np.full((3, 7), -1), Dn, V)
    assert not n_none.any() and not S_none.any()


def pin_layers_test_two_routes(O):
    layers = [tuple(W.to_numpy(t) for t in W.linear_layer(4, 6, 8, 16, seed=1)),
              tuple(W.to_numpy(t) for t in W.linear_layer(4, 6, 16, 8, seed=2))]
    a = O.linear_layers_norm_test(layers, eta=0.5, b_cur=4, b_max=2, two_pass=True)
    c = O.linear_layers_norm_test(layers, eta=0.5, b_cur=4, b_max=2, two_pass=False)
    assert math.isclose(a.stat, c.stat, rel_tol=1e-9)
    assert math.isclose(a.mean_sqnorm, c.mean_sqnorm, rel_tol=1e-13)
    assert np.allclose(a.per_sample_sqnorm, c.per_sample_sqnorm, rtol=1e-13)
    assert (a.b_req, a.flags, a.accum_steps, a.b_micro) == (c.b_req, c.flags, c.accum_steps, c.b_micro)
    # exact rational check of the flattened definition on integer layers
    Xs, Ds = W.small_integer_layer(3, 2, 2, 3, seed=6)
    G = [sum(_explicit_weight_grad(Xs[i].float().tolist(), Ds[i].float().tolist()), []) for i in range(3)]
    n, N, V, stat, b_req = exact_norm_test(G, 0.5, 1)
    r = O.linear_layers_norm_test([(W.to_numpy(Xs), W.to_numpy(Ds))], eta=0.5, b_cur=1, b_max=1 << 30)
    if N != 0:
        assert math.isclose(r.stat, float(stat), rel_tol=1e-13) and r.b_req == max(1, b_req)


def pin_outer_step_fixture(O):
    for line in _rows("outer_step_dyadic.txt"):
        lhs, rhs = line.split("|")
        f = lhs.split()
        nesterov, K, lr, mu, theta, v = int(f[1]), int(f[2]), float(f[3]), float(f[4]), float(f[5]), float(f[6])
        inst = [np.array([float(x)], dtype=np.float32) for x in f[7:7 + K]]
        d, v_new, th_new = (float(x) for x in rhs.split())
        th, vv = O.outer_step(np.array([theta], dtype=np.float32), inst, np.array([v], dtype=np.float32),
                              lr=lr, momentum=mu, nesterov=bool(nesterov))
        assert th[0] == th_new and vv[0] == v_new, line


def pin_outer_step_special_cases(O):
    theta, inst, mom = W.outer_state(5, 333, seed=8, zero_momentum=False)
    th, inst_n, v = W.to_numpy(theta), [W.to_numpy(t) for t in inst], W.to_numpy(mom)
    mean = np.mean(np.stack([x.astype(np.float64) for x in inst_n]), axis=0)
    # K = 1, lr = 1, mu = 0 returns the instance parameters
    a, _ = O.outer_step(th, inst_n[:1], v, lr=1.0, momentum=0.0)
    assert np.allclose(a, inst_n[0].astype(np.float64), rtol=0, atol=1e-17)
    # any K, lr = 1, mu = 0: the LocalSGD average
    a, va = O.outer_step(th, inst_n, v, lr=1.0, momentum=0.0)
    assert np.allclose(a, mean, rtol=0, atol=1e-16)
    assert np.allclose(va, th.astype(np.float64) - mean, rtol=0, atol=1e-16)
    # zero momentum buffer: theta' = theta - lr (1 + mu)(theta - mean), v' = theta - mean
    a, va = O.outer_step(th, inst_n, np.zeros_like(v), lr=0.7, momentum=0.9)
    d = th.astype(np.float64) - mean
    assert np.allclose(a, th - 0.7 * 1.9 * d, rtol=0, atol=1e-15)
    assert np.allclose(va, d, rtol=0, atol=1e-16)
    # instance permutation
    p, vp = O.outer_step(th, inst_n[::-1], np.zeros_like(v), lr=0.7, momentum=0.9)
    assert np.allclose(p, a, rtol=0, atol=1e-16) and np.allclose(vp, va, rtol=0, atol=1e-16)
    # bf16 instances are widened exactly
    inst_b = [t.to(torch.bfloat16) for t in inst]
    b, _ = O.outer_step(th, [W.to_numpy(t) for t in inst_b], v, lr=1.0, momentum=0.0)
    assert np.allclose(b, np.mean(np.stack([t.double().numpy() for t in inst_b]), axis=0), rtol=0, atol=1e-16)


def pin_outer_step_matches_library_sgd(O):
    """With the pseudo-gradient as the gradient, the reading of OuterOpt is the
    library's SGD with momentum (dampening 0), Nesterov or not, over several steps."""
    theta, inst, mom = W.outer_state(3, 64, seed=12)
    for nesterov in (True, False):
        p = torch.nn.Parameter(theta.double().clone())
        opt = torch.optim.SGD([p], lr=0.7, momentum=0.9, nesterov=nesterov, dampening=0.0)
        th, v = W.to_numpy(theta).astype(np.float64), np.zeros(64)
        for step in range(3):
            cur = [(t.double() + 0.01 * step).numpy() for t in inst]
            p.grad = torch.from_numpy(np.mean([th - c for c in cur], axis=0))
            opt.step()
            th, v = O.outer_step(th, cur, v, lr=0.7, momentum=0.9, nesterov=nesterov)
            assert np.allclose(th, p.detach().numpy(), rtol=1e-13, atol=1e-16)


def pin_merge(O):
    assert O.check_merge([8, 2, 5, 2], 2) == [1, 3]
    assert O.check_merge([8, 2, 5, 2], 0) == []
    assert O.check_merge([8], 1) == []
    assert O.check_merge([8, 2], 3) == []
    assert O.check_merge([8, 2, 5], 3) == [1, 2, 0]
    xs = [np.array([1.0, 2.0], dtype=np.float32), np.array([3.0, -2.0], dtype=np.float32),
          np.array([0.0, 8.0], dtype=np.float32)]
    x, rep = O.do_merge(xs, [1, 3, 4])
    assert np.array_equal(x, np.array([10.0 / 8, (2 - 6 + 32) / 8.0])) and rep == 2
    x, rep = O.do_merge(xs[:2], [2, 2])
    assert np.array_equal(x, np.array([2.0, 0.0])) and rep == 0


def exact_inner_product_tests(G, theta, nu, ddof):
    """The two inner-product statistics in exact rationals, from their definitions."""
    b, P = len(G), len(G[0])
    g = [[Fraction(x) for x in row] for row in G]
    gbar = [sum(g[i][j] for i in range(b)) / b for j in range(P)]
    N = sum(x * x for x in gbar)
    p = [sum(g[i][j] * gbar[j] for j in range(P)) for i in range(b)]
    pbar = sum(p) / b
    var_ip = sum((x - pbar) ** 2 for x in p) / (b - ddof)
    o = [[g[i][j] - p[i] / N * gbar[j] for j in range(P)] for i in range(b)]
    obar = [sum(o[i][j] for i in range(b)) / b for j in range(P)]
    var_o = sum((o[i][j] - obar[j]) ** 2 for i in range(b) for j in range(P)) / (b - ddof)
    return var_ip / (Fraction(theta) ** 2 * N * N), var_o / (Fraction(nu) ** 2 * N)


def pin_inner_product_tests(O):
    rng = np.random.default_rng(17)
    for b, P, theta, nu, ddof in [(3, 4, 0.5, 0.25, 1), (5, 6, 0.125, 0.5, 1), (4, 3, 2.0, 1.0, 0)]:
        G = int_matrix(rng, b, P)
        G[:, 0] += 3.0      # keep the mean away from zero
        s_ip, s_or = exact_inner_product_tests(G.tolist(), theta, nu, ddof)
        r = O.inner_product_tests(G, theta=theta, nu=nu, ddof=ddof, b_cur=1)
        assert math.isclose(r.stat_ip, float(s_ip), rel_tol=1e-12)
        assert math.isclose(r.stat_orth, float(s_or), rel_tol=1e-12)
        assert r.b_ip == max(1, math.ceil(s_ip))
        assert r.b_aug == max(r.b_ip, max(1, math.ceil(s_or)))
    # orthonormal gradients: every <g_i, gbar> equals ||gbar||^2, so the inner-product
    # statistic vanishes; the orthogonal parts e_i - gbar give variance 1 and b / nu^2
    G = np.eye(16, dtype=np.float32)[:8]
    r = O.inner_product_tests(G, theta=0.01, nu=0.5, b_cur=1)
    assert r.stat_ip < 1e-25 and r.b_ip == 1
    assert math.isclose(r.var_orth, 1.0, rel_tol=1e-14) and math.isclose(r.stat_orth, 32.0, rel_tol=1e-14)
    assert r.b_aug == 32 and r.flags & O.FLAG_GROW
    # collinear gradients g_i = a_i u: no orthogonal part; stat_ip = Var(a) / (theta^2 abar^2)
    a = np.array([1.0, 2.0, 3.0, 6.0])
    u = np.zeros(8); u[2] = 1.0
    G = (a[:, None] * u[None, :]).astype(np.float32)
    r = O.inner_product_tests(G, theta=0.5, nu=0.3, b_cur=1)
    assert r.var_orth < 1e-25 and math.isclose(r.stat_ip, a.var(ddof=1) / (0.25 * a.mean() ** 2), rel_tol=1e-14)
    assert r.b_aug == r.b_ip == math.ceil(a.var(ddof=1) / (0.25 * 9.0))
    # scale invariance of both statistics, caps, degenerate cases
    G = W.to_numpy(W.per_sample_grads(6, 300, sigma=0.5, seed=4))
    x = O.inner_product_tests(G, theta=0.1, nu=0.3)
    y = O.inner_product_tests(G * np.float32(8.0), theta=0.1, nu=0.3)
    assert math.isclose(x.stat_ip, y.stat_ip, rel_tol=1e-12) and math.isclose(x.stat_orth, y.stat_orth, rel_tol=1e-12)
    assert O.inner_product_tests(G, theta=0.1, nu=0.3, b_cap=3).b_aug == 3
    z = O.inner_product_tests(G[:1], theta=0.1, nu=0.3, b_cur=5)
    assert z.flags & O.FLAG_UNDEFINED and z.b_ip == z.b_aug == 5
    zero = np.array([[1.0, -1.0], [-1.0, 1.0]], dtype=np.float32)
    assert O.inner_product_tests(zero, theta=0.1, nu=0.3).flags & O.FLAG_ZERO_MEAN
    with pytest.raises(ValueError):
        O.inner_product_tests(G, theta=0.0, nu=0.3)


def pin_nonfinite_sums_leave_the_batch_alone(O):
    # an Inf or NaN anywhere leaves no statistic: flag 16, V = stat = 0, b stays at max(1, b_cur), no NaN in the plan
    for bad in (math.inf, -math.inf, math.nan):
        for args in ((bad, 1.0, 1.0), (10.0, bad, 1.0), (10.0, 1.0, bad)):
            r = O.decide(*args, 8, eta=0.5, b_cur=6, b_max=4)
            assert r.flags == O.FLAG_NONFINITE and r.b_req == 6 and r.stat == 0.0 and r.variance == 0.0
            assert (r.accum_steps, r.b_micro) == (1, 4)
    assert O.decide(math.nan, 1.0, 1.0, 1, eta=0.5, b_cur=0).b_req == 1        # checked before UNDEFINED
    assert O.decide(math.nan, 1.0, 1.0, 8, eta=0.5, b_cur=3, b_max=1).flags == O.FLAG_NONFINITE | O.FLAG_ACCUMULATE
    G = W.to_numpy(W.per_sample_grads(4, 64, seed=3)).copy()
    for bad in (np.float32(np.inf), np.float32(np.nan), np.float32(3e38)):     # 3e38 squared overflows only in fp32
        H = G.copy()
        H[2, 5] = bad
        r = O.norm_test(H, eta=0.5, b_cur=4, b_max=32)
        if np.isfinite(bad):
            assert r.flags & O.FLAG_NONFINITE == 0 and math.isfinite(r.stat)   # fp64 holds 9e76
        else:
            assert r.flags & O.FLAG_NONFINITE and r.b_req == 4
            ip = O.inner_product_tests(H, theta=0.1, nu=0.3, b_cur=4)
            assert ip.flags & O.FLAG_NONFINITE and ip.b_ip == ip.b_aug == 4
    assert O.decide(10.0, 1.0, 1.0, 8, eta=0.5).flags & O.FLAG_NONFINITE == 0


PINS = [v for k, v in sorted(globals().items()) if k.startswith("pin_")]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(ORACLE)


# ------------------------------------------------------------- mutation checks
MUTANTS = [
    # (description, text in the oracle source, replacement)
    ("variance normaliser", "V = dev / (b - ddof)", "V = dev / b"),
    ("mean not divided by b", "gbar = total / b", "gbar = total"),
    ("deviation from zero instead of the mean", "c = g - gbar", "c = g"),
    ("eta not squared", "variance / (eta * eta * mean_sqnorm)", "variance / (eta * mean_sqnorm)"),
    ("floor instead of ceil", "max(1, math.ceil(r.stat))", "max(1, math.floor(r.stat))"),
    ("switch threshold >= ", "if b_req > switch_n * b_max:", "if b_req >= switch_n * b_max:"),
    ("switch threshold without n", "if b_req > switch_n * b_max:", "if b_req > b_max:"),
    ("accum floor", "return True, -(-b_req // b_max), b_max", "return True, b_req // b_max, b_max"),
    ("micro-batch not clipped", "return False, 1, min(b_req, b_max)", "return False, 1, b_req"),
    ("grow compares >=", "if r.b_req > b_cur:", "if r.b_req >= b_cur:"),
    ("weight gradient transposed", "return widen(D_i).T @ widen(X_i)", "return widen(X_i).T @ widen(D_i)"),
    ("identity with the wrong sign", "V = (Q - b * N) / (b - ddof)", "V = (Q + b * N) / (b - ddof)"),
    ("identity without b", "V = (Q - b * N) / (b - ddof)", "V = (Q - N) / (b - ddof)"),
    ("mean norm from the sum", "m = np.asarray(S, dtype=np.float64).ravel() / b", "m = np.asarray(S, dtype=np.float64).ravel()"),
    ("pseudo-gradient sign", "acc += th - widen(instances[k])", "acc += widen(instances[k]) - th"),
    ("pseudo-gradient not averaged", "d = acc / K", "d = acc"),
    ("momentum term dropped", "v_new = momentum * v + d", "v_new = d"),
    ("nesterov look-ahead uses old v", "u = d + momentum * v_new if nesterov", "u = d + momentum * v if nesterov"),
    ("lr dropped", "return th - lr * u, v_new", "return th - u, v_new"),
    ("update sign", "return th - lr * u, v_new", "return th + lr * u, v_new"),
    ("bf16 widening shift", "<< np.uint32(16)", "<< np.uint32(15)"),
    ("merge takes the largest", "order = sorted(range(k), key=lambda i: (b_req[i], i))",
     "order = sorted(range(k), key=lambda i: (-b_req[i], i))"),
    ("merge unweighted", "x += float(b) * widen(p)", "x += widen(p)"),
    ("embedding rows overwritten instead of summed", "np.add.at(G_i, ids[i][inside], widen(D[i])[inside])",
     "G_i[ids[i][inside]] = widen(D[i])[inside]"),
    ("padding ids wrap around into the table", "inside = (ids[i] >= 0) & (ids[i] < V)", "inside = ids[i] < V"),
    ("non-finite sums pass through", "if not (math.isfinite(sum_sqnorm) and math.isfinite(mean_sqnorm) and math.isfinite(variance)):",
     "if False:"),
    ("vector parameter summed over features", "g = (d * widen(X[i])).sum(axis=0) if X is not None else d.sum(axis=0)",
     "g = (d * widen(X[i])).sum(axis=1) if X is not None else d.sum(axis=1)"),
    ("gain gradient without the input", "g = (d * widen(X[i])).sum(axis=0) if X is not None else d.sum(axis=0)",
     "g = d.sum(axis=0)"),
    ("inner products against the sum", "p[i] = float(np.dot(widen(G[i]), gbar))", "p[i] = float(np.dot(widen(G[i]), total))"),
    ("inner-product statistic with ||gbar||^2 only", "r.var_ip / (theta * theta * N * N)", "r.var_ip / (theta * theta * N)"),
    ("projection not normalised", "c = widen(G[i]) - (p[i] / N) * gbar - obar", "c = widen(G[i]) - p[i] * gbar - obar"),
    ("orthogonal statistic with theta", "r.var_orth / (nu * nu * N)", "r.var_orth / (theta * theta * N)"),
    ("augmented test takes the min", "r.b_aug = max(r.b_ip, b_orth)", "r.b_aug = min(r.b_ip, b_orth)"),
    ("inner-product variance uncentred", "float(((p - pbar) ** 2).sum()) / (b - ddof)", "float((p ** 2).sum()) / (b - ddof)"),
]


def _mutated_oracle(old, new):
    path = ORACLE.__file__
    with open(path) as f:
        src = f.read()
    assert src.count(old) >= 1, f"mutation target not found: {old!r}"
    mod = types.ModuleType("oracle_mutant")
    mod.__file__ = path
    sys.modules["oracle_mutant"] = mod          # dataclasses look the module up by name
    try:
        exec(compile(src.replace(old, new), path, "exec"), mod.__dict__)
    finally:
        sys.modules.pop("oracle_mutant", None)
    return mod


@pytest.mark.parametrize("desc,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutants_are_caught(desc, old, new):
    mutant = _mutated_oracle(old, new)
    caught = []
    for pin in PINS:
        try:
            pin(mutant)
        except AssertionError:
            caught.append(pin.__name__)
        except Exception:
            caught.append(pin.__name__)
    assert caught, f"no pin notices: {desc}"
