"""GPU parity: adloco_gram_sqnorm (Gram-identity per-sample norms and the
mean-gradient GEMM on the tensor cores) against the fp64 oracle, which forms
every per-sample weight gradient explicitly."""
import math

import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_BF16, assert_test_result

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _gpu_layer(ctx, X, D, want_S=True, method="gram"):
    B = X.shape[0]
    n = torch.full((B,), -5.0, device=DEV)
    S = torch.full((D.shape[2], X.shape[2]), -5.0, device=DEV) if want_S else None
    if method == "gram":
        ctx.gram_sqnorm(X, D, n, grad_sum=S)
    else:
        ctx.linear_sqnorm(X, D, n, grad_sum=S, method=method)
    torch.cuda.synchronize()
    return n, S


METHODS = ["gram", "gram_pair", "direct", "pair", "auto"]


@pytest.mark.parametrize("method", METHODS)
def test_small_integer_layer_is_exact(ctx, method):
    # every product and partial sum is an integer below 2^24: the result must be exact
    X, D = W.small_integer_layer(3, 5, 8, 16, seed=9, device=DEV)
    n, S = _gpu_layer(ctx, X, D, method=method)
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.array_equal(n.cpu().numpy().astype(np.float64), n_ref)
    assert np.array_equal(S.cpu().numpy().astype(np.float64), S_ref)


@pytest.mark.parametrize("B,T,d_in,d_out", [
    (2, 128, 64, 64),        # one tile, one chunk
    (3, 256, 128, 192),      # off-diagonal tiles, several chunks
    (2, 200, 72, 40),        # ragged T (not a multiple of 128 or 64), ragged d (multiples of 8 only)
    (5, 1, 8, 8),            # a single token: n_i = |x|^2 |delta|^2
    (1, 384, 768, 256),      # 3x3 token tiles, 12 + 4 chunks: the ring wraps
    (4, 130, 264, 520),      # d_in > 256 and d_out > 512: several output tiles, ragged
    (33, 64, 32, 48),
    (2, 2048, 256, 512),     # long sequence: 16 token blocks per side, 72 tile items per sample
    (1, 1153, 64, 64),       # odd number of blocks (10) with a ragged last one
])
@pytest.mark.parametrize("method", METHODS)
def test_layer_matches_oracle(ctx, B, T, d_in, d_out, method):
    X, D = W.linear_layer(B, T, d_in, d_out, seed=B + T, device=DEV)
    n, S = _gpu_layer(ctx, X, D, method=method)
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16, atol=0), (n.cpu().numpy() / n_ref)
    scale = np.abs(S_ref).max()
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * scale * 0.05)
    if T == 1:
        x2 = (X.double() ** 2).sum((1, 2)).cpu().numpy()
        d2 = (D.double() ** 2).sum((1, 2)).cpu().numpy()
        assert np.allclose(n.cpu().numpy(), x2 * d2, rtol=1e-5)


def test_accumulate_flags_and_unsupported_shapes(ctx):
    X, D = W.linear_layer(2, 96, 64, 64, seed=1, device=DEV)
    n, S = _gpu_layer(ctx, X, D)
    n2, S2 = n.clone(), S.clone()
    ctx.gram_sqnorm(X, D, n2, accumulate_norms=True, grad_sum=S2, accumulate_sum=True)
    torch.cuda.synchronize()
    # fp32 reductions into S arrive in no fixed order: allow for a few ulp of the largest terms
    assert torch.allclose(n2, 2 * n, rtol=1e-5) and torch.allclose(S2, 2 * S, rtol=1e-5, atol=1e-5 * float(S.abs().max()))
    # without the sum buffer only the norms are computed
    n3 = torch.zeros(2, device=DEV)
    ctx.gram_sqnorm(X, D, n3)
    torch.cuda.synchronize()
    assert torch.allclose(n3, n, rtol=1e-5)
    Xb, Db = W.linear_layer(2, 16, 12, 64, seed=1, device=DEV)      # d_in not a multiple of 8
    before = ctx.launch_count
    with pytest.raises(A.AdlocoError) as e:
        ctx.gram_sqnorm(Xb, Db, n3)
    assert e.value.status == A.ERR_UNSUPPORTED and ctx.launch_count == before


def test_direct_route_accumulates_and_may_skip_the_sum(ctx):
    X, D = W.linear_layer(3, 200, 72, 264, seed=4, device=DEV)
    n, S = _gpu_layer(ctx, X, D, method="direct")
    n2, S2 = n.clone(), S.clone()
    ctx.linear_sqnorm(X, D, n2, accumulate_norms=True, grad_sum=S2, accumulate_sum=True, method="direct")
    n3 = torch.zeros(3, device=DEV)
    ctx.linear_sqnorm(X, D, n3, method="direct")              # no sum buffer
    torch.cuda.synchronize()
    assert torch.allclose(n2, 2 * n, rtol=1e-5) and torch.allclose(S2, 2 * S, rtol=1e-5, atol=1e-5 * float(S.abs().max()))
    assert torch.allclose(n3, n, rtol=1e-5)
    ng, Sg = _gpu_layer(ctx, X, D, method="gram")            # the two routes agree with each other as well
    assert torch.allclose(ng, n, rtol=2e-3) and torch.allclose(Sg, S, rtol=1e-4, atol=1e-4 * float(S.abs().max()))
    with pytest.raises(A.AdlocoError) as e:
        ctx.lib.adloco_linear_sqnorm  # noqa: B018  (symbol exists)
        ctx.check(ctx.lib.adloco_linear_sqnorm(ctx.h, X.data_ptr(), D.data_ptr(), 3, 200, 72, 264, n.data_ptr(), 0,
                                               None, 0, 7, None), "adloco_linear_sqnorm")
    assert e.value.status == A.ERR_INVALID_ARG


def test_whole_model_switch_mode_small(ctx):
    """Two blocks of four linear layers, a batch of 12 processed as 3 accumulated
    micro-batches of 4: per-sample norms accumulate across layers, gradient sums
    across micro-batches, one test at the end."""
    shapes = [(64, 192), (64, 64), (64, 256), (256, 64)] * 2
    n_micro, b, T = 3, 4, 160
    data = [[W.linear_layer(b, T, di, do, seed=1000 * j + l, device=DEV) for l, (di, do) in enumerate(shapes)]
            for j in range(n_micro)]
    sums = [torch.empty(do, di, device=DEV) for di, do in shapes]
    acc = A.Accumulator(ctx, sums)
    acc.reset()
    n_mb = torch.zeros(b, device=DEV)
    for j in range(n_micro):
        for l, (X, D) in enumerate(data[j]):
            ctx.gram_sqnorm(X, D, n_mb, accumulate_norms=(l > 0), grad_sum=sums[l], accumulate_sum=True)
        acc.accumulate(per_sample_sqnorm=n_mb)
    p = A.make_params(0.5, b_cur=12, b_max=4)
    r = acc.finalize(p)
    layers = [(np.concatenate([W.to_numpy(data[j][l][0]) for j in range(n_micro)]),
               np.concatenate([W.to_numpy(data[j][l][1]) for j in range(n_micro)])) for l in range(len(shapes))]
    ora = O.linear_layers_norm_test(layers, eta=0.5, b_cur=12, b_max=4, two_pass=True)
    # V comes from Q - b N here: scale the tolerance by the cancellation it suffers
    kappa = ora.sum_sqnorm / (ora.variance * 11)
    assert_test_result(r, ora, p, TOL_BF16, stat_tol=TOL_BF16 * max(1.0, kappa), what="whole model")
    assert r.flags & A.FLAG_ACCUMULATE
    acc.close()


@pytest.mark.parametrize("method", ["gram", "gram_pair", "direct", "pair"])
def test_a_wait_that_runs_out_raises_the_status_and_the_context_stays_usable(method):
    """Every in-kernel wait is bounded.  With the bound set to one nanosecond the
    first wait that is not satisfied at once gives up: the kernel must leave through
    its teardown (copies landed, tensor memory freed), raise ADLOCO_ERR_TIMEOUT in the
    status word, and the next call with the normal bound must be correct again."""
    c = A.Context(0)
    X, D = W.linear_layer(8, 512, 256, 512, seed=77, device=DEV)
    n = torch.zeros(8, device=DEV)
    S = torch.zeros(512, 256, device=DEV)
    assert c.device_status() == 0
    c.set_wait_limit(1)
    c.linear_sqnorm(X, D, n, grad_sum=S, method=method)
    assert c.device_status(clear=True) == A.ERR_TIMEOUT
    assert c.device_status() == 0
    c.set_wait_limit(2_000_000_000)
    c.linear_sqnorm(X, D, n, grad_sum=S, method=method)
    assert c.device_status() == 0
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    c.close()


def test_every_parameter_kind_in_one_accumulated_test(ctx):
    """A small transformer-shaped parameter set -- token and positional embeddings, a
    LayerNorm gain and bias, two linear layers with biases -- tested as one model over two
    micro-batches.  The oracle materialises every per-sample gradient, concatenates them
    and applies the definition of the norm test."""
    B, n_micro, T, d, V = 4, 2, 96, 64, 30
    sizes = {"tok": (V, d), "pos": (T, d), "ln_g": (d,), "ln_b": (d,), "w1": (128, d), "b1": (128,), "w2": (d, 128), "b2": (d,)}
    S = {k: torch.empty(*shape, device=DEV) for k, shape in sizes.items()}
    acc = A.Accumulator(ctx, list(S.values()))
    acc.reset()
    pos = torch.arange(T, device=DEV, dtype=torch.int32).repeat(B, 1).contiguous()
    flat = []
    for j in range(n_micro):
        g = torch.Generator(device=DEV)
        g.manual_seed(500 + j)
        ids = torch.randint(0, V, (B, T), generator=g, device=DEV, dtype=torch.int32)
        Xh, De = W.linear_layer(B, T, d, d, seed=10 + j, delta_std=0.3, device=DEV)      # normalised input, grad at the embedding / LN output
        X1, D1 = W.linear_layer(B, T, d, 128, seed=20 + j, delta_std=0.1, device=DEV)
        X2, D2 = W.linear_layer(B, T, 128, d, seed=30 + j, delta_std=0.1, device=DEV)
        n = torch.zeros(B, device=DEV)
        ctx.embedding_sqnorm(ids, De, V, n, grad_sum=S["tok"], accumulate_sum=True)
        ctx.embedding_sqnorm(pos, De, T, n, accumulate_norms=True, grad_sum=S["pos"], accumulate_sum=True)
        ctx.vector_param_sqnorm(De, n, X=Xh, accumulate_norms=True, grad_sum=S["ln_g"], accumulate_sum=True)
        ctx.vector_param_sqnorm(De, n, accumulate_norms=True, grad_sum=S["ln_b"], accumulate_sum=True)
        ctx.linear_sqnorm(X1, D1, n, accumulate_norms=True, grad_sum=S["w1"], accumulate_sum=True, method="gram")
        ctx.vector_param_sqnorm(D1, n, accumulate_norms=True, grad_sum=S["b1"], accumulate_sum=True)
        ctx.linear_sqnorm(X2, D2, n, accumulate_norms=True, grad_sum=S["w2"], accumulate_sum=True, method="direct")
        ctx.vector_param_sqnorm(D2, n, accumulate_norms=True, grad_sum=S["b2"], accumulate_sum=True)
        acc.accumulate(per_sample_sqnorm=n)
        # the oracle's explicit per-sample gradients, in the same parameter order
        idn, De_n, Xh_n = ids.cpu().numpy(), O.widen(W.to_numpy(De)), O.widen(W.to_numpy(Xh))
        for i in range(B):
            tok = np.zeros((V, d)); np.add.at(tok, idn[i], De_n[i])
            parts = [tok.ravel(), De_n[i].ravel(), (De_n[i] * Xh_n[i]).sum(0), De_n[i].sum(0),
                     O.per_sample_weight_grad(W.to_numpy(X1[i]), W.to_numpy(D1[i])).ravel(), O.widen(W.to_numpy(D1[i])).sum(0),
                     O.per_sample_weight_grad(W.to_numpy(X2[i]), W.to_numpy(D2[i])).ravel(), O.widen(W.to_numpy(D2[i])).sum(0)]
            flat.append(np.concatenate(parts))
    p = A.make_params(0.5, b_cur=B * n_micro, b_max=B)
    r = acc.finalize(p)
    ora = O.norm_test(np.stack(flat), eta=0.5, b_cur=B * n_micro, b_max=B, want_sum=True)
    kappa = ora.sum_sqnorm / max(ora.variance * (B * n_micro - 1), 1e-300)
    assert_test_result(r, ora, p, TOL_BF16, stat_tol=TOL_BF16 * max(1.0, kappa), what="all parameter kinds")
    got = np.concatenate([S[k].cpu().numpy().ravel() for k in sizes])
    assert np.allclose(got, ora.grad_sum, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(ora.grad_sum).max() * 0.05)
    acc.close()
