"""GPU parity: adloco_vector_param_sqnorm (per-sample gradient norms of biases and
elementwise gains) against the oracle."""
import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_BF16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("B,T,d", [(3, 5, 8), (32, 1024, 768), (4, 1000, 3072), (7, 33, 264), (1, 1, 16), (5, 130, 520)])
@pytest.mark.parametrize("gain", [False, True])
def test_matches_oracle(ctx, B, T, d, gain):
    X, D = W.linear_layer(B, T, d, d, seed=B + T + d, delta_std=1.0, device=DEV)
    n = torch.full((B,), -3.0, device=DEV)
    S = torch.full((d,), -3.0, device=DEV)
    ctx.vector_param_sqnorm(D, n, X=X if gain else None, grad_sum=S)
    torch.cuda.synchronize()
    n_ref, S_ref = O.vector_param_terms(W.to_numpy(D), W.to_numpy(X) if gain else None)
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)


def test_integer_inputs_exact_accumulation_and_errors(ctx):
    X, D = W.small_integer_layer(3, 50, 24, 24, seed=5, device=DEV)
    n = torch.zeros(3, device=DEV)
    S = torch.zeros(24, device=DEV)
    ctx.vector_param_sqnorm(D, n, X=X, grad_sum=S)
    n_ref, S_ref = O.vector_param_terms(W.to_numpy(D), W.to_numpy(X))
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy().astype(np.float64), n_ref) and np.array_equal(S.cpu().numpy().astype(np.float64), S_ref)
    ctx.vector_param_sqnorm(D, n, X=X, grad_sum=S, accumulate_norms=True, accumulate_sum=True)
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy().astype(np.float64), 2 * n_ref) and np.array_equal(S.cpu().numpy().astype(np.float64), 2 * S_ref)
    n2 = torch.zeros(3, device=DEV)
    ctx.vector_param_sqnorm(D, n2)                      # bias, no sum buffer
    torch.cuda.synchronize()
    assert np.array_equal(n2.cpu().numpy().astype(np.float64), O.vector_param_terms(W.to_numpy(D))[0])
    before = ctx.launch_count
    with pytest.raises(A.AdlocoError) as e:
        ctx.vector_param_sqnorm(D[:, :, :12].contiguous(), n2)
    assert e.value.status == A.ERR_UNSUPPORTED and ctx.launch_count == before
