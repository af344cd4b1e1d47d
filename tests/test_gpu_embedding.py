"""GPU parity: adloco_embedding_sqnorm (per-sample gradient norms of an embedding
table -- by grouping a sample's tokens by id and summing each group's rows, or, for
sequences beyond 4096 tokens, through the Gram identity with a token-equality mask;
scatter-added gradient sum) against the oracle, which scatters every sample's gradient
explicitly."""
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


def _ids(B, T, V, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randint(0, V, (B, T), generator=g, device=DEV, dtype=torch.int32)


@pytest.mark.parametrize("B,T,d,V", [(3, 7, 8, 5), (4, 128, 64, 20), (2, 300, 72, 40), (5, 1024, 768, 1000),
                                     (3, 257, 136, 3), (1, 1, 8, 1), (6, 513, 256, 50257),
                                     (2, 4096, 72, 300),     # the longest sequence the grouping kernel takes (160 KB of shared memory)
                                     (1, 4100, 64, 50),      # beyond it: the masked Gram kernel
                                     (40, 96, 1048, 7),      # d > 1024: several feature passes; groups of ~14 rows
                                     (2, 900, 264, 4)])      # groups of > 64 rows: summed by the whole block
def test_matches_oracle(ctx, B, T, d, V):
    _, D = W.linear_layer(B, T, 8, d, seed=B + T, delta_std=1.0, device=DEV)
    ids = _ids(B, T, V, seed=d)
    n = torch.full((B,), -1.0, device=DEV)
    S = torch.full((V, d), -1.0, device=DEV)
    ctx.embedding_sqnorm(ids, D, V, n, grad_sum=S)
    torch.cuda.synchronize()
    n_ref, S_ref = O.embedding_terms(ids.cpu().numpy(), W.to_numpy(D), V)
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16), (n.cpu().numpy() / n_ref)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    assert ctx.device_status() == 0


def test_exact_on_integers_and_special_id_patterns(ctx):
    _, D = W.small_integer_layer(3, 200, 8, 24, seed=3, device=DEV)
    Dn = W.to_numpy(D)
    n = torch.zeros(3, device=DEV)
    S = torch.zeros(9, 24, device=DEV)
    ids = _ids(3, 200, 9, seed=1)
    ctx.embedding_sqnorm(ids, D, 9, n, grad_sum=S)
    torch.cuda.synchronize()
    n_ref, S_ref = O.embedding_terms(ids.cpu().numpy(), Dn, 9)
    assert np.array_equal(n.cpu().numpy().astype(np.float64), n_ref) and np.array_equal(S.cpu().numpy().astype(np.float64), S_ref)
    # accumulate flags
    ctx.embedding_sqnorm(ids, D, 9, n, accumulate_norms=True, grad_sum=S, accumulate_sum=True)
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy().astype(np.float64), 2 * n_ref) and np.array_equal(S.cpu().numpy().astype(np.float64), 2 * S_ref)
    # positions as ids (a learned positional embedding): every token distinct, n_i = sum_t |delta_t|^2
    pos = torch.arange(200, device=DEV, dtype=torch.int32).repeat(3, 1).contiguous()
    ctx.embedding_sqnorm(pos, D, 200, n)
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy().astype(np.float64), (D.double() ** 2).sum((1, 2)).cpu().numpy())
    # one id everywhere: the bias case
    same = torch.full((3, 200), 4, device=DEV, dtype=torch.int32)
    ctx.embedding_sqnorm(same, D, 9, n)
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy().astype(np.float64), O.vector_param_terms(Dn)[0])
    before = ctx.launch_count
    with pytest.raises(A.AdlocoError) as e:
        ctx.embedding_sqnorm(ids, D[:, :, :12].contiguous(), 9, n)
    assert e.value.status == A.ERR_UNSUPPORTED and ctx.launch_count == before


def test_ids_outside_the_table_are_dropped_from_norms_and_sum(ctx):
    """Padding / ignore ids (-100, ids >= V) look up no row: they add nothing to n_i or S, and two
    tokens that share such an id do not pair up in the masked Gram sum."""
    B, T, d, V = 4, 300, 64, 11
    _, D = W.small_integer_layer(B, T, 8, d, seed=8, device=DEV)
    ids = _ids(B, T, V, seed=2)
    ids[0, 5:90] = -100                     # a run of one repeated padding id, crossing a 128-token block
    ids[1, ::3] = V                         # first id past the table
    ids[2, 200:] = V + 1000
    ids[3, :] = -1                          # a sample with no token inside the table
    n = torch.full((B,), -1.0, device=DEV)
    S = torch.full((V, d), -1.0, device=DEV)
    ctx.embedding_sqnorm(ids, D, V, n, grad_sum=S)
    torch.cuda.synchronize()
    n_ref, S_ref = O.embedding_terms(ids.cpu().numpy(), W.to_numpy(D), V)
    assert np.array_equal(n.cpu().numpy().astype(np.float64), n_ref) and n_ref[3] == 0.0
    assert np.array_equal(S.cpu().numpy().astype(np.float64), S_ref)
