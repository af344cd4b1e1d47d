"""GPU parity of the tensor-core kernels on the path they take at full size: a CTA
that runs several work units in a row.  Then the second accumulator buffer in tensor
memory, the barrier phases on re-use, the shared-memory ring wrapping across units and
the gradient-sum tile carried across samples are all in play; a single-unit launch
exercises none of them.  Every case is compared element by element with the oracle's
explicit per-sample gradients."""
import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import TOL_BF16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SMS = 148


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _check_layer(ctx, X, D, method, what):
    B = X.shape[0]
    n = torch.full((B,), -3.0, device=DEV)
    S = torch.full((D.shape[2], X.shape[2]), -3.0, device=DEV)
    ctx.linear_sqnorm(X, D, n, grad_sum=S, method=method)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0, what
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16, atol=0), (what, n.cpu().numpy() / n_ref)
    scale = np.abs(S_ref).max()
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * scale * 0.05), what
    # the norms alone (no sum buffer) take the same multi-unit path
    n2 = torch.full((B,), -3.0, device=DEV)
    ctx.linear_sqnorm(X, D, n2, method=method)
    torch.cuda.synchronize()
    assert np.allclose(n2.cpu().numpy(), n_ref, rtol=TOL_BF16, atol=0), what


# (B, T, d_in, d_out): what the split of the (tile, sample) units looks like on 148 SMs
#   128x256 tiles (direct) / 256x256 tiles (mean gradient)
MULTI_UNIT_SHAPES = [
    (3, 128, 2048, 2560),    # 160 / 80 tiles: direct has more tiles than SMs, whole batch per item, 12 CTAs take two items
    (7, 128, 768, 3072),     # 72 / 36 tiles: chunks of 4 and 3 samples (ragged last chunk), odd unit counts
    (5, 200, 520, 1032),     # ragged T, d_in, d_out: 27 / 15 tiles, several samples per CTA with clipped boxes
    (9, 64, 256, 128),       # one tile, nine samples in nine CTAs ... and
    (40, 64, 512, 1024),     # 16 / 8 tiles: chunks of 5 / 3 samples
    (2, 1024, 4096, 1280),   # 160 tiles again with a long contraction: the ring wraps many times per unit
]


@pytest.mark.parametrize("B,T,d_in,d_out", MULTI_UNIT_SHAPES)
@pytest.mark.parametrize("method", ["direct", "pair", "gram", "gram_pair"])
def test_ctas_with_several_units_match_the_oracle(ctx, B, T, d_in, d_out, method):
    X, D = W.linear_layer(B, T, d_in, d_out, seed=7 * B + T, device=DEV)
    _check_layer(ctx, X, D, method, f"{method} B={B} T={T} {d_in}->{d_out}")


@pytest.mark.parametrize("method", ["direct", "pair", "gram", "gram_pair"])
def test_several_units_exact_on_integers(ctx, method):
    # T = 16 keeps every entry of a per-sample gradient below 2^8 and every sum below 2^24: exact in fp32
    X, D = W.small_integer_layer(11, 16, 768, 1536, seed=5, device=DEV)
    n = torch.zeros(11, device=DEV)
    S = torch.zeros(1536, 768, device=DEV)
    ctx.linear_sqnorm(X, D, n, grad_sum=S, method=method)
    torch.cuda.synchronize()
    n_ref, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
    assert np.array_equal(S.cpu().numpy().astype(np.float64), S_ref)
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=1e-5)      # n_i ~ 3e8 exceeds 2^24: hundreds of fp32 adds, each rounded


def test_config3_layer_direct_route_full_size(ctx):
    """B=32, T=1024, 768 -> 3072 by the direct route: 72 tiles x 2 chunks of 16 samples."""
    X, D = W.linear_layer(32, 1024, 768, 3072, seed=3, device=DEV)
    _check_layer(ctx, X, D, "direct", "config 3 direct")
    _check_layer(ctx, X, D, "pair", "config 3 pair")
    _check_layer(ctx, X, D, "auto", "config 3 auto")
    # the Gram identity over CTA pairs: 320 items of 256 x 256 tokens over 74 pairs, four or five per pair
    _check_layer(ctx, X, D, "gram_pair", "config 3 Gram over CTA pairs")


def test_embedding_at_full_size(ctx):
    """B=32, T=1024, d=768 with a 2000-row table (about 230 ids per sample occur more than once),
    then with three ids only (groups of ~340 rows, summed block-wide)."""
    B, T, d, V = 32, 1024, 768, 2000
    _, D = W.linear_layer(B, T, 8, d, seed=17, delta_std=1.0, device=DEV)
    g = torch.Generator(device=DEV)
    g.manual_seed(18)
    ids = torch.randint(0, V, (B, T), generator=g, device=DEV, dtype=torch.int32)
    n = torch.full((B,), -1.0, device=DEV)
    S = torch.full((V, d), -1.0, device=DEV)
    ctx.embedding_sqnorm(ids, D, V, n, grad_sum=S)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    n_ref, S_ref = O.embedding_terms(ids.cpu().numpy(), W.to_numpy(D), V)
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16), (n.cpu().numpy() / n_ref)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05)
    # few distinct ids: three long groups per sample
    ids2 = torch.randint(0, 3, (B, T), generator=g, device=DEV, dtype=torch.int32)
    ctx.embedding_sqnorm(ids2, D, V, n)
    torch.cuda.synchronize()
    n_ref2, _ = O.embedding_terms(ids2.cpu().numpy(), W.to_numpy(D), V)
    assert np.allclose(n.cpu().numpy(), n_ref2, rtol=TOL_BF16)


def test_embedding_gram_kernel_with_several_items_per_cta(ctx):
    """Sequences beyond 4096 tokens go through the masked Gram kernel: B=2, T=4352 gives 34 blocks
    per side, 306 + 17 work items per sample on 148 CTAs, so each CTA alternates between its two
    accumulator buffers four or five times."""
    B, T, d, V = 2, 4352, 128, 900
    _, D = W.linear_layer(B, T, 8, d, seed=19, delta_std=1.0, device=DEV)
    g = torch.Generator(device=DEV)
    g.manual_seed(20)
    ids = torch.randint(0, V, (B, T), generator=g, device=DEV, dtype=torch.int32)
    n = torch.full((B,), -1.0, device=DEV)
    ctx.embedding_sqnorm(ids, D, V, n)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    n_ref, _ = O.embedding_terms(ids.cpu().numpy(), W.to_numpy(D), V)
    assert np.allclose(n.cpu().numpy(), n_ref, rtol=TOL_BF16), (n.cpu().numpy() / n_ref)


# ---------------------------------------------------------------- groups of layers in one launch
def _group_case(ctx, shapes, B, T, method, seed, accumulate=False):
    data = [W.linear_layer(B, T, di, do, seed=seed + l, device=DEV) for l, (di, do) in enumerate(shapes)]
    sums = [torch.full((do, di), 2.0 if accumulate else -7.0, device=DEV) if (l % 5) != 3 else None
            for l, (di, do) in enumerate(shapes)]                       # some layers give no sum buffer
    n = torch.full((B,), 1.0 if accumulate else -7.0, device=DEV)
    ctx.linear_sqnorm_group([(X, D, S) for (X, D), S in zip(data, sums)], n, method=method,
                            accumulate_norms=accumulate, accumulate_sum=accumulate)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    n_ref = np.zeros(B)
    for (X, D), S in zip(data, sums):
        n_l, S_ref = O.linear_layer_terms(W.to_numpy(X), W.to_numpy(D))
        n_ref += n_l
        if S is not None:
            got = S.cpu().numpy() - (2.0 if accumulate else 0.0)
            assert np.allclose(got, S_ref, rtol=TOL_BF16, atol=TOL_BF16 * np.abs(S_ref).max() * 0.05 + (1e-5 if accumulate else 0))
    got_n = n.cpu().numpy() - (1.0 if accumulate else 0.0)
    assert np.allclose(got_n, n_ref, rtol=TOL_BF16, atol=1e-4 if accumulate else 0), (method, got_n / n_ref)


@pytest.mark.parametrize("method", ["direct", "pair", "auto"])
def test_group_of_layers_matches_the_oracle(ctx, method):
    """One launch over layers of unlike shapes: the per-sample norms add up over the layers, every
    layer's gradient sum lands in its own buffer; ragged widths, a layer narrower than one tile,
    a transformer block's four shapes (scaled down), layers without a sum buffer."""
    shapes = [(256, 768), (256, 256), (256, 1024), (1024, 256), (72, 40), (8, 8), (520, 136), (136, 520)]
    _group_case(ctx, shapes, B=6, T=200, method=method, seed=300)
    _group_case(ctx, shapes[:3], B=2, T=64, method=method, seed=400, accumulate=True)


@pytest.mark.parametrize("method", ["direct", "pair"])
def test_group_longer_than_one_launch_holds(ctx, method):
    # 53 layers: the argument block of one launch holds 48, so the call is split in two
    shapes = [(64 + 8 * (l % 5), 32 + 16 * (l % 7)) for l in range(53)]
    _group_case(ctx, shapes, B=3, T=96, method=method, seed=500)


def test_group_of_one_block_at_full_size(ctx):
    """The four linear layers of a GPT-2-small block, B=32, T=1024, as one group by the
    automatic route: about 2000 work items of four samples over the SMs."""
    shapes = list(W.GPT2_SMALL_BLOCK_LINEARS)
    _group_case(ctx, shapes, B=32, T=1024, method="auto", seed=600)


def test_group_argument_errors(ctx):
    X, D = W.linear_layer(2, 64, 64, 64, seed=1, device=DEV)
    n = torch.zeros(2, device=DEV)
    before = ctx.launch_count
    with pytest.raises(A.AdlocoError) as e:
        ctx.linear_sqnorm_group([(X, D, None)], n, method="gram")          # the group call has no Gram route
    assert e.value.status == A.ERR_INVALID_ARG
    X2, D2 = W.linear_layer(2, 64, 12, 64, seed=1, device=DEV)
    with pytest.raises(A.AdlocoError) as e:
        ctx.linear_sqnorm_group([(X, D, None), (X2, D2, None)], n)         # d_in = 12 is not a multiple of 8
    assert e.value.status == A.ERR_UNSUPPORTED and ctx.launch_count == before
