"""GPU parity: adloco_outer_step / adloco_outer_step_host / adloco_merge against
the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle.adloco_oracle as O
from paper_2508_18182_b200 import binding as A
from paper_2508_18182_b200 import workloads as W
from parity import assert_outer_step

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = A.Context(0)
    yield c
    c.close()


def _reference(theta, inst, mom, lr, mu, nesterov):
    # the library takes lr and momentum as fp32: the oracle gets the same two numbers
    lr, mu = float(np.float32(lr)), float(np.float32(mu))
    th, v = W.to_numpy(theta), W.to_numpy(mom)
    inst_n = [W.to_numpy(t) for t in inst]
    th_ref, v_ref = O.outer_step(th, inst_n, v, lr=lr, momentum=mu, nesterov=nesterov)
    d = np.mean([th.astype(np.float64) - O.widen(x) for x in inst_n], axis=0)
    return th.astype(np.float64), v.astype(np.float64), th_ref, v_ref, d


@pytest.mark.parametrize("K,P,dtype", [(4, 1 << 20, torch.float32), (8, 1 << 20, torch.bfloat16),
                                       (1, 1003, torch.float32), (3, 8191, torch.bfloat16), (5, 7, torch.bfloat16),
                                       (9, 300007, torch.float32), (64, 10001, torch.bfloat16), (2, 1, torch.float32)])
@pytest.mark.parametrize("nesterov", [True, False])
def test_outer_step_matches_oracle_two_steps(ctx, K, P, dtype, nesterov):
    theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=K * 7 + 1, device=DEV)
    for step in range(2):                      # second step runs with non-zero momentum
        th0, v0, th_ref, v_ref, d = _reference(theta, inst, mom, 0.7, 0.9, nesterov)
        th_out, v_out = torch.empty_like(theta), torch.empty_like(mom)
        ctx.outer_step(inst, theta, mom, lr=0.7, momentum=0.9, nesterov=nesterov, theta_out=th_out, mom_out=v_out)
        assert_outer_step(th_out.cpu().numpy(), v_out.cpu().numpy(), th_ref, v_ref, th0, v0, d, 0.7, 0.9,
                          what=f"K={K} P={P} step={step}")
        # in place gives the same bits
        th_in, v_in = theta.clone(), mom.clone()
        ctx.outer_step(inst, th_in, v_in, lr=0.7, momentum=0.9, nesterov=nesterov)
        assert torch.equal(th_in, th_out) and torch.equal(v_in, v_out)
        theta, mom = th_out, v_out


def test_special_cases(ctx):
    theta, inst, mom = W.outer_state(4, 4099, seed=3, device=DEV, zero_momentum=False)
    # K = 1, lr = 1, momentum = 0 returns the instance (within 2 ulp of fp32 rounding)
    th, v = ctx.outer_step(inst[:1], theta.clone(), mom.clone(), lr=1.0, momentum=0.0)
    th0, v0, th_ref, v_ref, d = _reference(theta, inst[:1], mom, 1.0, 0.0, True)
    assert np.allclose(th_ref, inst[0].double().cpu().numpy(), rtol=0, atol=1e-17)
    assert_outer_step(th.cpu().numpy(), v.cpu().numpy(), th_ref, v_ref, th0, v0, d, 1.0, 0.0)
    # lr = 1, momentum = 0: the plain average of the instances (LocalSGD synchronisation)
    th, v = ctx.outer_step(inst, theta.clone(), mom.clone(), lr=1.0, momentum=0.0)
    mean = torch.stack([t.double() for t in inst]).mean(0).cpu().numpy()
    th0, v0, th_ref, v_ref, d = _reference(theta, inst, mom, 1.0, 0.0, True)
    assert np.allclose(th_ref, mean, rtol=0, atol=1e-16)
    assert_outer_step(th.cpu().numpy(), v.cpu().numpy(), th_ref, v_ref, th0, v0, d, 1.0, 0.0)
    # permutation of the instances stays inside the same band around the oracle
    th, v = ctx.outer_step(inst[::-1], theta.clone(), mom.clone(), lr=0.7, momentum=0.9)
    th0, v0, th_ref, v_ref, d = _reference(theta, inst, mom, 0.7, 0.9, True)
    assert_outer_step(th.cpu().numpy(), v.cpu().numpy(), th_ref, v_ref, th0, v0, d, 0.7, 0.9)
    # dyadic hand-worked example: exact
    t = torch.tensor([1.0] * 8, device=DEV)
    a, b = torch.tensor([0.5] * 8, device=DEV), torch.zeros(8, device=DEV)
    th, v = ctx.outer_step([a, b], t.clone(), torch.zeros(8, device=DEV), lr=0.5, momentum=0.5)
    assert th.tolist() == [0.4375] * 8 and v.tolist() == [0.75] * 8
    th2, v2 = ctx.outer_step([th.clone(), th.clone()], th.clone(), v.clone(), lr=0.5, momentum=0.5)
    assert th2.tolist() == [0.34375] * 8 and v2.tolist() == [0.375] * 8


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_writeback_refreshes_instances(ctx, dtype):
    theta, inst, mom = W.outer_state(3, 5003, inst_dtype=dtype, seed=9, device=DEV)
    wb = [torch.empty_like(inst[0]), None, inst[2]]          # one fresh buffer, one skipped, one in place
    keep = inst[2].clone()
    th, v = ctx.outer_step([inst[0], inst[1], keep], theta.clone(), mom.clone(), lr=0.7, momentum=0.9,
                           writeback=[wb[0], None, keep])
    plain_th, _ = ctx.outer_step(inst, theta.clone(), mom.clone(), lr=0.7, momentum=0.9)
    assert torch.equal(th, plain_th)
    assert torch.equal(wb[0], th.to(dtype)) and torch.equal(keep, th.to(dtype))


def test_argument_errors(ctx):
    theta, inst, mom = W.outer_state(2, 64, seed=1, device=DEV)
    n = ctx.launch_count
    with pytest.raises(A.AdlocoError) as e:
        ctx.outer_step(inst * 33, theta, mom, lr=0.7, momentum=0.9)          # K = 66 > 64
    assert e.value.status == A.ERR_UNSUPPORTED
    with pytest.raises(A.AdlocoError) as e:
        ctx.outer_step(inst, theta[1:], mom[1:], lr=0.7, momentum=0.9)       # misaligned
    assert e.value.status == A.ERR_ALIGNMENT
    with pytest.raises(A.AdlocoError) as e:
        ctx.outer_step(inst, theta, mom, lr=float("nan"), momentum=0.9)
    assert e.value.status == A.ERR_INVALID_ARG
    assert ctx.launch_count == n


@pytest.mark.parametrize("K,P,dtype", [(4, 3_000_017, torch.bfloat16), (2, 4099, torch.float32)])
def test_host_entry_point(ctx, K, P, dtype):
    theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=5, device="cpu", zero_momentum=False)
    th0, v0, th_ref, v_ref, d = _reference(theta, inst, mom, 0.7, 0.9, True)
    th_h, v_h = theta.clone().pin_memory(), mom.clone().pin_memory()
    ctx.outer_step_host([t.pin_memory() for t in inst], th_h, v_h, lr=0.7, momentum=0.9)
    assert_outer_step(th_h.numpy(), v_h.numpy(), th_ref, v_ref, th0, v0, d, 0.7, 0.9, what="host")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_merge_matches_oracle(ctx, dtype):
    _, inst, _ = W.outer_state(5, 10007, inst_dtype=dtype, seed=2, device=DEV)
    weights = [3, 17, 17, 1, 8]
    out = torch.empty_like(inst[0])
    rep = ctx.merge(inst, weights, out)
    x, rep_o = O.do_merge([W.to_numpy(t) for t in inst], weights)
    assert rep == rep_o == 1
    tol = 2e-6 if dtype == torch.float32 else 2 ** -8
    assert np.allclose(out.double().cpu().numpy(), x, rtol=tol, atol=1e-9)
    # merging into one of the members, exactly aliased
    ctx.merge(inst, weights, inst[1])
    assert torch.equal(inst[1], out)


@pytest.mark.parametrize("world", [2, 3, 8])
def test_sharded_outer_step_equals_the_whole(ctx, world):
    """Every rank updating its own slice (no exchange: the update is elementwise) gives
    bit for bit the result of the unsharded call.  The ranks' kernels are independent; they
    are simply run one after the other here."""
    theta, inst, mom = W.outer_state(4, 100003, inst_dtype=torch.bfloat16, seed=77, device=DEV, zero_momentum=False)
    th_ref, v_ref = ctx.outer_step(inst, theta.clone(), mom.clone(), lr=0.7, momentum=0.9)
    th, v = theta.clone(), mom.clone()
    covered = 0
    for r in range(world):
        lo, hi = A.outer_step_shard(ctx, inst, th, v, r, world, lr=0.7, momentum=0.9)
        assert lo == covered
        covered = hi
    assert covered == theta.numel()
    assert torch.equal(th, th_ref) and torch.equal(v, v_ref)
