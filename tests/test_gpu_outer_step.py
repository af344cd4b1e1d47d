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


# ---------------------------------------------------------------- outer step split around an exchange
@pytest.mark.parametrize("K,P,dtype", [(2, 100003, torch.bfloat16), (4, 65536, torch.float32), (3, 13, torch.bfloat16),
                                       (4, 1 << 20, torch.bfloat16)])
def test_exchange_form_matches_oracle(ctx, K, P, dtype):
    """One instance per rank: pseudo-gradient kernel on every rank, the K terms summed slice-wise (here
    by torch, standing in for the reduce-scatter between GPUs), update kernel on every slice, refresh.
    Result against the oracle's outer step on the whole vector.  The terms theta - theta_k cross the
    exchange as fp32 and are summed there in fp32, so beside the 2 ulp of the output rounding the result
    carries their rounding: at most (K - 1/2) ulp of sum_k |theta - theta_k| on the sum, i.e. that / K on d
    and v', times lr (1 + mu) on theta' -- visible where the K terms cancel and the update is small."""
    from paper_2508_18182_b200.exchange import slice_length
    theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=91, device=DEV, zero_momentum=False)
    th0, v0 = W.to_numpy(theta).astype(np.float64), W.to_numpy(mom).astype(np.float64)
    inst_n = [W.to_numpy(t) for t in inst]
    lr, mu = float(np.float32(0.7)), float(np.float32(0.9))
    th_ref, v_ref = O.outer_step(W.to_numpy(theta), inst_n, W.to_numpy(mom), lr=lr, momentum=mu)
    d = np.mean([th0 - O.widen(x) for x in inst_n], axis=0)
    L = slice_length(P, K)
    g = [torch.zeros(L * K, device=DEV) for _ in range(K)]
    for k in range(K):
        ctx.pseudo_gradient(theta, inst[k], g[k][:P])
        ref = (th0 - O.widen(inst_n[k])).astype(np.float32)                  # each term, rounded to fp32 once
        assert np.array_equal(g[k][:P].cpu().numpy(), ref)
        assert not g[k][P:].any()
    total = g[0].clone()
    for k in range(1, K):
        total += g[k]
    th, v = theta.clone(), mom.clone()
    for r in range(K):
        lo, hi = min(P, r * L), min(P, r * L + L)
        if hi > lo:
            ctx.outer_apply(total[lo:hi], K, th[lo:hi], v[lo:hi], lr=0.7, momentum=0.9)
    torch.cuda.synchronize()
    from parity import ulp32
    terms = np.sum([np.abs(th0 - O.widen(x)) for x in inst_n], axis=0)
    exch = (K - 0.5) / K * ulp32(terms)
    mag_t = np.maximum(np.maximum(np.abs(th0), np.abs(th_ref)), np.abs(th0 - th_ref))
    mag_v = np.maximum(np.maximum(np.abs(v_ref), np.abs(mu * v0)), np.abs(d))
    et = np.abs(th.cpu().numpy().astype(np.float64) - th_ref) / (2 * ulp32(mag_t) + lr * (1 + mu) * exch)
    ev = np.abs(v.cpu().numpy().astype(np.float64) - v_ref) / (2 * ulp32(mag_v) + exch)
    assert et.max() <= 1.0 and ev.max() <= 1.0, (K, P, float(et.max()), float(ev.max()))
    # where no term needed rounding (theta and theta_k close: most elements) the fused kernel's 2 ulp hold
    exact = np.all([(th0 - O.widen(x)).astype(np.float32).astype(np.float64) == th0 - O.widen(x) for x in inst_n], axis=0)
    exact &= (sum(g[k][:P].double() for k in range(K)).cpu().numpy() == total[:P].cpu().numpy().astype(np.float64))
    assert exact.mean() > 0.5 or K > 2
    e2 = np.abs(th.cpu().numpy().astype(np.float64) - th_ref)[exact] / ulp32(mag_t)[exact]
    assert e2.size == 0 or e2.max() <= 2.0
    for k in range(K):
        ctx.refresh_instance(th, inst[k])
        assert torch.equal(inst[k], th.to(dtype))
    with pytest.raises(A.AdlocoError) as e:
        ctx.outer_apply(total[1:9], K, th[:8], v[:8], lr=0.7, momentum=0.9)   # misaligned sum buffer
    assert e.value.status == A.ERR_ALIGNMENT


def test_exchanged_outer_step_through_a_process_group_of_one():
    """The same path through ExchangedOuterStep with a real process group on the GPU (one rank: the
    reduce-scatter and the gather move the slice to itself) -- the NCCL plumbing and the buffers."""
    import torch.distributed as dist
    from paper_2508_18182_b200.exchange import ExchangedOuterStep, slice_length
    import os
    c = A.Context(0)
    P = 30011
    theta, inst, mom = W.outer_state(1, P, inst_dtype=torch.bfloat16, seed=17, device=DEV, zero_momentum=False)
    lr, mu = float(np.float32(0.7)), float(np.float32(0.9))
    th_ref, v_ref = O.outer_step(W.to_numpy(theta), [W.to_numpy(inst[0])], W.to_numpy(mom), lr=lr, momentum=mu)
    th0, v0 = W.to_numpy(theta).astype(np.float64), W.to_numpy(mom).astype(np.float64)
    d = th0 - O.widen(W.to_numpy(inst[0]))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29700 + os.getpid() % 200))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        L = slice_length(P, 1)
        v_slice = torch.zeros(L, device=DEV)
        v_slice[:P] = mom
        state = ExchangedOuterStep(c, theta, inst[0], v_slice)
        th = state.step(lr=0.7, momentum=0.9)
        torch.cuda.synchronize()
        from parity import ulp32
        mag_t = np.maximum(np.maximum(np.abs(th0), np.abs(th_ref)), np.abs(th0 - th_ref))
        et = np.abs(th.cpu().numpy().astype(np.float64) - th_ref) / (2 * ulp32(mag_t) + lr * (1 + mu) * 0.5 * ulp32(d))
        ev = np.abs(state.mom[:P].cpu().numpy().astype(np.float64) - v_ref) / (2 * ulp32(np.maximum(np.abs(v_ref), np.abs(d))) + 0.5 * ulp32(d))
        assert et.max() <= 1.0 and ev.max() <= 1.0, (float(et.max()), float(ev.max()))
        assert torch.equal(state.instance, th.to(torch.bfloat16))
    finally:
        dist.destroy_process_group()
        c.close()
