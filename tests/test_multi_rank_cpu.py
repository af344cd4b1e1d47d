"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, the step time
is the max over ranks and the value the aggregate over replicas.  (The path has
no exchange step, so this reduction of timings is the only collective.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [1.0 + rank, 5.0 - rank, 2.0]
        red = bench.reduce_max_over_ranks(mine)
        out[rank] = (red, bench.aggregate_throughput(10.0, world, red[0]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_aggregate():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(world):
        red, value = out[r]
        assert red == [2.0, 5.0, 2.0]
        assert value == 2 * 10.0 / 2.0


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert bench.aggregate_throughput(4.0, 1, 2.0) == 2.0
    ab = bench.algorithmic_bytes()
    assert ab["nt2"] == 4 * 64 * (1 << 24) and ab["os2"] == (2 * 8 + 16) * 124_439_808
    assert ab["os5"] == (2 * 4 + 16) * 1_300_000_000 and ab["acc5"] == 8 * (4 * 32 + 8) * (1 << 22)
    flops, launches = bench.model_flops()
    assert launches == 4 and flops == 4 * 12 * 2 * 32 * 1024 * (768 * 2304 + 768 * 768 + 2 * 768 * 3072)


def test_shard_bounds_partition_the_vector():
    from paper_2508_18182_b200.binding import shard_bounds
    for P in (0, 1, 7, 8, 9, 1000, 124_439_808, 1_300_000_000, 12345677):
        for world in (1, 2, 3, 4, 8, 13):
            prev = 0
            for r in range(world):
                lo, hi = shard_bounds(P, r, world)
                assert lo == prev and hi >= lo and (lo % 8 == 0 or lo == P)
                prev = hi
            assert prev == P
            sizes = [shard_bounds(P, r, world)[1] - shard_bounds(P, r, world)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 8 + 7        # balanced to within one aligned unit


# ---------------------------------------------------------------- outer step with one instance per rank
class _OracleKernels:
    """Stand-in for binding.Context on a machine without a GPU: the three elementwise steps of the
    exchanged outer step, each written with the oracle's arithmetic, so that this test exercises the
    exchange itself (slicing, padding, reduce-scatter, gather) between real processes."""

    def pseudo_gradient(self, theta, instance, out, *, stream=None):
        import oracle.adloco_oracle as O
        from paper_2508_18182_b200 import workloads as W
        d = O.widen(W.to_numpy(theta)) - O.widen(W.to_numpy(instance))
        out.copy_(torch.from_numpy(d.astype("float32")))

    def outer_apply(self, pseudo_grad_sum, K, theta, mom, *, lr, momentum, nesterov=True, stream=None):
        import oracle.adloco_oracle as O
        th = theta.numpy().astype("float64")
        virtual = th - pseudo_grad_sum.numpy().astype("float64") / K      # one instance whose difference is the mean
        th_new, v_new = O.outer_step(th, [virtual], mom.numpy(), lr=lr, momentum=momentum, nesterov=nesterov)
        theta.copy_(torch.from_numpy(th_new.astype("float32")))
        mom.copy_(torch.from_numpy(v_new.astype("float32")))

    def refresh_instance(self, theta, instance, *, stream=None):
        instance.copy_(theta.to(instance.dtype))


def _exchange_worker(rank, world, port, P, dtype_name, out):
    sys.path.insert(0, ROOT)
    from paper_2508_18182_b200 import workloads as W
    from paper_2508_18182_b200.exchange import ExchangedOuterStep, slice_length
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dtype = getattr(torch, dtype_name)
        theta, inst, mom = W.outer_state(world, P, inst_dtype=dtype, zero_momentum=False, seed=123)   # same draw on every rank
        L = slice_length(P, world)
        mom_pad = torch.zeros(L * world)
        mom_pad[:P] = mom
        state = ExchangedOuterStep(_OracleKernels(), theta.clone(), inst[rank].clone(), mom_pad[rank * L:(rank + 1) * L].clone())
        th1 = state.step(lr=0.7, momentum=0.9).clone()
        inst1 = state.instance.clone()
        th2 = state.step(lr=0.7, momentum=0.9).clone()          # second step: every instance equals theta, d = 0
        out[rank] = (th1.numpy(), th2.numpy(), state.mom.numpy().copy(), inst1.float().numpy(), state.lo, state.hi)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def _run_exchange(world, P, dtype_name):
    import numpy as np
    import oracle.adloco_oracle as O
    from paper_2508_18182_b200 import workloads as W
    from paper_2508_18182_b200.exchange import slice_length
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 31000 + (os.getpid() % 2000) + world
    procs = [ctx.Process(target=_exchange_worker, args=(r, world, port, P, dtype_name, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    dtype = getattr(torch, dtype_name)
    theta, inst, mom = W.outer_state(world, P, inst_dtype=dtype, zero_momentum=False, seed=123)
    lr, mu = float(np.float32(0.7)), float(np.float32(0.9))
    th1_ref, v1_ref = O.outer_step(W.to_numpy(theta), [W.to_numpy(t) for t in inst], W.to_numpy(mom), lr=lr, momentum=mu)
    th1_f32 = th1_ref.astype(np.float32)
    th2_ref, v2_ref = O.outer_step(th1_f32, [W.to_numpy(torch.from_numpy(th1_f32).to(dtype))] * world, v1_ref.astype(np.float32),
                                   lr=lr, momentum=mu)
    L = slice_length(P, world)
    tol_t = 4 * np.spacing(np.abs(th1_f32).max())
    for r in range(world):
        th1, th2, v_slice, inst1, lo, hi = out[r]
        assert (lo, hi) == (min(P, r * L), min(P, r * L + L))
        assert np.abs(th1 - th1_ref).max() <= tol_t, r                       # every rank holds the whole new theta
        assert np.abs(th2 - th2_ref).max() <= 2 * tol_t, r
        assert np.array_equal(inst1, torch.from_numpy(th1).to(dtype).float().numpy())   # the worker restarts from theta
        assert np.allclose(v_slice[:hi - lo], v2_ref[lo:hi], rtol=1e-5, atol=1e-9), r   # its slice of the momentum
    assert np.array_equal(out[0][0], out[world - 1][0])                      # bit-identical theta on all ranks


def test_exchanged_outer_step_two_gloo_ranks():
    _run_exchange(2, 10007, "bfloat16")


def test_exchanged_outer_step_three_ranks_tiny_vector():
    # P = 13 over 3 ranks of 8-element slices: the last rank's slice lies wholly in the padding
    _run_exchange(3, 13, "float32")
