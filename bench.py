#!/usr/bin/env python
"""Benchmark of the AdLoCo hot path on B200.

One step = one pass of the whole path over one batch of synthetic input, at the
sizes of the workload configurations:
  1. norm test on materialised per-sample gradients (B=64, P=2^24 fp32), with the
     batch decision for eta in {0.1, 0.5, 1.0} from one pass over the gradients;
  2. outer step over K=8 bf16 instances of a 124M-parameter vector (fp32 global
     parameters and momentum, lr 0.7, Nesterov momentum 0.9), in place;
  3. Gram-identity per-sample norms + mean-gradient GEMM for one linear layer
     (X bf16 [32,1024,768], Delta bf16 [32,1024,3072]), accumulated into a
     switch-mode accumulator and finalised into one test;
  4. the whole-model test in switch mode: 12 blocks x 4 linear layers x 4
     micro-batches of 32 sequences through adloco_linear_sqnorm_group (automatic
     route, one launch per micro-batch), per-sample norms accumulated over
     layers, gradient sums over micro-batches, one test at the end;
  5. outer step over K=4 bf16 instances of a 1.3B-parameter vector, in place;
  6. the norm test over 8 accumulated micro-batches of 32 x 2^22 fp32 gradients.
The headline value is the HBM throughput of the streaming sections (1, 2, 5, 6):
algorithmic bytes / device time.  The tensor-core sections (3, 4) are reported
beside it; the roofline entry is the dominant kernel of the step by time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs the same workload on its own GPU
(the path has no exchange step: weak scaling, no collective on the data path);
the time is the max over ranks and the value the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_18182_b200 import workloads as W  # noqa: E402

METRIC = "norm-test + outer-merge HBM GB/s"
UNIT = "GB/s"

# the streaming workload the metric is quoted on
NT_B, NT_P = 64, 1 << 24
OUT_K, OUT_P = 8, W.GPT2_SMALL_P
ETAS = (0.1, 0.5, 1.0)
LR, MU = 0.7, 0.9
# the tensor-core workload: one linear layer (configs[2]) ...
GR_B, GR_T, GR_DIN, GR_DOUT = 32, 1024, 768, 3072
# ... the whole model in switch mode (configs[3]): 12 blocks x 4 linear layers, 4 micro-batches of 32
C4_SHAPES = list(W.GPT2_SMALL_BLOCK_LINEARS) * 12
C4_B, C4_MICRO = 32, 4
# the large outer merge and the accumulated test (configs[4])
C5_K, C5_P = 4, W.LARGE_P
C5_B, C5_MICRO, C5_ACC_P = 32, 8, 1 << 22


def algorithmic_bytes():
    """Bytes each streaming section must move once (read + written), per step."""
    nt = 4 * NT_B * NT_P                               # every gradient element read once
    outer = (2 * OUT_K + 8) * OUT_P + 8 * OUT_P        # K bf16 instances + theta + v read; theta + v written
    outer5 = (2 * C5_K + 8) * C5_P + 8 * C5_P
    acc5 = C5_MICRO * (4 * C5_B + 8) * C5_ACC_P        # micro-batch rows read + S read-modify-written
    return {"nt2": nt, "os2": outer, "os5": outer5, "acc5": acc5}


def gram_flops():
    sym = GR_B * GR_T * (GR_T + 1) * (GR_DIN + GR_DOUT)          # symmetric half of both Gram products
    tiles = (GR_T // 128) * (GR_T // 128 + 1) // 2
    executed = 2 * GR_B * tiles * 128 * 128 * (GR_DIN + GR_DOUT)  # at 128-token tile granularity
    mean_grad = 2 * GR_B * GR_T * GR_DIN * GR_DOUT
    return sym, executed, mean_grad


def model_flops():
    """Algorithmic flops of the whole-model test by the direct route: one GEMM
    2 b T d_in d_out per (layer, micro-batch); one grouped launch per micro-batch."""
    per_mb = sum(2 * C4_B * GR_T * di * do for di, do in C4_SHAPES)
    return per_mb * C4_MICRO, C4_MICRO


def reduce_max_over_ranks(values, device="cpu"):
    """Max over ranks of each entry (the time of a multi-rank step is its slowest
    rank's); identity when no process group is initialised."""
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Whole-job throughput of `world` replicas that each process `units_per_rank`."""
    return world * units_per_rank / max_seconds


# DRAM traffic of norm_test_kernel per gradient element, from the ncu capture of the
# profiling case (B=64, P=2^21: 537.0 MB read + 7.0 MB written for 2^27 elements);
# traffic grows in proportion to B*P, so a full launch is this times its element count.
NT_TRAFFIC_BYTES_PER_ELEMENT = (537.0e6 + 7.0e6) / float(64 * (1 << 21))
# DRAM traffic of the grouped direct kernel (CTA-pair form) per transformer block of four
# layers at B=32, T=1024, from the ncu capture of the profiling case (one block: 902.3 MB
# read + 24.0 MB written for 805.3 MB of operands); every block's operands are read once,
# so a launch over n blocks moves n times this.
DG_TRAFFIC_BYTES_PER_BLOCK = 902.34e6 + 24.0e6


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------
# reference arm / CPU baseline: the fp64 oracle on the host cores
# ------------------------------------------------------------------------------------
def oracle_sample_run(steps: int, warmup: int):
    """Times the oracle, as it stands, on a bounded sample of the streaming
    workload: the norm test on B=64 x P=2^22, the outer steps on K=8 x P=2^23 and
    K=4 x P=2^23, and the accumulated test on 8 micro-batches of 32 x P=2^18.
    Returns (GB/s over the sample's algorithmic bytes, ms per step, info)."""
    import oracle.adloco_oracle as O
    try:
        from threadpoolctl import threadpool_info
        pool = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pool = 1
    sP, oP, aP = 1 << 22, 1 << 23, 1 << 18
    G = W.to_numpy(W.per_sample_grads(NT_B, sP, sigma=0.5, seed=1))
    theta, inst, mom = W.outer_state(OUT_K, oP, inst_dtype=torch.bfloat16, seed=2)
    th, v, ins = W.to_numpy(theta), W.to_numpy(mom), [W.to_numpy(t) for t in inst]
    theta5, inst5, mom5 = W.outer_state(C5_K, oP, inst_dtype=torch.bfloat16, seed=3)
    th5, v5, ins5 = W.to_numpy(theta5), W.to_numpy(mom5), [W.to_numpy(t) for t in inst5]
    mbs = [W.to_numpy(m) for m in W.micro_batches(C5_MICRO, C5_B, aP, sigma=1.0, mean_scale="raw", seed=4)]
    nbytes = (4 * NT_B * sP + (2 * OUT_K + 16) * oP + (2 * C5_K + 16) * oP + C5_MICRO * (4 * C5_B + 8) * aP)

    def one():
        r = O.norm_test(G, eta=ETAS[0], b_cur=NT_B, b_max=32)
        for eta in ETAS[1:]:
            O.decide(r.sum_sqnorm, r.mean_sqnorm, r.variance, NT_B, eta=eta, b_cur=NT_B, b_max=32)
        O.outer_step(th, ins, v, lr=LR, momentum=MU, nesterov=True)
        O.outer_step(th5, ins5, v5, lr=LR, momentum=MU, nesterov=True)
        O.accumulated_norm_test(mbs, eta=0.5, b_cur=C5_B * C5_MICRO, b_max=32)

    for _ in range(warmup):
        one()
    t0, c0 = time.perf_counter(), time.process_time()
    for _ in range(steps):
        one()
    wall = time.perf_counter() - t0
    cpu = time.process_time() - c0
    dt = wall / max(steps, 1)
    sample = (f"norm test B={NT_B} P=2^22 fp32 (1/4) + outer step K={OUT_K} bf16 P=2^23 (1/15) + outer step K={C5_K} bf16 "
              f"P=2^23 (1/155) + accumulated test {C5_MICRO} x {C5_B} x 2^18 fp32 (1/16); the tensor-core part is not sampled")
    # cores actually busy = CPU time of all threads of this process / wall time
    info = {"cores": round(max(cpu / wall, 1.0), 2), "blas_pool_threads": pool, "sample": sample,
            "cores_note": "process CPU time / wall time: the elementwise passes run on one thread, BLAS dot products on the pool"}
    return nbytes / dt / 1e9, dt * 1e3, info


def run_reference(args, rank):
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))
    warm = max(1, min(args.warmup, 2))
    gbs, ms, info = oracle_sample_run(steps, warm)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(),
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": info["cores"], "kind": "oracle", "sample": info["sample"],
                         "blas_pool_threads": info["blas_pool_threads"], "cores_note": info["cores_note"]},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config():
    if NT_P != 1 << 24:
        return {"workload": f"profiling case: norm test B={NT_B} P={NT_P}, outer step K={OUT_K} P={OUT_P}, Gram layer B={GR_B}, "
                            f"{len(C4_SHAPES)} layers x {C4_MICRO} micro-batches by the automatic route, outer step K={C5_K} P={C5_P}, "
                            f"accumulated test {C5_MICRO} x {C5_B} x {C5_ACC_P}",
                "l2": "inputs larger than L2 except the single layers", "parallelism": "replicas"}
    return {"workload": "configs[4] large outer merge + accumulated test: outer step K=4 bf16 P=1,300,000,000 (fp32 theta and "
                        "momentum, lr 0.7, Nesterov 0.9, in place) and the norm test over 8 accumulated micro-batches of "
                        "32 x 4,194,304 fp32; configs[3] whole-model switch mode: 12 blocks x 4 linear layers "
                        "(768->2304, 768->768, 768->3072, 3072->768; T=1024 bf16) x 4 micro-batches of 32 through "
                        "adloco_linear_sqnorm_group(auto), accumulated and tested once; configs[1] streaming scale-up: norm test "
                        "B=64 P=16,777,216 fp32 (eta 0.1/0.5/1.0) + outer step K=8 bf16 P=124,439,808; configs[2] Gram layer "
                        "B=32 T=1024 768->3072 bf16 (Gram identity + mean-gradient GEMM). value = bytes of the four streaming "
                        "sections / their device time; the tensor-core sections are reported in roofline and kernels",
            "l2": "inputs larger than L2 (72 GB resident; every section streams more than 126 MB except the single layers, "
                  "whose operands are evicted by the 30 GB that pass between two visits), no flush needed",
            "parallelism": "replicas (no exchange step on the path)"}


# ------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------
SECTIONS = ("nt2", "os2", "gram3", "model4", "fin4", "os5", "acc5")


def run_ours(args, rank, world, local_rank):
    from paper_2508_18182_b200 import binding as A
    from paper_2508_18182_b200.build import build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ctx = A.Context(local_rank)

    # ---- resident inputs (about 72 GB at full size)
    G = W.per_sample_grads(NT_B, NT_P, sigma=0.5, seed=10 + rank, device=dev)
    theta, inst, mom = W.outer_state(OUT_K, OUT_P, inst_dtype=torch.bfloat16, seed=20 + rank, device=dev)
    X, D = W.linear_layer(GR_B, GR_T, GR_DIN, GR_DOUT, seed=30 + rank, device=dev)
    S_layer = torch.zeros(GR_DOUT, GR_DIN, device=dev)
    n_layer = torch.zeros(GR_B, device=dev)
    acc = A.Accumulator(ctx, [S_layer])
    params = [A.make_params(eta, b_cur=NT_B, b_max=32) for eta in ETAS]
    gparams = A.make_params(0.5, b_cur=GR_B, b_max=32)
    # whole model: every (micro-batch, layer) pair of operands is resident
    data4 = [[W.linear_layer(C4_B, GR_T, di, do, seed=1000 * j + l + 7 * rank, device=dev)
              for l, (di, do) in enumerate(C4_SHAPES)] for j in range(C4_MICRO)]
    sums4 = [torch.zeros(do, di, device=dev) for di, do in C4_SHAPES]
    groups4 = [ctx.make_layer_group([(Xl, Dl, S) for (Xl, Dl), S in zip(data4[j], sums4)]) for j in range(C4_MICRO)]
    acc4 = A.Accumulator(ctx, sums4)
    n_mb = torch.zeros(C4_B, device=dev)
    p4 = A.make_params(0.5, b_cur=C4_B * C4_MICRO, b_max=32)
    # large outer merge, accumulated test
    theta5, inst5, mom5 = W.outer_state(C5_K, C5_P, inst_dtype=torch.bfloat16, seed=50 + rank, device=dev)
    mbs5 = W.micro_batches(C5_MICRO, C5_B, C5_ACC_P, sigma=1.0, mean_scale="raw", seed=60 + rank, device=dev)
    S5 = torch.zeros(C5_ACC_P, device=dev)
    acc5 = A.Accumulator(ctx, [S5])
    p5 = A.make_params(0.5, b_cur=C5_B * C5_MICRO, b_max=32)
    stream = torch.cuda.current_stream()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(m=None):
        def mark(name):
            if m is not None:
                e = ev()
                e.record(stream)
                m.append((name, e))
        mark("begin")
        # configs[1]: norm test with the eta sweep, outer step
        ctx.norm_test(G, params[0], sync=False)
        for p in params[1:]:
            ctx.test_decide(p, sync=False)
        mark("nt2")
        ctx.outer_step(inst, theta, mom, lr=LR, momentum=MU, nesterov=True)
        mark("os2")
        # configs[2]: one layer by the Gram identity + mean-gradient GEMM, accumulated and tested
        acc.reset()
        ctx.gram_sqnorm(X, D, n_layer, grad_sum=S_layer, accumulate_sum=True)
        acc.accumulate(per_sample_sqnorm=n_layer)
        acc.finalize(gparams, sync=False)
        mark("gram3")
        # configs[3]: whole model, 4 micro-batches x 48 layers (one grouped launch per micro-batch), one test
        acc4.reset()
        mark("fin4")
        for j in range(C4_MICRO):
            ctx.linear_sqnorm_group(groups4[j], n_mb, method="auto", accumulate_sum=True)
            mark("model4")
            acc4.accumulate(per_sample_sqnorm=n_mb)
            if j == C4_MICRO - 1:
                acc4.finalize(p4, sync=False)
            mark("fin4")
        # configs[4]: large outer merge, accumulated norm test
        ctx.outer_step(inst5, theta5, mom5, lr=LR, momentum=MU, nesterov=True)
        mark("os5")
        acc5.reset()
        for mb in mbs5:
            acc5.accumulate(mb)
        acc5.finalize(p5, sync=False)
        mark("acc5")

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    marks = [[] for _ in range(args.steps)]
    launches0 = ctx.launch_count
    torch.cuda.synchronize()
    t_begin, t_end = ev(), ev()
    t_begin.record(stream)
    for s in range(args.steps):
        step(marks[s])
    t_end.record(stream)
    torch.cuda.synchronize()
    if use_dist:
        import torch.distributed as dist
        dist.barrier()
    clocks = sampler.stop()
    launches = ctx.launch_count - launches0
    res5 = ctx._read_result()

    total_ms = t_begin.elapsed_time(t_end)
    sec_ms = {k: 0.0 for k in SECTIONS}
    for m in marks:
        for (_, e0), (name, e1) in zip(m[:-1], m[1:]):
            sec_ms[name] += e0.elapsed_time(e1) / args.steps
    vals = reduce_max_over_ranks([total_ms] + [sec_ms[k] for k in SECTIONS], device=dev)
    total_ms = vals[0]
    sec_ms = dict(zip(SECTIONS, vals[1:]))
    timed_s = total_ms * 1e-3

    # the tensor-core kernels of one layer one by one (outside the timed steps): the call without a
    # sum buffer runs the Gram kernel alone, the difference to the full call is the GEMM
    reps = 20
    g0, g1, g2, g3, g4, g5, g6 = ev(), ev(), ev(), ev(), ev(), ev(), ev()
    torch.cuda.synchronize()
    time.sleep(1.0)           # let the clocks recover from the timed region: these are burst figures
    g0.record(stream)
    for _ in range(reps):
        ctx.gram_sqnorm(X, D, n_layer)
    g1.record(stream)
    for _ in range(reps):
        ctx.gram_sqnorm(X, D, n_layer, grad_sum=S_layer, accumulate_sum=True)
    g2.record(stream)
    torch.cuda.synchronize()
    g3.record(stream)
    for _ in range(reps):
        ctx.linear_sqnorm(X, D, n_layer, grad_sum=S_layer, accumulate_sum=True, method="direct")
    g4.record(stream)
    for _ in range(reps):
        ctx.linear_sqnorm(X, D, n_layer, grad_sum=S_layer, accumulate_sum=True, method="pair")
    g5.record(stream)
    for _ in range(reps):
        ctx.linear_sqnorm(X, D, n_layer, method="gram_pair")
    g6.record(stream)
    torch.cuda.synchronize()
    gram_only_ms = g0.elapsed_time(g1) / reps
    gram_pair_ms = g5.elapsed_time(g6) / reps
    # the streaming kernels by themselves, after a pause that lets the clocks recover from the power cap
    # the tensor-core sections of the step run into (the cap holds the SM clock, and with it the on-chip
    # network, well below its maximum for the whole step)
    time.sleep(1.0)
    alone = {}

    def time_alone(name, fn, n=20):
        fn()
        torch.cuda.synchronize()
        a0, a1 = ev(), ev()
        a0.record(stream)
        for _ in range(n):
            fn()
        a1.record(stream)
        torch.cuda.synchronize()
        alone[name] = a0.elapsed_time(a1) / n

    def acc5_only():
        for mb in mbs5:
            acc5.accumulate(mb)

    time_alone("nt2", lambda: ctx.norm_test(G, params[0], sync=False))
    time_alone("os2", lambda: ctx.outer_step(inst, theta, mom, lr=LR, momentum=MU, nesterov=True))
    time_alone("os5", lambda: ctx.outer_step(inst5, theta5, mom5, lr=LR, momentum=MU, nesterov=True), n=10)
    time_alone("acc5", acc5_only)
    # what a plain copy reaches under the step's own conditions: torch's copy of 1 GiB timed between bursts
    # of the whole-model kernel, in a loop as long as a quarter of the timed region's steps (the power cap
    # holds the clocks there as it does in the step; the copy is the measured-peak recipe, not library code)
    ca = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    cb = torch.empty_like(ca)
    cmarks = []
    for _ in range(max(12, args.steps // 4)):
        for j in range(C4_MICRO):
            ctx.linear_sqnorm_group(groups4[j], n_mb, method="auto", accumulate_sum=True)
        c0, c1 = ev(), ev()
        c0.record(stream)
        for _ in range(4):
            cb.copy_(ca)
        c1.record(stream)
        cmarks.append((c0, c1))
    torch.cuda.synchronize()
    cts = sorted(x.elapsed_time(y) / 4 for x, y in cmarks[len(cmarks) // 3:])
    copy_in_loop_gbs = 2 * ca.numel() / (cts[len(cts) // 2] * 1e-3) / 1e9
    del ca, cb
    mean_grad_ms = max(g1.elapsed_time(g2) / reps - gram_only_ms, 1e-6)
    direct_ms = g3.elapsed_time(g4) / reps
    pair_ms = g4.elapsed_time(g5) / reps

    ab = algorithmic_bytes()
    peaks = load_peaks()
    stream_bytes = sum(ab.values())
    stream_ms = sec_ms["nt2"] + sec_ms["os2"] + sec_ms["os5"] + sec_ms["acc5"]
    value = aggregate_throughput(stream_bytes, world, stream_ms * 1e-3) / 1e9
    sym, executed, mg = gram_flops()
    m256 = (GR_T + 255) // 256
    executed_pair = 2 * GR_B * (m256 * (m256 + 1) // 2) * 256 * 256 * (GR_DIN + GR_DOUT)
    mflops, mlaunches = model_flops()

    # ---- end to end through the host-memory entry points (rank-local pinned buffers): the
    # configs[1] pair, whose host copies (8.3 GB) fit any host; the other sections have no host form
    e2e = None
    if not args.no_e2e:
        Gh = torch.empty((NT_B, NT_P), dtype=torch.float32).pin_memory()
        Gh.copy_(G)
        th_h = theta.cpu().pin_memory()
        v_h = mom.cpu().pin_memory()
        inst_h = [t.cpu().pin_memory() for t in inst]
        ereps = max(1, min(args.steps, 3))
        ctx.norm_test_host(Gh, params[0])                   # warm-up: allocates the staging buffers
        ctx.outer_step_host(inst_h, th_h, v_h, lr=LR, momentum=MU)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(ereps):
            ctx.norm_test_host(Gh, params[0])               # the eta sweep needs no further data movement
            ctx.outer_step_host(inst_h, th_h, v_h, lr=LR, momentum=MU)
        torch.cuda.synchronize()
        e2e_s = reduce_max_over_ranks([(time.perf_counter() - t0) / ereps], device=dev)[0]
        e2e = {"value": aggregate_throughput(ab["nt2"] + ab["os2"], world, e2e_s) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": ab["nt2"] + (2 * OUT_K + 8) * OUT_P,
               "d2h_bytes_per_step": 8 * OUT_P + 80, "ms_per_step": e2e_s * 1e3, "steps": ereps,
               "workload": "configs[1] pair through adloco_norm_test_host + adloco_outer_step_host (pinned host buffers)"}
        del Gh, th_h, v_h, inst_h

    if rank != 0:
        return

    # the tensor peak that fits the timed region: the sustained figure when the region lasts a second or
    # more, or when the sampled clocks show the power cap holding the SM clock below 95 % of its maximum
    # (the step's tensor-core sections reach the cap within tens of milliseconds); else the burst figure
    burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    capped = ("sw_power_cap" in clocks.get("reasons", []) and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
              and clocks["sm_mhz"] < 0.95 * clocks["sm_max_mhz"])
    regime = "sustained" if (timed_s >= 1.0 or capped) else "burst"
    tpeak = burst if regime == "burst" else sustained

    def tensor_entry(flops, ms, peak, **extra):
        tf = flops / (ms * 1e-3) / 1e12
        d = {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
             "frac_of_burst": tf / burst, "frac_of_sustained": tf / sustained, "algorithmic_flops": flops}
        d.update(extra)
        return d

    def hbm_entry(nbytes, ms, in_step=True, **extra):
        gbs = nbytes / (ms * 1e-3) / 1e9
        d = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
             "frac_of_nominal_8TBs": gbs / 8000.0, "algorithmic_bytes": nbytes}
        if in_step:     # the copy timed between bursts of tensor-core work is the reference for in-step figures only
            d["frac_of_copy_between_tensor_bursts"] = gbs / copy_in_loop_gbs
        d.update(extra)
        return d

    model_ms = sec_ms["model4"]
    kernel_is_pair = True     # the automatic route takes the CTA-pair kernel on every device that launches clusters
    kernels = {
        "norm_test_kernel": hbm_entry(ab["nt2"], sec_ms["nt2"], ms_per_launch=sec_ms["nt2"], section="configs[1] norm test + eta sweep",
                                      traffic=NT_TRAFFIC_BYTES_PER_ELEMENT * NT_B * NT_P),
        "outer_step_kernel": hbm_entry(ab["os2"], sec_ms["os2"], ms_per_launch=sec_ms["os2"], section="configs[1] outer step K=8"),
        "outer_step_kernel_large": hbm_entry(ab["os5"], sec_ms["os5"], ms_per_launch=sec_ms["os5"], section="configs[4] outer step K=4, P=1.3e9"),
        "norm_test_kernel_micro": hbm_entry(ab["acc5"], sec_ms["acc5"], ms_per_launch=sec_ms["acc5"] / C5_MICRO,
                                            section="configs[4] accumulate x8 + finalize (incl. the reset of S)"),
        "streaming_kernels_alone": {
            "note": "the same four kernels timed by themselves after a 1 s pause (20 launches each, clocks unconstrained)",
            "norm_test_kernel": hbm_entry(ab["nt2"], alone["nt2"], in_step=False),
            "outer_step_kernel": hbm_entry(ab["os2"], alone["os2"], in_step=False),
            "outer_step_kernel_large": hbm_entry(ab["os5"], alone["os5"], in_step=False),
            "norm_test_kernel_micro": hbm_entry(ab["acc5"], alone["acc5"], in_step=False, includes="the 8 accumulate launches, no reset / finalize"),
        },
        "gram_path": tensor_entry(sym + mg, sec_ms["gram3"], tpeak, ms_per_step=sec_ms["gram3"],
                                  executed_tflops=(executed + mg) / (sec_ms["gram3"] * 1e-3) / 1e12, peak_regime=regime,
                                  includes="configs[2]: reset + gram + mean-grad + accumulate + finalize, inside the step"),
        "whole_model_finalize": {"ms_per_step": sec_ms["fin4"], "includes": "reset of 48 sum buffers (340 MB), 4 accumulate "
                                 "calls, squared norm of the sums (340 MB) and the batch rule"},
        "gram_sqnorm_kernel": tensor_entry(sym, gram_only_ms, burst, ms_per_launch=gram_only_ms,
                                           executed_tflops=executed / (gram_only_ms * 1e-3) / 1e12,
                                           timed="alone, 20 launches back to back (a burst), incl. the memset of n"),
        "gram_pair_kernel": tensor_entry(sym, gram_pair_ms, burst, ms_per_launch=gram_pair_ms,
                                         executed_tflops=executed_pair / (gram_pair_ms * 1e-3) / 1e12,
                                         timed="alone, 20 launches back to back: the Gram identity over CTA pairs "
                                               "(256-token blocks; the sub-block below the diagonal of a diagonal "
                                               "block is computed and dropped)"),
        "mean_grad_kernel": tensor_entry(mg, mean_grad_ms, burst, ms_per_launch=mean_grad_ms,
                                         timed="alone: full call minus the Gram-only call"),
        "direct_sqnorm_kernel_one_layer": tensor_entry(mg, direct_ms, burst, ms_per_launch=direct_ms,
                                                       timed="alone, 20 launches back to back: adloco_linear_sqnorm(direct) on "
                                                             "the configs[2] layer, same n_i and S as gram + mean-grad"),
        "direct_pair_kernel_one_layer": tensor_entry(mg, pair_ms, burst, ms_per_launch=pair_ms,
                                                     timed="alone, 20 launches back to back: adloco_linear_sqnorm(pair) on the "
                                                           "configs[2] layer (256 x 256 tiles over CTA pairs)"),
    }
    # the dominant kernel of the step by time: the direct per-sample-gradient GEMM of the whole model
    roofline = tensor_entry(mflops / mlaunches, model_ms / mlaunches, tpeak, kernel="direct_group_kernel",
                            ms_per_launch=model_ms / mlaunches, launches_per_step=mlaunches, peak_regime=regime,
                            peak_source=peaks["source"],
                            traffic=(DG_TRAFFIC_BYTES_PER_BLOCK * len(C4_SHAPES) / 4 if kernel_is_pair else None),
                            operand_bytes=sum(2 * C4_B * GR_T * (di + do) for di, do in C4_SHAPES),
                            section="configs[3]: one launch per micro-batch over its 48 layers (adloco_linear_sqnorm_group, "
                                    "automatic route); flops per launch = sum over the layers of 2 b T d_in d_out")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (streaming sections, fp64 combines); bf16 x bf16 -> f32 (tensor-core sections)",
        "data": "synthetic",
        "config": workload_config(),
        "clocks": clocks,
        "gpu_launches": launches,
        "timed_region_s": timed_s,
        "stream_ms_per_step": stream_ms,
        "hbm_copy_between_tensor_bursts_gbs": copy_in_loop_gbs,
        "tensor_ms_per_step": sec_ms["gram3"] + sec_ms["model4"] + sec_ms["fin4"],
        "section_ms": sec_ms,
        "ms_x_sm_mhz": (total_ms / args.steps) * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
        "roofline": roofline,
        "kernels": kernels,
        "last_result": {"stat": res5.stat, "b_req": res5.b_req, "flags": res5.flags},
    }
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        gbs, ms, info = oracle_sample_run(2, 1)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": info["cores"], "kind": "oracle", "sample": info["sample"],
                                "blas_pool_threads": info["blas_pool_threads"], "cores_note": info["cores_note"]}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------
# per-configuration table (python bench.py --table): one JSON line per row
# ------------------------------------------------------------------------------------
def run_table(args):
    """Times every kernel of the five workload configurations on one GPU, with the
    oracle beside it (whole where it finishes in seconds, else on a stated sample and
    extrapolated).  Configurations whose inputs fit in L2 are timed with an L2 flush
    (a 512 MB write) between repetitions."""
    import numpy as np
    import oracle.adloco_oracle as O
    from paper_2508_18182_b200 import binding as A
    from paper_2508_18182_b200.build import build

    build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = A.Context(0)
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def gpu_ms(fn, reps=20, flush=False, warm=3):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            if flush:
                flush_buf.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ts.sort()
        return ts[len(ts) // 2]

    def gpu_ms_rotating(fns, rounds=10):
        """Throughput of a small kernel: the calls in `fns` (the same kernel on different buffers, together
        larger than L2) run back to back for `rounds` rounds with no synchronisation in between."""
        for fn in fns:
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(rounds):
            for fn in fns:
                fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (rounds * len(fns))

    def cpu_s(fn):
        t0 = time.perf_counter()
        fn()
        return time.perf_counter() - t0

    def emit(config, kernel, ms, *, nbytes=None, flops=None, oracle_s=None, oracle_note="", note=""):
        row = {"config": config, "kernel": kernel, "gpu_ms": round(ms, 4)}
        if nbytes is not None:
            gbs = nbytes / (ms * 1e-3) / 1e9
            row.update({"algorithmic_bytes": nbytes, "GB/s": round(gbs, 1),
                        "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 3), "frac_nominal_8TBs": round(gbs / 8000, 3)})
        if flops is not None:
            tf = flops / (ms * 1e-3) / 1e12
            row.update({"algorithmic_flops": flops, "TFLOP/s": round(tf, 1),
                        "frac_measured_bf16": round(tf / peaks["bf16_tflops"], 3), "frac_nominal_2250": round(tf / 2250, 3)})
        if oracle_s is not None:
            row.update({"oracle_s": round(oracle_s, 3), "oracle_note": oracle_note,
                        "speedup": round(oracle_s / (ms * 1e-3), 1)})
        if note:
            row["note"] = note
        print(json.dumps(row), flush=True)

    def outer_case(config, K, P, dtype):
        theta, inst, mom = W.outer_state(K, P, inst_dtype=dtype, seed=7, device=dev)
        es = 2 if dtype == torch.bfloat16 else 4
        ms = gpu_ms(lambda: ctx.outer_step(inst, theta, mom, lr=LR, momentum=MU), flush=(P * (es * K + 16) < (1 << 29)))
        sl = min(P, 1 << 24)
        th, v, ins = W.to_numpy(theta[:sl]), W.to_numpy(mom[:sl]), [W.to_numpy(t[:sl]) for t in inst]
        o_s = cpu_s(lambda: O.outer_step(th, ins, v, lr=LR, momentum=MU)) * (P / sl)
        emit(config, f"outer_step (K={K} {'bf16' if es == 2 else 'fp32'}, P={P})", ms, nbytes=(es * K + 16) * P,
             oracle_s=o_s, oracle_note="whole" if sl == P else f"timed on {sl} elements, extrapolated")
        del theta, inst, mom

    # config 1
    G = W.per_sample_grads(16, 1 << 20, seed=1, device=dev)
    p = A.make_params(0.5, b_cur=16, b_max=32)
    ms = gpu_ms(lambda: ctx.norm_test(G, p, sync=False), flush=True)
    Gn = W.to_numpy(G)
    emit(1, "norm_test (B=16, P=2^20)", ms, nbytes=4 * 16 * (1 << 20), oracle_s=cpu_s(lambda: O.norm_test(Gn, eta=0.5)),
         oracle_note="whole", note="L2 flushed between repetitions; launch-latency bound")
    outer_case(1, 4, 1 << 20, torch.float32)
    # the same two kernels back to back over four rotating input sets (256 MB / 134 MB in all, more than L2):
    # throughput without the launch latency a lone call pays
    Gs = [W.per_sample_grads(16, 1 << 20, seed=100 + r, device=dev) for r in range(4)]
    ms = gpu_ms_rotating([(lambda g=g: ctx.norm_test(g, p, sync=False)) for g in Gs])
    emit(1, "norm_test (B=16, P=2^20), back to back over 4 rotating inputs", ms, nbytes=4 * 16 * (1 << 20),
         note="throughput; the row above is the latency of one call")
    states = [W.outer_state(4, 1 << 20, inst_dtype=torch.float32, seed=200 + r, device=dev) for r in range(4)]
    ms = gpu_ms_rotating([(lambda st=st: ctx.outer_step(st[1], st[0], st[2], lr=LR, momentum=MU)) for st in states])
    emit(1, "outer_step (K=4 fp32, P=1048576), back to back over 4 rotating states", ms, nbytes=(4 * 4 + 16) * (1 << 20),
         note="throughput; the row above is the latency of one call")
    del G, Gs, states
    # config 2
    G = W.per_sample_grads(NT_B, 1 << 24, seed=2, device=dev)
    p = A.make_params(0.1, b_cur=64, b_max=32)

    def c2():
        ctx.norm_test(G, p, sync=False)
        ctx.test_decide(A.make_params(0.5, b_cur=64, b_max=32), sync=False)
        ctx.test_decide(A.make_params(1.0, b_cur=64, b_max=32), sync=False)
    ms = gpu_ms(c2)
    Gn = W.to_numpy(G)
    emit(2, "norm_test + eta sweep (B=64, P=2^24)", ms, nbytes=4 * 64 * (1 << 24),
         oracle_s=cpu_s(lambda: O.norm_test(Gn, eta=0.1)), oracle_note="whole")
    Ssum = torch.empty(1 << 24, device=dev)
    ctx.norm_test(G, p, grad_sum=Ssum, sync=False)
    ms = gpu_ms(lambda: ctx.inner_product_test(G, Ssum, theta=0.01, nu=0.3, b_cur=64), reps=10)
    Gs = Gn[:, : 1 << 21]
    o_s = cpu_s(lambda: O.inner_product_tests(Gs, theta=0.01, nu=0.3)) * 8
    emit(2, "inner_product_test (second pass, B=64, P=2^24)", ms, nbytes=4 * 64 * (1 << 24) + 4 * (1 << 24),
         oracle_s=o_s, oracle_note="timed on P=2^21, extrapolated", note="includes the host synchronisation of the call")
    del G, Gn, Gs, Ssum
    outer_case(2, 8, W.GPT2_SMALL_P, torch.bfloat16)
    # config 3
    X, D = W.linear_layer(GR_B, GR_T, GR_DIN, GR_DOUT, seed=3, device=dev)
    n = torch.zeros(GR_B, device=dev)
    S = torch.zeros(GR_DOUT, GR_DIN, device=dev)
    sym, executed, mg = gram_flops()
    ms_g = gpu_ms(lambda: ctx.gram_sqnorm(X, D, n))
    ms_gs = gpu_ms(lambda: ctx.gram_sqnorm(X, D, n, grad_sum=S))
    ms_d = gpu_ms(lambda: ctx.linear_sqnorm(X, D, n, grad_sum=S, method="direct"))
    ms_p = gpu_ms(lambda: ctx.linear_sqnorm(X, D, n, grad_sum=S, method="pair"))
    Xn, Dn = W.to_numpy(X), W.to_numpy(D)
    o_s = cpu_s(lambda: O.linear_layer_terms(Xn, Dn))
    emit(3, "gram_sqnorm (norms only)", ms_g, flops=sym, note=f"executed {executed / (ms_g * 1e-3) / 1e12:.0f} TFLOP/s")
    emit(3, "gram_sqnorm + mean-gradient GEMM", ms_gs, flops=sym + mg, oracle_s=o_s, oracle_note="whole (BLAS dgemm per sample)")
    emit(3, "mean-gradient GEMM (difference)", ms_gs - ms_g, flops=mg)
    emit(3, "linear_sqnorm direct (norms + gradient sum)", ms_d, flops=mg, oracle_s=o_s, oracle_note="whole",
         note="same outputs as the row above from one GEMM")
    emit(3, "linear_sqnorm pair (CTA-pair direct kernel)", ms_p, flops=mg, oracle_s=o_s, oracle_note="whole")
    ms_gp = gpu_ms(lambda: ctx.linear_sqnorm(X, D, n, method="gram_pair"))
    emit(3, "gram_pair (Gram identity over CTA pairs, norms only)", ms_gp, flops=sym,
         note="40 of 128x128 sub-blocks computed per sample for 36 needed")
    Sb = torch.zeros(GR_DOUT, device=dev)
    ms_b = gpu_ms(lambda: ctx.vector_param_sqnorm(D, n, grad_sum=Sb), flush=True)
    Dn8 = Dn[:8]
    emit(3, "vector_param_sqnorm (bias of the layer, Delta [32,1024,3072])", ms_b, nbytes=2 * GR_B * GR_T * GR_DOUT,
         oracle_s=cpu_s(lambda: O.vector_param_terms(Dn8)) * 4, oracle_note="8 samples timed, x4", note="L2 flushed")
    # throughput of the same kernel back to back (no L2 flush needed: the 201 MB operand exceeds L2, and
    # two operands alternate)
    D2 = D.clone()
    ms_b2 = gpu_ms_rotating([lambda: ctx.vector_param_sqnorm(D, n, grad_sum=Sb), lambda: ctx.vector_param_sqnorm(D2, n, grad_sum=Sb)])
    emit(3, "vector_param_sqnorm, back to back over 2 alternating operands", ms_b2, nbytes=2 * GR_B * GR_T * GR_DOUT,
         note="throughput; the row above is the latency of one call after an L2 flush")
    del D2
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    ids = torch.randint(0, 50257, (GR_B, GR_T), generator=gen, device=dev, dtype=torch.int32)
    De = X                                               # [32, 1024, 768] bf16 stands in for the output gradient
    Se = torch.zeros(50257, GR_DIN, device=dev)
    ms_e = gpu_ms(lambda: ctx.embedding_sqnorm(ids, De, 50257, n))
    ms_es = gpu_ms(lambda: ctx.embedding_sqnorm(ids, De, 50257, n, grad_sum=Se, accumulate_sum=True))
    emit(3, "embedding_sqnorm (norms only; ids [32,1024], V=50257, d=768)", ms_e, nbytes=GR_B * GR_T * (2 * GR_DIN + 4),
         note="grouping kernel: every delta row read once (the masked Gram form of the same norms took 0.043 ms)")
    emit(3, "embedding scatter-add of the gradient sum (difference)", ms_es - ms_e,
         nbytes=GR_B * GR_T * GR_DIN * (2 + 4), note="2 bytes read + 4 bytes added per element")
    del Se
    # config 4: 12 blocks x 4 layers x 4 micro-batches, all inputs resident (38.7 GB)
    shapes = list(W.GPT2_SMALL_BLOCK_LINEARS) * 12
    data = [[W.linear_layer(32, 1024, di, do, seed=1000 * j + l, device=dev) for l, (di, do) in enumerate(shapes)]
            for j in range(4)]
    sums = [torch.zeros(do, di, device=dev) for di, do in shapes]
    acc = A.Accumulator(ctx, sums)
    n_mb = torch.zeros(32, device=dev)
    p4 = A.make_params(0.5, b_cur=128, b_max=32)

    def whole_model(method):
        acc.reset()
        for j in range(4):
            for l, (Xl, Dl) in enumerate(data[j]):
                if method == "gram":
                    ctx.gram_sqnorm(Xl, Dl, n_mb, accumulate_norms=(l > 0), grad_sum=sums[l], accumulate_sum=True)
                else:
                    ctx.linear_sqnorm(Xl, Dl, n_mb, accumulate_norms=(l > 0), grad_sum=sums[l], accumulate_sum=True,
                                      method=method)
            acc.accumulate(per_sample_sqnorm=n_mb)
        acc.finalize(p4, sync=False)
    f_sym = sum(32 * 1024 * 1025 * (di + do) for di, do in shapes) * 4
    f_mg = sum(2 * 32 * 1024 * di * do for di, do in shapes) * 4
    ms4 = gpu_ms(lambda: whole_model("gram"), reps=5, warm=1)
    Xb = [(W.to_numpy(data[0][l][0]), W.to_numpy(data[0][l][1])) for l in range(4)]
    o4 = cpu_s(lambda: [O.linear_layer_terms(x, d) for x, d in Xb]) * 48
    emit(4, "whole model, Gram route (48 layers x 4 micro-batches + finalize)", ms4, flops=f_sym + f_mg, oracle_s=o4,
         oracle_note="one block x one micro-batch timed, x48 extrapolated")
    ms4d = gpu_ms(lambda: whole_model("direct"), reps=5, warm=1)
    emit(4, "whole model, one-CTA direct kernel, one launch per layer", ms4d, flops=f_mg, oracle_s=o4, oracle_note="as above")
    ms4p = gpu_ms(lambda: whole_model("auto"), reps=5, warm=1)
    emit(4, "whole model, linear_sqnorm auto (CTA-pair direct kernel), one launch per layer", ms4p, flops=f_mg, oracle_s=o4,
         oracle_note="as above")
    groups = [ctx.make_layer_group([(Xl, Dl, S) for (Xl, Dl), S in zip(data[j], sums)]) for j in range(4)]

    def whole_model_grouped(method):
        acc.reset()
        for j in range(4):
            ctx.linear_sqnorm_group(groups[j], n_mb, method=method, accumulate_sum=True)
            acc.accumulate(per_sample_sqnorm=n_mb)
        acc.finalize(p4, sync=False)
    ms4g1 = gpu_ms(lambda: whole_model_grouped("direct"), reps=5, warm=1)
    emit(4, "whole model, linear_sqnorm_group (one-CTA kernel), one launch per micro-batch", ms4g1, flops=f_mg, oracle_s=o4,
         oracle_note="as above")
    ms4g2 = gpu_ms(lambda: whole_model_grouped("auto"), reps=5, warm=1)
    emit(4, "whole model, linear_sqnorm_group auto (CTA-pair kernel), one launch per micro-batch", ms4g2, flops=f_mg,
         oracle_s=o4, oracle_note="as above")
    acc.close()
    del data, sums
    torch.cuda.empty_cache()
    # config 5
    outer_case(5, 4, W.LARGE_P, torch.bfloat16)
    mbs = W.micro_batches(8, 32, 1 << 22, sigma=1.0, mean_scale="raw", seed=5, device=dev)
    Sacc = torch.zeros(1 << 22, device=dev)
    acc = A.Accumulator(ctx, [Sacc])
    p5 = A.make_params(0.5, b_cur=256, b_max=32)

    def c5():
        acc.reset()
        for m in mbs:
            acc.accumulate(m)
        acc.finalize(p5, sync=False)
    ms = gpu_ms(c5, reps=10)
    mbn = [W.to_numpy(m) for m in mbs]
    emit(5, "accumulate x8 + finalize (B=256, P=2^22)", ms, nbytes=8 * (4 * 32 + 8) * (1 << 22),
         oracle_s=cpu_s(lambda: O.accumulated_norm_test(mbn, eta=0.5)), oracle_note="whole")
    acc.close()
    # trainer merge
    _, inst, _ = W.outer_state(4, W.GPT2_SMALL_P, inst_dtype=torch.bfloat16, seed=9, device=dev)
    out = torch.empty_like(inst[0])
    ms = gpu_ms(lambda: ctx.merge(inst, [3, 17, 5, 8], out))
    emit("merge", "adloco_merge (K=4 bf16, P=124,439,808)", ms, nbytes=(2 * 4 + 2) * W.GPT2_SMALL_P)
    # the three kernels of the outer step with one instance per GPU (the exchange between them needs several GPUs
    # and is not timed here): one rank's share at the GPT-2-small size, its slice of a world of 8 for the update
    P = W.GPT2_SMALL_P
    theta, inst, mom = W.outer_state(1, P, inst_dtype=torch.bfloat16, seed=11, device=dev)
    g = torch.empty(P, device=dev)
    ms = gpu_ms(lambda: ctx.pseudo_gradient(theta, inst[0], g))
    emit("exchange form", "adloco_pseudo_gradient (bf16 instance, P=124,439,808)", ms, nbytes=(4 + 2 + 4) * P)
    L = P // 8
    ms = gpu_ms(lambda: ctx.outer_apply(g[:L], 8, theta[:L], mom[:L], lr=LR, momentum=MU), flush=True)
    emit("exchange form", "adloco_outer_apply (one rank's slice of 8, P/8 elements)", ms, nbytes=(4 + 8 + 8) * L,
         note="L2 flushed; 311 MB per call")
    ms = gpu_ms(lambda: ctx.refresh_instance(theta, inst[0]))
    emit("exchange form", "adloco_refresh_instance (bf16 instance, P=124,439,808)", ms, nbytes=(4 + 2) * P)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--table", action="store_true", help="per-configuration table, one JSON line per row")
    ap.add_argument("--small", action="store_true",
                    help="profiling case: same kernels on inputs of a few hundred MB (not a bench value)")
    args = ap.parse_args()
    if args.small:
        global NT_P, OUT_P, C4_SHAPES, C4_MICRO, C5_P, C5_MICRO, C5_ACC_P
        NT_P, OUT_P = 1 << 21, 1 << 24      # the Gram layer (252 MB) stays at its full size
        C4_SHAPES, C4_MICRO = list(W.GPT2_SMALL_BLOCK_LINEARS), 1     # one transformer block, one micro-batch
        C5_P, C5_MICRO, C5_ACC_P = 1 << 25, 2, 1 << 21
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.table:
        if rank == 0:
            run_table(args)
        return
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
