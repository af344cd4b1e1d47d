"""Seeded synthetic inputs shaped like the paper's LLM workloads.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic, so both the CUDA tests and the CPU oracle tests may use
it.  Every generator takes a seed and a torch device and returns torch
tensors; bfloat16 tensors are produced by rounding the float32 draw.

Recipes
  * per-sample gradients: g_i = m + sigma * z_i, z_i ~ N(0, I_P); the common
    mean m is N(0, I)/sqrt(P) (noise-dominated, ||m||^2 ~ 1) or N(0, I)
    (signal-dominated, ||m||^2 ~ P).
  * outer step: theta ~ N(0, 0.02^2) (GPT-2 initialisation scale), the K
    instances theta_k = theta + N(0, (1e-3)^2), optionally rounded to bf16;
    momentum zero or N(0, (1e-3)^2).
  * linear layer: activations X ~ N(0, 1) [B, T, d_in] and output gradients
    Delta ~ N(0, (1e-2)^2) [B, T, d_out], both rounded to bf16.
"""
from __future__ import annotations

import torch

GPT2_SMALL_P = 124_439_808          # flat parameter count of a GPT-2-small sized model
LARGE_P = 1_300_000_000             # "1.3B" flat parameter vector

# the four weight matrices of one GPT-2-small transformer block: (d_in, d_out)
GPT2_SMALL_BLOCK_LINEARS = ((768, 2304), (768, 768), (768, 3072), (3072, 768))


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, gen, device, chunk_rows=None):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def per_sample_grads(B: int, P: int, *, sigma: float = 0.5, mean_scale: str = "unit",
                     seed: int = 0, device="cpu", row_stride: int | None = None):
    """G [B, P] float32 with G[i] = m + sigma * z_i.  mean_scale "unit" draws
    m ~ N(0,1)/sqrt(P); "raw" draws m ~ N(0,1).  With row_stride > P the rows
    live in a wider buffer (the view returned is [B, P], stride row_stride)."""
    gen = _gen(seed, device)
    m = _randn((P,), gen, device)
    if mean_scale == "unit":
        m = m / float(P) ** 0.5
    elif mean_scale != "raw":
        raise ValueError(mean_scale)
    stride = P if row_stride is None else int(row_stride)
    buf = torch.empty((B, stride), dtype=torch.float32, device=device)
    G = buf[:, :P]
    for i in range(B):                       # row by row keeps the peak footprint low
        z = _randn((P,), gen, device)
        G[i] = m + sigma * z
    return G


def micro_batches(n_micro: int, b_micro: int, P: int, *, sigma: float, mean_scale: str = "unit",
                  seed: int = 0, device="cpu"):
    """Switch-mode workload: one batch of n_micro*b_micro samples delivered as
    n_micro separate [b_micro, P] float32 tensors sharing one mean m."""
    G = per_sample_grads(n_micro * b_micro, P, sigma=sigma, mean_scale=mean_scale,
                         seed=seed, device=device)
    return [G[j * b_micro:(j + 1) * b_micro] for j in range(n_micro)]


def outer_state(K: int, P: int, *, inst_dtype=torch.float32, zero_momentum: bool = True,
                seed: int = 0, device="cpu"):
    """(theta fp32 [P], list of K instance tensors [P] in inst_dtype, momentum fp32 [P]).
    Every instance is a separate allocation."""
    gen = _gen(seed, device)
    theta = 0.02 * _randn((P,), gen, device)
    inst = []
    for _ in range(K):
        t = theta + 1e-3 * _randn((P,), gen, device)
        inst.append(t.to(inst_dtype).contiguous())
        del t
    if zero_momentum:
        mom = torch.zeros(P, dtype=torch.float32, device=device)
    else:
        mom = 1e-3 * _randn((P,), gen, device)
    return theta, inst, mom


def linear_layer(B: int, T: int, d_in: int, d_out: int, *, delta_std: float = 1e-2,
                 seed: int = 0, device="cpu"):
    """(X bf16 [B, T, d_in], Delta bf16 [B, T, d_out])."""
    gen = _gen(seed, device)
    X = _randn((B, T, d_in), gen, device).to(torch.bfloat16)
    D = (delta_std * _randn((B, T, d_out), gen, device)).to(torch.bfloat16)
    return X, D


def small_integer_layer(B: int, T: int, d_in: int, d_out: int, *, seed: int = 0, device="cpu"):
    """X, Delta with small integer entries (exact in bf16 and in every partial
    sum), for brute-force checks."""
    gen = _gen(seed, device)
    X = torch.randint(-3, 4, (B, T, d_in), generator=gen, device=device).to(torch.bfloat16)
    D = torch.randint(-3, 4, (B, T, d_out), generator=gen, device=device).to(torch.bfloat16)
    return X, D


def to_numpy(t: torch.Tensor):
    """Host numpy view of a tensor's bytes; bfloat16 comes back as uint16 bit patterns."""
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view("uint16")
    return t.numpy()
