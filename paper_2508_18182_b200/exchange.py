"""The outer step with one whole model instance per GPU (last loop of Algorithm 3 as a
distributed job): every rank holds its trained instance theta_k, the shared starting
point theta, and one slice of the momentum.  The only exchange is the reduce-scatter of
the pseudo-gradients theta - theta_k -- the single communication of the method -- then
each rank updates its slice and the new theta is gathered so that every worker restarts
from it.

`torch.distributed` moves the bytes (NCCL between GPUs, gloo between CPU processes);
the arithmetic runs in the library's kernels (`kernels` is a binding.Context).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def slice_length(P: int, world: int, align: int = 8) -> int:
    """Elements per rank when [0, P) is cut into `world` equal slices whose length is a
    multiple of `align` (so fp32 and bf16 slices start on 16-byte boundaries); the last
    slices may reach beyond P and are padded with zeros in the exchange buffer."""
    if P < 0 or world < 1 or align < 1:
        raise ValueError("bad slice request")
    per = -(-P // world)
    return max(align, -(-per // align) * align)


class ExchangedOuterStep:
    """State of one rank: buffers sized once, reused every outer step.

    theta      fp32 [P]   the starting point shared by all ranks (updated in place)
    instance   [P]        this rank's trained copy theta_k (fp32 or bf16; refreshed in place)
    momentum   fp32 [L]   this rank's slice of v, L = slice_length(P, world)
    """

    def __init__(self, kernels, theta, instance, momentum_slice, *, group=None):
        self.k = kernels
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.P = theta.numel()
        self.L = slice_length(self.P, self.world)
        if momentum_slice.numel() != self.L or instance.numel() != self.P:
            raise ValueError("momentum slice must have slice_length(P, world) elements, the instance P")
        self.theta, self.instance, self.mom = theta, instance, momentum_slice
        dev = theta.device
        self.padded = self.L * self.world
        self.g = torch.zeros(self.padded, dtype=torch.float32, device=dev)        # pseudo-gradient, zero tail
        self.g_sum = torch.empty(self.L, dtype=torch.float32, device=dev)         # this rank's slice of the sum
        self.theta_pad = torch.zeros(self.padded, dtype=torch.float32, device=dev)
        self.lo = min(self.P, self.rank * self.L)
        self.hi = min(self.P, self.lo + self.L)

    def step(self, *, lr: float, momentum: float, nesterov: bool = True):
        """One outer step.  Returns theta (updated in place on every rank)."""
        k = self.k
        k.pseudo_gradient(self.theta, self.instance, self.g[:self.P])
        dist.reduce_scatter_tensor(self.g_sum, self.g, op=dist.ReduceOp.SUM, group=self.group)
        n = self.hi - self.lo
        my = self.theta_pad[self.rank * self.L:(self.rank + 1) * self.L]
        if n > 0:
            my[:n].copy_(self.theta[self.lo:self.hi])
            k.outer_apply(self.g_sum[:n], self.world, my[:n], self.mom[:n], lr=lr, momentum=momentum, nesterov=nesterov)
        dist.all_gather_into_tensor(self.theta_pad, my.clone(), group=self.group)
        self.theta.copy_(self.theta_pad[:self.P])
        k.refresh_instance(self.theta, self.instance)
        return self.theta
