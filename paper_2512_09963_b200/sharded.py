"""A verification round sharded over ranks (one process per GPU).

The path shards by draft server: attention, the LM head (every rank holds its own copy of W),
acceptance and the estimator updates are independent per server, so each rank runs them on its own
servers with no exchange.  Only the scheduler couples the servers, through the budget
sum_i S_i <= C (Eq. goodspeed_sched): before it runs, the ranks all-gather their estimator state
(alpha_hat_i, X_i: 16 bytes per server), every rank solves the same global allocation with the same
deterministic routine, and keeps the slice of its own servers.

`ShardedScheduler` is that exchange.  Tensors on a CUDA device go through NCCL and gs_schedule;
host tensors go through gloo and gs_schedule_host (the same allocation, bit for bit).  No arithmetic
of the method happens here: packing, one collective, one library call, one slice.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import binding as B


class ShardedScheduler:
    """Buffers and the per-round exchange for `n_local` servers on each of `world` ranks.

    budget_total is the global token budget C (for weak scaling: the per-rank budget times world).
    s_min / s_max, if given, are the GLOBAL boxes, [n_local * world] int32, rank-major.
    """

    def __init__(self, n_local: int, rank: int, world: int, budget_total: int, device,
                 s_min: Optional[torch.Tensor] = None, s_max: Optional[torch.Tensor] = None, group=None):
        self.n, self.rank, self.world, self.C = int(n_local), int(rank), int(world), int(budget_total)
        self.dev = torch.device(device)
        self.group = group
        f64, i32 = torch.float64, torch.int32
        n_all = self.n * self.world
        self.est_local = torch.empty(2 * self.n, dtype=f64, device=self.dev)     # [alpha_hat | X] of this rank
        self.est_all = torch.empty(2 * n_all, dtype=f64, device=self.dev)        # rank-major gather
        self.alpha_all = torch.empty(n_all, dtype=f64, device=self.dev)
        self.X_all = torch.empty(n_all, dtype=f64, device=self.dev)
        self.S_all = torch.empty(n_all, dtype=i32, device=self.dev)
        for t in (s_min, s_max):
            if t is not None and (t.numel() != n_all or t.dtype != i32):
                raise ValueError("s_min / s_max must be int32 tensors with one entry per server of every rank")
        self.s_min, self.s_max = s_min, s_max

    def step(self, alpha_hat: torch.Tensor, X: torch.Tensor, S_local_out: torch.Tensor,
             d_status: Optional[torch.Tensor] = None) -> torch.Tensor:
        """alpha_hat, X: this rank's [n_local] fp64 estimates.  Writes this rank's slice of the global
        allocation to S_local_out ([n_local] int32) and returns the global allocation (a buffer that
        the next call overwrites)."""
        n, w = self.n, self.world
        self.est_local[:n].copy_(alpha_hat)
        self.est_local[n:].copy_(X)
        if w > 1:
            dist.all_gather_into_tensor(self.est_all, self.est_local, group=self.group)
        else:
            self.est_all.copy_(self.est_local)
        g = self.est_all.view(w, 2, n)
        self.alpha_all.copy_(g[:, 0, :].reshape(-1))
        self.X_all.copy_(g[:, 1, :].reshape(-1))
        if self.dev.type == "cuda":
            B.gs_schedule(self.X_all, self.alpha_all, self.C, self.S_all, self.s_min, self.s_max, d_status)
        else:
            B.gs_schedule_host(self.X_all, self.alpha_all, self.C, self.S_all, self.s_min, self.s_max)
        S_local_out.copy_(self.S_all[self.rank * n:(self.rank + 1) * n])
        return self.S_all


def aggregate_throughput(ms_local: float, units_local: int, device, group=None):
    """Whole-job figures from per-rank ones: the slowest rank's time (MAX) and all ranks' units (SUM)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(ms_local), int(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    u = torch.tensor([units_local], dtype=torch.int64, device=device)
    dist.all_reduce(u, group=group)
    return float(t.item()), int(u.item())
