"""Running the sweep on several GPUs: trials are independent (Algorithm 2's loop over iterations), so each
rank sweeps its own trials with no exchange inside ``dc_simulate``.  This module holds the small host-side
pieces of that: how trials are split, how a benchmark time is agreed on, and the one exchange a caller
needs if it wants the statistics of ALL trials — a sum over ranks of 4K+2 doubles.

Everything here works on whatever device the tensors live on and with whatever ``torch.distributed``
backend the caller initialised (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Optional, Tuple

import torch

from . import workloads as W

MEAN_STEP, DONE_FRAC, THR, THR_MEAN, S_EFF = range(5)


def trial_range(T: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous share of trials ``[t0, t1)`` of rank ``rank``; shares differ by at most one trial and
    cover 0..T exactly."""
    if not (0 <= rank < world) or T < 0:
        raise ValueError("bad rank/world/T")
    base, extra = divmod(T, world)
    t0 = rank * base + min(rank, extra)
    return t0, t0 + base + (1 if rank < extra else 0)


def rank_workload(w: W.Workload, rank: int) -> W.Workload:
    """The benchmark's weak-scaling input of one rank: the same shape, law and grid, its own seed."""
    return W.Workload(w.name, w.T, w.N, w.M, w.K, w.tau_lo, w.tau_hi, w.tau_unit, w.t_comm, w.law, seed=w.seed + rank)


def max_over_ranks(value: float, device, group=None) -> float:
    """The slowest rank's time (the number a multi-GPU benchmark must report)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def combine_stats(stats: torch.Tensor, baseline: torch.Tensor, T_local: int, N: int, M: int, group=None
                  ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Statistics over the trials of all ranks from each rank's ``dc_reduce_trials`` output.

    Means over trials combine as trial-weighted means; the two ratios of sums are rebuilt from the
    summed numerators and denominators:  thr = sum(done) / sum(step),  thr_sync = T N M / sum(sync).
    One all-reduce (SUM) of 4K+2 doubles."""
    import torch.distributed as dist
    K = stats.shape[1]
    Tl = float(T_local)
    packed = torch.empty(4 * K + 2, dtype=torch.float64, device=stats.device)
    packed[0 * K:1 * K] = stats[MEAN_STEP] * Tl            # sum of step
    packed[1 * K:2 * K] = stats[DONE_FRAC] * Tl            # sum of done / (N M)
    packed[2 * K:3 * K] = stats[THR_MEAN] * Tl
    packed[3 * K:4 * K] = stats[S_EFF] * Tl
    packed[4 * K] = baseline[0] * Tl                       # sum of sync
    packed[4 * K + 1] = Tl
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(packed, op=dist.ReduceOp.SUM, group=group)
    Tg = packed[4 * K + 1]
    out = torch.empty_like(stats)
    out[MEAN_STEP] = packed[0 * K:1 * K] / Tg
    out[DONE_FRAC] = packed[1 * K:2 * K] / Tg
    out[THR] = packed[1 * K:2 * K] * float(N * M) / packed[0 * K:1 * K]
    out[THR_MEAN] = packed[2 * K:3 * K] / Tg
    out[S_EFF] = packed[3 * K:4 * K] / Tg
    base = torch.empty_like(baseline)
    base[0] = packed[4 * K] / Tg
    base[1] = Tg * float(N * M) / packed[4 * K]
    return out, base
