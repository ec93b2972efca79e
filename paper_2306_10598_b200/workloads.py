"""Seeded synthetic latency tensors and threshold grids.

This module only draws random inputs: it contains none of the simulator's
arithmetic and is the one module both the CUDA path's tests/benchmark and the
CPU oracle's tests read their inputs from.

The paper's measured micro-batch latency traces are not available, so each
workload is a synthetic tensor ``latencies[T, N, M]`` (trials x workers x
gradient accumulations, fp32 seconds) shaped like the paper's runs: about 200
measured workers and an extrapolation to 2048 (Fig. 1), 12 to 64 accumulations
(Sec. 5.2, Fig. 4, Fig. 6), additive straggler noise (App. B.1), plus a tiny
case and a bandwidth-stress case.

Draw order.  A tensor is filled in chunks of whole trials.  Chunk ``c`` uses
its own ``torch.Generator`` seeded with ``seed * 1_000_003 + c`` on the target
device, and inside a chunk the draws are made in the order written in the
``_fill_*`` function of the law.  Any range of trials can therefore be
regenerated on the same kind of device without generating the rest.  CPU and
CUDA generators give different bits, so a comparison always copies one tensor
to both sides and never regenerates it.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Callable, Dict, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    N: int
    M: int
    K: int
    tau_lo: float       # grid start, in units of `tau_unit`
    tau_hi: float       # grid end (inclusive), in units of `tau_unit`
    tau_unit: float     # seconds: 1.0 for an absolute grid, else the analytic mean worker time
    t_comm: float
    law: str
    seed: int = 0

    @property
    def samples(self) -> int:
        return self.T * self.N * self.M

    @property
    def latency_bytes(self) -> int:
        return 4 * self.samples

    def with_trials(self, T: int) -> "Workload":
        return Workload(self.name, T, self.N, self.M, self.K, self.tau_lo, self.tau_hi, self.tau_unit,
                        self.t_comm, self.law, self.seed)


# Analytic mean of one worker's total compute time under each law (so that the
# grid does not depend on the draw).
_MEAN_PAPER = 32 * 0.025 + 0.05                                           # 0.85 s
_MEAN_EXTRA = 16 * (0.03 * math.exp(0.1 ** 2 / 2) + 0.005 * 0.3)          # 0.506406 s
_MEAN_CORR = 64 * math.exp(0.05 ** 2 / 2) * 0.01 * math.exp(0.15 ** 2 / 2)  # 0.648050 s
_MEAN_STRESS = 128 * (0.005 + 2 * 0.001)                                  # 0.896 s

WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in (
        Workload("tiny", 1024, 8, 4, 16, 0.2, 0.6, 1.0, 0.05, "shifted_exp"),
        Workload("paper_scale", 16384, 200, 32, 64, 0.5, 1.5, _MEAN_PAPER, 0.1, "normal_head_exp"),
        Workload("extrapolation", 4096, 2048, 16, 128, 0.8, 2.0, _MEAN_EXTRA, 0.2, "lognormal_straggler"),
        Workload("correlated", 8192, 4096, 64, 256, 0.7, 1.5, _MEAN_CORR, 0.15, "correlated_lognormal"),
        Workload("bandwidth_stress", 32768, 2048, 128, 256, 0.6, 1.4, _MEAN_STRESS, 0.1, "shifted_gamma2"),
    )
}


def make_taus(w: Workload) -> np.ndarray:
    """K evenly spaced thresholds including both ends, computed in fp64 and rounded once to fp32."""
    grid = np.linspace(w.tau_lo * w.tau_unit, w.tau_hi * w.tau_unit, w.K, dtype=np.float64)
    return grid.astype(np.float32)


def worker_scales(N: int, seed: int = 0, spread: float = 0.2) -> np.ndarray:
    """Per-worker threshold scales s_n for the heterogeneous-worker sweep: fp32, uniform on [1 - spread, 1 + spread]
    (a fleet whose workers' paces differ by up to +-spread), drawn with numpy's seeded generator."""
    rng = np.random.default_rng(7_000_003 * (seed + 1) + N)
    return rng.uniform(1.0 - spread, 1.0 + spread, N).astype(np.float32)


# --- the laws -------------------------------------------------------------
# Every function fills out[t0:t1] (a [n_trials, N, M] fp32 view) using generator g.

def _fill_shifted_exp(out: torch.Tensor, g: torch.Generator) -> None:
    # 0.1 s + Exponential(mean 0.02 s), iid
    out.exponential_(1.0 / 0.02, generator=g)
    out.add_(0.1)


def _fill_normal_head_exp(out: torch.Tensor, g: torch.Generator) -> None:
    # Normal(0.025, sd 0.002) clipped at 0, iid; then Exponential(mean 0.05) per (trial, worker) added to m = 0
    out.normal_(0.025, 0.002, generator=g)
    out.clamp_(min=0.0)
    head = torch.empty(out.shape[:2], dtype=out.dtype, device=out.device)
    head.exponential_(1.0 / 0.05, generator=g)
    out[:, :, 0].add_(head)


def _fill_lognormal_straggler(out: torch.Tensor, g: torch.Generator) -> None:
    # 0.03 s x LogNormal(0, 0.1), iid; with probability 0.005 a sample gets Uniform(0.1, 0.5) s added
    out.log_normal_(0.0, 0.1, generator=g)
    out.mul_(0.03)
    u = torch.empty_like(out).uniform_(0.0, 1.0, generator=g)
    extra = torch.empty_like(out).uniform_(0.1, 0.5, generator=g)
    out.add_(torch.where(u < 0.005, extra, torch.zeros_like(extra)))


def _fill_correlated_lognormal(out: torch.Tensor, g: torch.Generator) -> None:
    # LogNormal(ln 0.01, 0.15) per sample x LogNormal(0, 0.05) per (trial, worker)
    out.log_normal_(math.log(0.01), 0.15, generator=g)
    slow = torch.empty(out.shape[:2], dtype=out.dtype, device=out.device)
    slow.log_normal_(0.0, 0.05, generator=g)
    out.mul_(slow.unsqueeze(-1))


def _fill_shifted_gamma2(out: torch.Tensor, g: torch.Generator) -> None:
    # 0.005 s + Gamma(shape 2, scale 0.001 s) = 0.005 + 0.001 (E1 + E2), E ~ Exponential(1), iid
    out.exponential_(1.0, generator=g)
    e2 = torch.empty_like(out).exponential_(1.0, generator=g)
    out.add_(e2)
    out.mul_(0.001)
    out.add_(0.005)


_LAWS: Dict[str, Callable[[torch.Tensor, torch.Generator], None]] = {
    "shifted_exp": _fill_shifted_exp,
    "normal_head_exp": _fill_normal_head_exp,
    "lognormal_straggler": _fill_lognormal_straggler,
    "correlated_lognormal": _fill_correlated_lognormal,
    "shifted_gamma2": _fill_shifted_gamma2,
}

# --- the paper's own synthetic settings (App. B.1 and C.3) -------------------------------------------
# App. C.3 simulates 12 accumulations of 0.45 s + eps with eps drawn from one of the laws of its two tables
# (all with mean 0.225; variance 0.05 unless stated).  App. B.1 adds to a base latency mu the bounded
# log-normal delay  mu * min(Z / alpha, beta),  Z ~ LogNormal(4, 1), alpha = 2 exp(4.5), beta = 5.5.
C3_BASE = 0.45
C3_M = 12
C3_NOISE = {
    # name: (kind, parameters as printed in the tables)
    "lognormal_0.05": ("lognormal", -1.84, 0.83),
    "normal_0.05": ("normal", 0.23, 0.22),
    "bernoulli_0.05": ("bernoulli", 0.45, 0.5),
    "exponential_0.05": ("exponential", 4.47),
    "gamma_0.05": ("gamma1", 4.5),
    "lognormal_0.10": ("lognormal", -2.04, 1.04),
    "lognormal_0.15": ("lognormal", -2.18, 1.17),
    "lognormal_0.20": ("lognormal", -2.29, 1.26),
    "lognormal_0.25": ("lognormal", -2.38, 1.33),
    "lognormal_0.30": ("lognormal", -2.46, 1.39),
}
B1_ALPHA = 2.0 * math.exp(4.5)
B1_BETA = 5.5


def _fill_c3(out: torch.Tensor, g: torch.Generator, name: str) -> None:
    spec = C3_NOISE[name]
    kind = spec[0]
    if kind == "lognormal":
        out.log_normal_(spec[1], spec[2], generator=g)
    elif kind == "normal":
        out.normal_(spec[1], spec[2], generator=g)
        out.clamp_(min=-C3_BASE)          # a latency cannot be negative (a -3.1 sigma draw)
    elif kind == "bernoulli":
        out.uniform_(0.0, 1.0, generator=g)
        out.copy_(torch.where(out < spec[2], torch.full_like(out, spec[1]), torch.zeros_like(out)))
    elif kind == "exponential":
        out.exponential_(spec[1], generator=g)
    elif kind == "gamma1":                # Gamma(shape 1, rate 4.5) is Exponential(rate 4.5)
        out.exponential_(spec[1], generator=g)
    else:
        raise ValueError(kind)
    out.add_(C3_BASE)


def _fill_b1(out: torch.Tensor, g: torch.Generator, mu: float) -> None:
    # base latency mu plus the bounded log-normal delay of App. B.1
    out.log_normal_(4.0, 1.0, generator=g)
    out.div_(B1_ALPHA)
    out.clamp_(max=B1_BETA)
    out.mul_(mu)
    out.add_(mu)


def c3_workload(name: str, N: int, T: int = 256, K: int = 64, t_comm: float = 0.5, seed: int = 0) -> Workload:
    """App. C.3: 12 accumulations of 0.45 s + eps, eps from the table row `name`; grid over [0.6, 2.0] x the
    mean worker time 12 * 0.675 s."""
    if name not in C3_NOISE:
        raise ValueError(name)
    return Workload(f"c3_{name}", T, N, C3_M, K, 0.6, 2.0, C3_M * (C3_BASE + 0.225), t_comm, f"c3:{name}", seed)


def b1_workload(N: int, mu: float = 0.45, M: int = 12, T: int = 256, K: int = 64, t_comm: float = 0.5, seed: int = 0) -> Workload:
    """App. B.1: every accumulation takes mu * (1 + min(Z / alpha, beta)); the delay has mean about 0.5 mu."""
    return Workload("b1_delay", T, N, M, K, 0.6, 2.5, M * mu * 1.5, t_comm, f"b1:{mu!r}", seed)


_CHUNK_FLOATS = 1 << 26  # 256 MB of fp32 per chunk of whole trials


def chunk_trials(w: Workload) -> int:
    return max(1, _CHUNK_FLOATS // (w.N * w.M))


def fill_latencies(w: Workload, device, out: Optional[torch.Tensor] = None,
                   t0: int = 0, t1: Optional[int] = None) -> torch.Tensor:
    """Trials ``t0:t1`` of workload ``w`` on ``device``: a contiguous fp32 ``[t1-t0, N, M]`` tensor.

    The result does not depend on which range is asked for: trial t always
    comes from chunk ``t // chunk_trials(w)`` of the seeded sequence."""
    t1 = w.T if t1 is None else t1
    assert 0 <= t0 <= t1 <= w.T
    device = torch.device(device)
    if out is None:
        out = torch.empty((t1 - t0, w.N, w.M), dtype=torch.float32, device=device)
    assert out.shape == (t1 - t0, w.N, w.M) and out.dtype == torch.float32 and out.is_contiguous()
    ct = chunk_trials(w)
    if w.law.startswith("c3:"):
        law = lambda o, g, _n=w.law[3:]: _fill_c3(o, g, _n)
    elif w.law.startswith("b1:"):
        law = lambda o, g, _m=float(w.law[3:]): _fill_b1(o, g, _m)
    else:
        law = _LAWS[w.law]
    c = t0 // ct
    while c * ct < t1:
        lo, hi = c * ct, min((c + 1) * ct, w.T)
        g = torch.Generator(device=device)
        g.manual_seed(w.seed * 1_000_003 + c)
        a, b = max(lo, t0), min(hi, t1)
        if a == lo and b == hi:
            law(out[a - t0:b - t0], g)
        else:  # partial chunk: draw the whole chunk, keep the part asked for
            tmp = torch.empty((hi - lo, w.N, w.M), dtype=torch.float32, device=device)
            law(tmp, g)
            out[a - t0:b - t0].copy_(tmp[a - lo:b - lo])
            del tmp
        c += 1
    return out


# --- small generic inputs for tests --------------------------------------

def iid_latencies(law: str, T: int, N: int, M: int, seed: int, device="cpu", **p) -> torch.Tensor:
    """Small iid tensors for closed-form checks: 'exp'(rate), 'normal'(mu, sd), 'shifted_exp'(shift, mean),
    'uniform'(lo, hi), 'dyadic' (values k/64, k in 1..hi: sums are exact in fp32)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = torch.empty((T, N, M), dtype=torch.float32, device=device)
    if law == "exp":
        out.exponential_(p["rate"], generator=g)
    elif law == "normal":
        out.normal_(p["mu"], p["sd"], generator=g)
    elif law == "shifted_exp":
        out.exponential_(1.0 / p["mean"], generator=g)
        out.add_(p["shift"])
    elif law == "uniform":
        out.uniform_(p["lo"], p["hi"], generator=g)
    elif law == "dyadic":
        k = torch.randint(1, int(p["hi"]) + 1, (T, N, M), generator=g, device=device)
        out.copy_(k.to(torch.float32) / 64.0)
    else:
        raise ValueError(law)
    return out
