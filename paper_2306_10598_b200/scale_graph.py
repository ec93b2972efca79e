"""Scale graph of App. C.3 / Fig. 1 (right): how the synchronous step time and the gain from DropCompute grow
with the number of workers, for one of the paper's synthetic noise laws.

    python -m paper_2306_10598_b200.scale_graph --noise lognormal_0.05 --workers 8 64 512 2048 --trials 512

For every N it runs the GPU sweep (dc_simulate_ex, dc_reduce_trials, dc_argmax_tau) on T trials of 12
accumulations of 0.45 s + eps and prints: E[T]/E[T_i] (mean slowest worker over mean single worker — the
indicator the paper tabulates), the automatically chosen tau*, S_eff(tau*), the drop rate at tau*, and the
closed-form S_eff at the same tau (dc_closed_form with the measured E[T]).  Nothing here computes the method:
all numbers come from the library's kernels."""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import api
from . import workloads as W


def scale_row(noise: str, N: int, trials: int, K: int, t_comm: float, seed: int = 0, device="cuda") -> dict:
    w = W.c3_workload(noise, N=N, T=trials, K=K, t_comm=t_comm, seed=seed) if noise != "b1_delay" else \
        W.b1_workload(N=N, T=trials, K=K, t_comm=t_comm, seed=seed)
    lat = W.fill_latencies(w, device)
    taus = torch.from_numpy(W.make_taus(w)).to(device)
    r = api.sweep(lat, taus, w.t_comm)
    single = float(lat.sum(-1, dtype=torch.float64).mean())            # E[T_i]: mean time of one worker alone
    var = float(lat.double().var())
    mu = single / w.M
    cf = torch.empty((3, w.K), dtype=torch.float64, device=device)
    sc = torch.empty(1, dtype=torch.float64, device=device)
    mean_T = float(r.baseline[0]) - w.t_comm
    api.dc_closed_form(mu, math.sqrt(var), w.M, N, w.t_comm, taus, cf, sc, mean_T=mean_T)
    k = int(r.k_star)
    return {"noise": noise, "N": N, "trials": trials, "E[T]/E[T_i]": mean_T / single, "tau_star": float(r.tau_star),
            "s_eff": float(r.value), "drop_rate": 1.0 - float(r.stats[api.STAT_DONE_FRAC, k]),
            "s_eff_closed_form_given_E[T]": float(cf[2, k]), "mean_sync": float(r.baseline[0])}


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--noise", default="lognormal_0.05", choices=sorted(W.C3_NOISE) + ["b1_delay"])
    ap.add_argument("--workers", type=int, nargs="+", default=[8, 32, 128, 512, 2048])
    ap.add_argument("--trials", type=int, default=512)
    ap.add_argument("--K", type=int, default=128)
    ap.add_argument("--t-comm", type=float, default=0.5)
    args = ap.parse_args()
    for N in args.workers:
        print(json.dumps(scale_row(args.noise, N, args.trials, args.K, args.t_comm)), flush=True)


if __name__ == "__main__":
    main()
