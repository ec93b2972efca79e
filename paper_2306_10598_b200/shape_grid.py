"""How the sweep's throughput depends on the shape of the input: a table of GB/s over worker counts N and
micro-batch counts M at a fixed number of latency bytes, for both completion rules.

    python -m paper_2306_10598_b200.shape_grid --bytes 4e8 3e9

Inputs are uniform latencies with an evenly spaced grid of 64 thresholds over [0.6, 1.4] x the mean row total;
a 256 MiB buffer is written between launches; each cell is the median of five launches of dc_simulate_ex
(CUDA events).  Useful to see which kernel and schedule a shape gets and what it costs: few workers per trial
(a block takes one trial at a time), very short rows, row lengths with a ragged last chunk."""
from __future__ import annotations

import argparse
import statistics

import torch

from . import api


def cell(T: int, N: int, M: int, K: int, rule: int, flush: torch.Tensor, device, reps: int = 5) -> float:
    g = torch.Generator(device=device).manual_seed(1)
    lat = torch.rand(T, N, M, device=device, generator=g) * 0.01 + 0.02
    mean = 0.025 * M
    taus = torch.linspace(0.6 * mean, 1.4 * mean, K, device=device)
    step = torch.empty(T, K, dtype=torch.float32, device=device)
    done = torch.empty(T, K, dtype=torch.int32, device=device)
    sync = torch.empty(T, dtype=torch.float32, device=device)
    ms = []
    for i in range(reps + 2):
        flush.fill_(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        api.dc_simulate_ex(lat, taus, 0.1, step, done, sync, rule)
        e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            ms.append(e0.elapsed_time(e1))
    return 4 * T * N * M / statistics.median(ms) / 1e6


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--bytes", type=float, nargs="+", default=[4e8, 3e9])
    ap.add_argument("--workers", type=int, nargs="+", default=[8, 32, 100, 200, 256, 300, 512, 1000, 2048, 5000])
    ap.add_argument("--microbatches", type=int, nargs="+", default=[4, 8, 12, 16, 24, 32, 48, 64, 100, 128, 256, 512])
    ap.add_argument("--thresholds", type=int, default=64)
    args = ap.parse_args()
    device = torch.device("cuda", torch.cuda.current_device())
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    for total in args.bytes:
        print(f"{total:.1e} latency bytes; rows: workers N, columns: micro-batches M; GB/s under rule 0 / rule 1")
        print("N\\M   " + "".join(f"{m:>12d}" for m in args.microbatches))
        for N in args.workers:
            row = []
            for M in args.microbatches:
                T = max(1, int(total / (4 * N * M)))
                row.append(f"{cell(T, N, M, args.thresholds, 0, flush, device):6.0f}/{cell(T, N, M, args.thresholds, 1, flush, device):5.0f}")
            print(f"{N:5d} " + "".join(f"{x:>12s}" for x in row), flush=True)
    api.dc_device_status()


if __name__ == "__main__":
    main()
