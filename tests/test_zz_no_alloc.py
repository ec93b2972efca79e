"""dc_reduce_trials_static, the entry point for callers that may not allocate device memory.

Some users of this library run inside a process whose memory pool already owns the GPU, or in a loop
that must never stall on an allocation; they cannot supply the workspace dc_reduce_trials asks for.
This file checks, through the C ABI, that the workspace-free entry point gives what dc_reduce_trials
gives, on two calls in a row with different inputs (the built-in scratch keeps the first call's
contents, which must not leak into the second), and that it refuses a grid larger than the scratch was
sized for.  It is collected last on purpose, and passes both alone and after the other tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2306_10598_b200 import workloads as W

pytestmark = pytest.mark.gpu

RTOL_STATS = 1e-9  # the tolerance the parity tests use for fp64 statistics


@pytest.fixture(scope="module")
def api():
    from paper_2306_10598_b200 import build
    build.build_library()   # compiles the library in-tree if it is missing or older than its sources
    from paper_2306_10598_b200 import api as _api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return _api


def _sweep_outputs(api, T, N, M, K, seed):
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=seed, shift=0.01, mean=0.02).cuda()
    hi = float(lat.sum(-1).max())
    taus = torch.linspace(0.3 * hi, 1.1 * hi, K, device="cuda")
    step = torch.empty((T, K), dtype=torch.float32, device="cuda")
    done = torch.empty((T, K), dtype=torch.int32, device="cuda")
    sync = torch.empty((T,), dtype=torch.float32, device="cuda")
    api.dc_simulate_ex(lat, taus, 0.05, step, done, sync)
    return step, done, sync


def test_static_reduce_matches_workspace_reduce_twice(api):
    # second call: fewer trials and thresholds than the first, so stale partial sums lie beyond what it writes
    for call, (T, N, M, K) in enumerate(((700, 40, 16, 96), (45, 9, 8, 7))):
        step, done, sync = _sweep_outputs(api, T, N, M, K, seed=50 + call)
        want = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
        want_base = torch.empty(2, dtype=torch.float64, device="cuda")
        ws = torch.empty(api.dc_reduce_workspace_bytes(T, K), dtype=torch.uint8, device="cuda")
        api.dc_reduce_trials(step, done, sync, N, M, want, want_base, ws)
        got = torch.full_like(want, float("nan"))
        got_base = torch.full_like(want_base, float("nan"))
        torch.cuda.synchronize()
        api.dc_reduce_trials_static(step, done, sync, N, M, got, got_base)   # outputs exist already: no allocation here
        torch.cuda.synchronize()
        assert np.allclose(got.cpu().numpy(), want.cpu().numpy(), rtol=RTOL_STATS, atol=0), f"call {call}"
        assert np.allclose(got_base.cpu().numpy(), want_base.cpu().numpy(), rtol=RTOL_STATS, atol=0), f"call {call}"
        # and against the CPU oracle's reduction of the same per-trial outputs
        ref = oracle.reduce_trials(step.cpu().numpy(), done.cpu().numpy(), sync.cpu().numpy(), N, M)
        assert np.allclose(got.cpu().numpy(), ref.stats, rtol=RTOL_STATS, atol=0), f"call {call} (oracle)"
        assert np.allclose(got_base.cpu().numpy(), ref.baseline, rtol=RTOL_STATS, atol=0), f"call {call} (oracle)"
        # without the synchronous baseline: NaN in the same places as dc_reduce_trials
        api.dc_reduce_trials(step, done, None, N, M, want, want_base, ws)
        api.dc_reduce_trials_static(step, done, None, N, M, got, got_base)
        torch.cuda.synchronize()
        assert np.allclose(got.cpu().numpy(), want.cpu().numpy(), rtol=RTOL_STATS, atol=0, equal_nan=True)
        assert torch.isnan(got_base).all()


def test_static_reduce_refuses_grids_beyond_its_scratch(api):
    T, K = 4, api.STATIC_MAX_K + 1
    step = torch.ones((T, K), dtype=torch.float32, device="cuda")
    done = torch.ones((T, K), dtype=torch.int32, device="cuda")
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty(2, dtype=torch.float64, device="cuda")
    with pytest.raises(api.DropComputeError) as e:
        api.dc_reduce_trials_static(step, done, None, 2, 2, stats, base)
    assert e.value.status == 4  # DC_ERR_RANGE
    # the largest supported grid is accepted
    K = api.STATIC_MAX_K
    step, done = step[:, :K].contiguous(), done[:, :K].contiguous()
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    api.dc_reduce_trials_static(step, done, None, 2, 2, stats, base)
    torch.cuda.synchronize()
    assert torch.allclose(stats[api.STAT_MEAN_STEP], torch.ones(K, dtype=torch.float64, device="cuda"))


def _device_free_bytes():
    """Free device memory as the CUDA runtime reports it (cudaMemGetInfo through the runtime torch has loaded)."""
    free, _total = torch.cuda.mem_get_info()
    return free


def test_static_reduce_requests_no_device_memory(api):
    """Nothing observable is allocated by the call: the bytes torch's pool has handed out and has reserved, and the
    device's free memory, are the same before and after (the first call on the device has happened above or happens
    in the warm-up here, so the library image with its built-in array is already resident)."""
    step, done, sync = _sweep_outputs(api, 300, 20, 8, 64, seed=60)
    got = torch.empty((api.NSTATS, 64), dtype=torch.float64, device="cuda")
    got_base = torch.empty(2, dtype=torch.float64, device="cuda")
    import gc
    api.dc_reduce_trials_static(step, done, sync, 20, 8, got, got_base)      # warm-up
    torch.cuda.synchronize()
    gc.collect()                                                             # tensors of earlier tests go now, not mid-measurement
    before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), _device_free_bytes())
    for _ in range(3):
        api.dc_reduce_trials_static(step, done, sync, 20, 8, got, got_base)
    torch.cuda.synchronize()
    after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), _device_free_bytes())
    assert after[0] <= before[0], (before, after)          # nothing new handed out by torch's pool
    assert after[1:] == before[1:], (before, after)        # the pool did not grow, the device's free memory did not move


def test_static_reduce_at_the_top_of_its_scratch(api):
    """The largest supported grid with enough trials to use every chunk of partial sums (64 chunks x (4 K + 1)
    doubles = the whole built-in array).  Both entry points launch the same kernels in the same order, so the bits
    must be equal, not just close; repeated after a smaller call has left other contents in the array."""
    K, N, M = api.STATIC_MAX_K, 3, 5
    g = torch.Generator(device="cuda").manual_seed(7)
    for T in (2560, 40, 2560):
        step = torch.rand((T, K), device="cuda", generator=g) + 0.5
        done = torch.randint(0, N * M + 1, (T, K), device="cuda", generator=g, dtype=torch.int32)
        sync = step.max(dim=1).values + 0.25
        want = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
        want_base = torch.empty(2, dtype=torch.float64, device="cuda")
        ws = torch.empty(api.dc_reduce_workspace_bytes(T, K), dtype=torch.uint8, device="cuda")
        assert T < 2048 or ws.numel() == 64 * (4 * K + 1) * 8     # every chunk in use
        api.dc_reduce_trials(step, done, sync, N, M, want, want_base, ws)
        got = torch.full_like(want, float("nan"))
        got_base = torch.full_like(want_base, float("nan"))
        api.dc_reduce_trials_static(step, done, sync, N, M, got, got_base)
        torch.cuda.synchronize()
        assert torch.equal(got, want) and torch.equal(got_base, want_base), T
        ref = oracle.reduce_trials(step.cpu().numpy(), done.cpu().numpy(), sync.cpu().numpy(), N, M)
        assert np.allclose(got.cpu().numpy(), ref.stats, rtol=RTOL_STATS, atol=0)
