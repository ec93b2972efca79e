"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on seeded
inputs.  Integers and step times must match bit for bit; fp64 statistics within 1e-9 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_2306_10598_b200 import workloads as W

pytestmark = pytest.mark.gpu

RTOL_STATS = 1e-9   # fp64 sums of <= 2^15 terms taken in a different order: far below this
INF = float("inf")


@pytest.fixture(scope="module")
def api():
    from paper_2306_10598_b200 import build
    build.build_library()   # compiles the library in-tree if it is missing or older than its sources
    from paper_2306_10598_b200 import api as _api
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return _api


def grid_for(lat: np.ndarray, K: int, seed: int) -> np.ndarray:
    """A sorted grid spanning below the smallest and above the largest worker time, with a repeated
    value, an exact worker total (a tie) and +inf at the end when K allows."""
    rng = np.random.default_rng(seed)
    tot = np.cumsum(lat, axis=-1, dtype=np.float32)
    hi = float(tot[..., -1].max())
    g = rng.uniform(-0.05 * hi, 1.15 * hi, K).astype(np.float32)
    if K >= 4:
        g[0] = tot.reshape(-1)[rng.integers(tot.size)]      # equals some running sum exactly
        g[1] = g[2]                                          # duplicate
        g[3] = np.float32(INF)
    g.sort()
    return g


def run_gpu(api, lat_d, taus_d, t_comm, rule=0, objective=4):
    r = api.sweep(lat_d, taus_d, t_comm, rule=rule, objective=objective)
    torch.cuda.synchronize()
    return r


def compare_sweep(res, ref, what=""):
    assert np.array_equal(res.out_done.cpu().numpy(), ref.done), f"out_done differs {what}"
    assert np.array_equal(res.out_step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32)), f"out_step differs {what}"
    assert np.array_equal(res.out_sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32)), f"out_sync differs {what}"


def compare_stats(res, ref_sweep, N, M, objective=4, what=""):
    st = oracle.reduce_trials(ref_sweep.step, ref_sweep.done, ref_sweep.sync, N, M)
    got = res.stats.cpu().numpy()
    assert np.allclose(got, st.stats, rtol=RTOL_STATS, atol=0, equal_nan=True), f"stats differ {what}"
    assert np.allclose(res.baseline.cpu().numpy(), st.baseline, rtol=RTOL_STATS, atol=0), f"baseline differs {what}"
    k_ref = oracle.argmax(st.stats[objective])
    assert int(res.k_star.item()) == k_ref, f"k* differs {what}"
    return st


EDGE_SHAPES = [
    # T, N, M, K                      what it exercises
    (1, 1, 1, 1),                    # everything degenerate (plain-load kernel)
    (3, 7, 1, 5),                    # M = 1
    (5, 1, 3, 4),                    # one worker, odd M
    (4, 33, 129, 17),                # odd M > 128, ragged warp
    (9, 8, 4, 16),                   # tiny's shape: 16-byte rows, no swizzle
    (7, 40, 8, 9),                   # 32-byte rows, 32-byte swizzle
    (6, 200, 12, 64),                # the paper's 12 accumulations: 48-byte rows, no swizzle
    (4, 100, 16, 33),                # 64-byte swizzle
    (3, 70, 20, 12), (3, 64, 24, 7), (2, 31, 28, 300),
    (5, 200, 32, 64),                # one 128-byte chunk, 200 rows in 7 warps
    (5, 300, 36, 40),                # two passes of 150 rows, ragged second column chunk
    (3, 9, 100, 50),                 # four column chunks, last one 16 bytes
    (3, 513, 64, 256),               # three passes of 171 rows
    (2, 2048, 128, 256),             # the stress shape: 8 passes x 4 chunks per trial
    (2, 256, 32, 4096),              # the largest grid
    (300, 5, 16, 3),                 # many short trials, more trials than blocks in flight
    (1, 1000, 8, 1),                 # one trial only
    # several whole trials of few workers share a tile (the last tile holds fewer trials than the others)
    (1000, 8, 4, 16), (1000, 8, 12, 16), (1000, 8, 32, 7), (333, 5, 4, 33), (333, 5, 12, 64), (333, 5, 32, 9),
    (77, 33, 4, 16), (77, 33, 12, 40), (77, 33, 32, 128), (50, 128, 4, 5), (50, 128, 12, 64), (50, 128, 32, 256),
    (5000, 3, 8, 20), (700, 1, 16, 4), (900, 100, 48, 64), (650, 64, 36, 30),
    # row lengths cut into equal chunks of 12, 16 or 24 floats (36, 48, 72, 80) and ones that are not (100, 56, 44, 88, 20, 28)
    (6, 300, 48, 40), (5, 256, 72, 64), (4, 150, 80, 33), (40, 260, 36, 50), (7, 200, 100, 64), (5, 90, 56, 20),
    (6, 130, 44, 30), (3, 70, 88, 64), (9, 64, 20, 16), (9, 64, 28, 16),
]


@pytest.mark.parametrize("T,N,M,K", EDGE_SHAPES)
def test_edge_shapes_match_oracle(api, T, N, M, K):
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=100 + T + N + M, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, seed=K)
    t_comm = 0.0625 + 0.001
    ref = oracle.sweep(lat, taus, t_comm)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    res = run_gpu(api, lat_d, taus_d, t_comm)
    compare_sweep(res, ref, f"{(T, N, M, K)}")
    compare_stats(res, ref, N, M, what=f"{(T, N, M, K)}")
    # plain dc_simulate (no sync output) gives the same step/done
    step2 = torch.full_like(res.out_step, -1.0)
    done2 = torch.full_like(res.out_done, -1)
    api.dc_simulate(lat_d, taus_d, t_comm, step2, done2)
    torch.cuda.synchronize()
    assert torch.equal(step2, res.out_step) and torch.equal(done2, res.out_done)
    # a second call gives the same bits
    res2 = run_gpu(api, lat_d, taus_d, t_comm)
    for a, b in zip(res, res2):
        assert torch.equal(a.reshape(-1).view(torch.uint8), b.reshape(-1).view(torch.uint8))
    api.dc_device_status()


@pytest.mark.parametrize("T,N,M,K", [(4, 50, 16, 11), (3, 300, 36, 40), (5, 7, 5, 9), (2, 600, 126, 64), (1, 1, 1, 3),
                                      (6, 33, 255, 20), (3, 20, 300, 16), (2, 9, 1030, 8)])
def test_base_pointer_only_4_byte_aligned(api, T, N, M, K):
    """Latency tensors that start 1, 2 or 3 floats past a 16-byte boundary (views into a larger buffer): rows of up
    to 255 samples take the flat kernel, whose bulk copies begin at the first and end at the last 16-byte boundary
    inside the tensor with the few floats outside moved by ordinary loads; longer rows take the plain-load kernel.
    Guard values around the view must not change anything."""
    lat = W.iid_latencies("uniform", T, N, M, seed=5 + M, lo=0.0, hi=0.1).numpy()
    taus = grid_for(lat, K, 3)
    taus_d = torch.from_numpy(taus).cuda()
    for rule in (0, 1):
        ref = oracle.sweep(lat, taus, 0.3, rule=rule)
        for shift in (1, 2, 3):
            buf = torch.full((T * N * M + shift + 5,), float("nan"), dtype=torch.float32, device="cuda")
            view = buf[shift:shift + T * N * M].view(T, N, M)
            view.copy_(torch.from_numpy(lat))
            assert api.dc_simulate_plan(view, K) == (2 if M <= 127 else 1)
            res = run_gpu(api, view, taus_d, 0.3, rule=rule)
            compare_sweep(res, ref, f"(shift {shift}, rule {rule})")
    assert api.dc_simulate_plan(torch.from_numpy(lat).cuda(), K) == (0 if M % 4 == 0 else (2 if M <= 127 else 1))
    api.dc_device_status()


@pytest.mark.parametrize("rule", [0, 1])
@pytest.mark.parametrize("T,N,M,K", [(5, 200, 32, 64), (3, 300, 36, 132), (4, 77, 10, 256)])
def test_outputs_only_4_byte_aligned(api, T, N, M, K, rule):
    # Output rows that start on 16-byte boundaries are written four thresholds at a time; outputs that are only
    # 4-byte aligned (views one element into a buffer) take the one-threshold-per-lane path.  Both must give the
    # oracle's bits.
    lat = W.iid_latencies("uniform", T, N, M, seed=21 + K, lo=0.0, hi=0.05).numpy()
    taus = grid_for(lat, K, 7)
    ref = oracle.sweep(lat, taus, 0.2, rule=rule)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    for shift in (0, 1):
        step = torch.full((T * K + shift,), -1.0, dtype=torch.float32, device="cuda")
        done = torch.full((T * K + shift,), -1, dtype=torch.int32, device="cuda")
        sync = torch.empty(T, dtype=torch.float32, device="cuda")
        api.dc_simulate_ex(lat_d, taus_d, 0.2, step[shift:].view(T, K), done[shift:].view(T, K), sync, rule)
        torch.cuda.synchronize()
        assert np.array_equal(done[shift:].view(T, K).cpu().numpy(), ref.done), f"out_done differs (shift {shift})"
        assert np.array_equal(step[shift:].view(T, K).cpu().numpy().view(np.uint32), ref.step.view(np.uint32)), \
            f"out_step differs (shift {shift})"
        assert np.array_equal(sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32))
        if shift:
            assert float(step[0]) == -1.0 and int(done[0]) == -1   # nothing written before the view
    api.dc_device_status()


def test_zero_and_tie_latencies(api):
    # dyadic values: many running sums coincide with thresholds exactly, zeros repeat a running sum
    T, N, M, K = 6, 37, 24, 40
    lat = W.iid_latencies("dyadic", T, N, M, seed=6, hi=8).numpy()
    lat[:, ::3, ::2] = 0.0
    taus = (np.arange(K, dtype=np.float32) / 16.0)
    ref = oracle.sweep(lat, taus, 0.25)
    res = run_gpu(api, torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda(), 0.25)
    compare_sweep(res, ref)
    compare_stats(res, ref, N, M)


@pytest.mark.parametrize("rule", [0, 1])
def test_subnormal_and_huge_latencies(api, rule):
    """Both sides add in IEEE binary32 without flushing: latencies and thresholds in the subnormal range, and
    latencies near the top of the range (row sums up to 3.2e38, still finite as the interface requires)."""
    rng = np.random.default_rng(3)
    T, N, M, K = 3, 40, 16, 24
    tiny = (rng.integers(0, 2000, (T, N, M)).astype(np.float64) * 1e-42).astype(np.float32)     # multiples of ~1e-42
    taus = np.sort((rng.integers(0, 20000, K).astype(np.float64) * 1e-42).astype(np.float32))
    assert tiny.max() < np.finfo(np.float32).tiny and tiny.max() > 0
    ref = oracle.sweep(tiny, taus, 0.0, rule=rule)
    res = run_gpu(api, torch.from_numpy(tiny).cuda(), torch.from_numpy(taus).cuda(), 0.0, rule=rule)
    compare_sweep(res, ref, "(subnormal)")
    assert ref.done.max() > 0 and ref.done.min() < N * M          # the grid really cuts through the data
    huge = rng.uniform(1e37, 2e37, (T, N, M)).astype(np.float32)
    taus = np.array([1e37, 1e38, 2e38, 3e38, 3.3e38, np.inf], np.float32)
    ref = oracle.sweep(huge, taus, 1e30, rule=rule)
    assert np.isfinite(ref.sync).all()
    res = run_gpu(api, torch.from_numpy(huge).cuda(), torch.from_numpy(taus).cuda(), 1e30, rule=rule)
    compare_sweep(res, ref, "(huge)")


def test_thresholds_outside_the_data(api):
    T, N, M = 5, 20, 8
    lat = W.iid_latencies("uniform", T, N, M, seed=7, lo=0.01, hi=0.02).numpy()
    for taus in ([-1.0, 0.0], [0.0], [INF], [-INF, INF], [1e30, INF, INF], [0.05] * 7):
        taus = np.array(taus, np.float32)
        ref = oracle.sweep(lat, taus, 0.5)
        res = run_gpu(api, torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda(), 0.5)
        compare_sweep(res, ref, str(taus))


def test_objectives(api):
    T, N, M, K = 64, 30, 12, 25
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=8, shift=0.02, mean=0.03).numpy()
    taus = np.linspace(0.3, 1.2, K).astype(np.float32)
    ref = oracle.sweep(lat, taus, 0.1)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    for obj in (api.STAT_S_EFF, api.STAT_THR, api.STAT_THR_MEAN):
        res = run_gpu(api, lat_d, taus_d, 0.1, objective=obj)
        st = compare_stats(res, ref, N, M, objective=obj)
        k = int(res.k_star.item())
        assert float(res.tau_star.item()) == float(taus[k])
        assert np.isclose(float(res.value.item()), st.stats[obj, k], rtol=RTOL_STATS)
    # without the synchronous baseline S_eff and the baseline are NaN, the rest unchanged
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty(2, dtype=torch.float64, device="cuda")
    ws = torch.empty(api.dc_reduce_workspace_bytes(T, K), dtype=torch.uint8, device="cuda")
    api.dc_reduce_trials(res.out_step, res.out_done, None, N, M, stats, base, ws)
    torch.cuda.synchronize()
    assert torch.isnan(stats[api.STAT_S_EFF]).all() and torch.isnan(base).all()
    assert torch.equal(stats[:4], res.stats[:4])


@pytest.mark.parametrize("rule,objective", [(0, 4), (1, 2), (0, 3)])
def test_sweep_device_equals_the_three_calls(api, rule, objective):
    """dc_sweep_device enqueues the same three steps: every output must carry the same bits as the separate calls,
    and errors any of the steps would raise are raised before anything runs."""
    T, N, M, K = 37, 300, 36, 40
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=77, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, 4)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    ref = run_gpu(api, lat_d, taus_d, 0.15, rule=rule, objective=objective)
    step = torch.empty((T, K), dtype=torch.float32, device="cuda")
    done = torch.empty((T, K), dtype=torch.int32, device="cuda")
    sync = torch.empty((T,), dtype=torch.float32, device="cuda")
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty((2,), dtype=torch.float64, device="cuda")
    k = torch.empty((), dtype=torch.int32, device="cuda")
    tau = torch.empty((), dtype=torch.float32, device="cuda")
    val = torch.empty((), dtype=torch.float64, device="cuda")
    ws = torch.empty((api.dc_reduce_workspace_bytes(T, K),), dtype=torch.uint8, device="cuda")
    api.dc_sweep_device(lat_d, taus_d, 0.15, rule, objective, step, done, sync, stats, base, k, tau, val, ws)
    torch.cuda.synchronize()
    for a, b in zip((step, done, sync, stats, base, k, tau, val), ref):
        assert torch.equal(a.reshape(-1).view(torch.uint8), b.reshape(-1).view(torch.uint8))
    sw = oracle.sweep(lat, taus, 0.15, rule=rule)
    assert np.array_equal(done.cpu().numpy(), sw.done)
    with pytest.raises(api.DropComputeError) as e:   # unknown objective: refused before the sweep is enqueued
        api.dc_sweep_device(lat_d, taus_d, 0.15, rule, 0, step, done, sync, stats, base, k, tau, val, ws)
    assert e.value.status == 7
    with pytest.raises(api.DropComputeError) as e:   # workspace too small
        api.dc_sweep_device(lat_d, taus_d, 0.15, rule, objective, step, done, sync, stats, base, k, tau, val, ws[:8])
    assert e.value.status == 9
    api.dc_device_status()


@pytest.mark.parametrize("T,N,M,K,rule", [(64, 8, 4, 16, 0), (40, 200, 32, 64, 1), (9, 300, 30, 33, 0), (3, 70, 301, 20, 1)])
def test_device_path_in_a_cuda_graph(api, T, N, M, K, rule):
    """The device-resident path neither allocates nor synchronises, so a stream capture can record it (after one
    ordinary call, which sets the kernels' attributes) and a replay must reproduce every output bit: tiled, flat
    and plain-load kernels."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=55 + M, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, 8)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    step = torch.empty((T, K), dtype=torch.float32, device="cuda")
    done = torch.empty((T, K), dtype=torch.int32, device="cuda")
    sync = torch.empty((T,), dtype=torch.float32, device="cuda")
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty((2,), dtype=torch.float64, device="cuda")
    k = torch.empty((), dtype=torch.int32, device="cuda")
    tau = torch.empty((), dtype=torch.float32, device="cuda")
    val = torch.empty((), dtype=torch.float64, device="cuda")
    ws = torch.empty((api.dc_reduce_workspace_bytes(T, K),), dtype=torch.uint8, device="cuda")
    outs = (step, done, sync, stats, base, k, tau, val)

    def call():
        api.dc_sweep_device(lat_d, taus_d, 0.2, rule, 4, step, done, sync, stats, base, k, tau, val, ws)

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        call()
        torch.cuda.synchronize()
        want = [o.clone() for o in outs]
        with torch.cuda.graph(graph, stream=side):
            call()
    for _ in range(2):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for o, w_ in zip(outs, want):
            assert torch.equal(o.reshape(-1).view(torch.uint8), w_.reshape(-1).view(torch.uint8))
    ref = oracle.sweep(lat, taus, 0.2, rule=rule)
    assert np.array_equal(done.cpu().numpy(), ref.done)
    assert np.array_equal(step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32))
    api.dc_device_status()


def test_check_inputs(api):
    lat = torch.rand(4, 5, 6, device="cuda")
    taus = torch.tensor([0.1, 0.2, 0.2, INF], device="cuda")
    api.dc_check_inputs(lat, taus)
    bad = lat.clone()
    bad[1, 2, 3] = -0.5
    with pytest.raises(api.DropComputeError) as e:
        api.dc_check_inputs(bad, taus)
    assert e.value.status == 8
    bad[1, 2, 3] = float("nan")
    with pytest.raises(api.DropComputeError):
        api.dc_check_inputs(bad, taus)
    over = lat.clone()
    over[2, 1, :] = 1e38                       # every value is fine, their sum is not
    with pytest.raises(api.DropComputeError) as e:
        api.dc_check_inputs(over, taus)
    assert e.value.status == 8
    over[2, 1, 3:] = 0.0                       # 3e38: finite again
    api.dc_check_inputs(over, taus)
    with pytest.raises(api.DropComputeError) as e:
        api.dc_check_inputs(lat, torch.tensor([0.3, 0.2], device="cuda"))
    assert e.value.status == 5
    with pytest.raises(api.DropComputeError):
        api.dc_check_inputs(lat, torch.tensor([0.3, float("nan")], device="cuda"))
    with pytest.raises(TypeError):
        api.dc_simulate(lat.double(), taus, 0.1, torch.empty(4, 4, device="cuda"),
                        torch.empty(4, 4, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("M,rule,objective", [(16, 0, 4), (16, 1, 2), (10, 0, 3), (7, 1, 4)])
def test_sweep_host_matches_oracle(api, M, rule, objective):
    """The host-memory entry point (chunked copies overlapped with the kernels), for both rules, every
    objective, and rows that take the tiled or the flat kernel; pageable host memory works too."""
    T, N, K = 37, 64, 20
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=9, shift=0.02, mean=0.01)
    taus = np.linspace(0.02 * M, 0.045 * M, K).astype(np.float32)
    ref = oracle.sweep(lat.numpy(), taus, 0.1, rule=rule)
    st = oracle.reduce_trials(ref.step, ref.done, ref.sync, N, M)
    for chunk, pinned in ((5, True), (37, True), (100, False)):
        ws = torch.empty(api.dc_sweep_host_workspace_bytes(T, N, M, K, chunk) + 1024, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 1024
        hs = api.dc_sweep_host(lat.pin_memory() if pinned else lat, torch.from_numpy(taus), 0.1, ws[off:], chunk,
                               rule=rule, objective=objective)
        assert np.allclose(hs.stats.numpy(), st.stats, rtol=RTOL_STATS, atol=0)
        assert np.allclose(hs.baseline.numpy(), st.baseline, rtol=RTOL_STATS, atol=0)
        assert hs.k_star == oracle.argmax(st.stats[objective]) and hs.tau_star == float(taus[hs.k_star])


# ---- the five benchmark workloads ---------------------------------------------------------------

def _full_parity(api, w):
    lat_d = W.fill_latencies(w, "cuda")
    taus = W.make_taus(w)
    res = run_gpu(api, lat_d, torch.from_numpy(taus).cuda(), w.t_comm)
    ref = oracle.sweep(lat_d.cpu().numpy(), taus, w.t_comm)
    compare_sweep(res, ref, w.name)
    compare_stats(res, ref, w.N, w.M, what=w.name)
    api.dc_device_status()


def test_workload_tiny(api):
    _full_parity(api, W.WORKLOADS["tiny"])


def test_workload_paper_scale(api):
    _full_parity(api, W.WORKLOADS["paper_scale"])


def test_workload_extrapolation(api):
    _full_parity(api, W.WORKLOADS["extrapolation"])


def _full_size_parity(api, w):
    """Full-size run in the benchmark's launch configuration, compared with the oracle on EVERY trial: the device
    tensor comes back in chunks of whole trials through one pinned buffer, the oracle sweeps each chunk, and
    every out_done / out_step / out_sync is compared bit for bit; the [K] statistics of the whole run are then
    compared at 1e-9 with the oracle's reduction of its own [T,K] outputs."""
    free, _ = torch.cuda.mem_get_info()
    if free < w.latency_bytes + (4 << 30):
        pytest.skip(f"needs {w.latency_bytes / 2**30:.1f} GiB of device memory")
    lat_d = W.fill_latencies(w, "cuda")
    taus = W.make_taus(w)
    taus_d = torch.from_numpy(taus).cuda()
    res = run_gpu(api, lat_d, taus_d, w.t_comm)
    got_done = res.out_done.cpu().numpy()
    got_step = res.out_step.cpu().numpy().view(np.uint32)
    got_sync = res.out_sync.cpu().numpy().view(np.uint32)
    ct = max(1, (1 << 30) // (4 * w.N * w.M))                 # 1 GiB of latencies per chunk
    stage = torch.empty((ct, w.N, w.M), dtype=torch.float32, pin_memory=True)
    ref_step = np.empty((w.T, w.K), np.float32)
    ref_done = np.empty((w.T, w.K), np.int32)
    ref_sync = np.empty((w.T,), np.float32)
    for t0 in range(0, w.T, ct):
        t1 = min(w.T, t0 + ct)
        stage[:t1 - t0].copy_(lat_d[t0:t1])
        torch.cuda.synchronize()
        ref = oracle.sweep(stage[:t1 - t0].numpy(), taus, w.t_comm)
        ref_step[t0:t1], ref_done[t0:t1], ref_sync[t0:t1] = ref.step, ref.done, ref.sync
        assert np.array_equal(got_done[t0:t1], ref.done), f"out_done differs in trials {t0}:{t1} of {w.name}"
        assert np.array_equal(got_step[t0:t1], ref.step.view(np.uint32)), f"out_step differs in trials {t0}:{t1} of {w.name}"
        assert np.array_equal(got_sync[t0:t1], ref.sync.view(np.uint32)), f"out_sync differs in trials {t0}:{t1} of {w.name}"
    del stage
    compare_stats(res, oracle.Sweep(ref_step, ref_done, ref_sync), w.N, w.M, what=w.name)
    # properties that hold at any size, on every output
    done, step, sync = res.out_done, res.out_step, res.out_sync
    assert bool((done[:, 1:] >= done[:, :-1]).all()) and bool((step[:, 1:] >= step[:, :-1]).all())
    assert int(done.min()) >= 0 and int(done.max()) <= w.N * w.M
    tc = torch.tensor(w.t_comm, dtype=torch.float32, device="cuda")
    assert bool((step <= (taus_d[None, :] + tc)).all()) and bool((step <= sync[:, None]).all())
    full = taus_d[None, :] > (sync[:, None] - tc) * 1.001       # thresholds clearly above the slowest worker
    assert bool((done[full] == w.N * w.M).all())
    api.dc_device_status()


def test_workload_correlated_every_trial(api):
    _full_size_parity(api, W.WORKLOADS["correlated"])


def test_workload_bandwidth_stress_every_trial(api):
    _full_size_parity(api, W.WORKLOADS["bandwidth_stress"])


def test_results_do_not_depend_on_tuning_or_timing(api):
    """The ring depth and the number of histogram copies change the timing of the pipeline (how soon a
    stage is refilled, how long shared-memory atomics queue up) but must never change a bit of the result.
    Runs the stress shape (where a stage released too early would be overwritten while still being read)
    several times under every setting."""
    w = W.WORKLOADS["bandwidth_stress"].with_trials(1536)
    lat_d = W.fill_latencies(w, "cuda")
    taus = W.make_taus(w)
    taus_d = torch.from_numpy(taus).cuda()
    idx = np.arange(0, w.T, 64)
    ref = oracle.sweep(lat_d[torch.from_numpy(idx).cuda()].cpu().numpy(), taus, w.t_comm)
    first = None
    try:
        for stages, copies in ((0, 0), (4, 1), (2, 1), (2, 2), (3, 1), (2, 4)):
            api.dc_tune(api.TUNE_STAGES, stages)
            api.dc_tune(api.TUNE_LANE_COPIES, copies)
            for _ in range(4):
                res = run_gpu(api, lat_d, taus_d, w.t_comm)
                if first is None:
                    first = res
                    assert np.array_equal(res.out_done[idx].cpu().numpy(), ref.done)
                    assert np.array_equal(res.out_step[idx].cpu().numpy().view(np.uint32), ref.step.view(np.uint32))
                    assert np.array_equal(res.out_sync[idx].cpu().numpy().view(np.uint32), ref.sync.view(np.uint32))
                else:
                    assert torch.equal(res.out_done, first.out_done), (stages, copies)
                    assert torch.equal(res.out_step, first.out_step), (stages, copies)
                    assert torch.equal(res.out_sync, first.out_sync), (stages, copies)
    finally:
        api.dc_tune(api.TUNE_STAGES, 0)
        api.dc_tune(api.TUNE_LANE_COPIES, 0)
    api.dc_device_status()


@pytest.mark.parametrize("rule", [0, 1])
@pytest.mark.parametrize("T,N,M,K,cap", [(23, 200, 32, 64, 8), (7, 200, 12, 64, 8), (41, 129, 16, 16, 8), (12, 255, 8, 128, 8),
                                         (9, 150, 100, 64, 8), (10, 200, 20, 100, 8), (16, 170, 36, 256, 8), (5, 200, 64, 64, 2),
                                         (3, 131, 4, 8, 5), (2000, 200, 16, 64, 8)])
def test_packed_tiles_match_oracle(api, T, N, M, K, cap, rule):
    """Trials of 129-255 workers may be taken several at a time as one run of consecutive rows cut into equal passes
    (a trial then starts in the middle of a pass and a thread's rows in different passes belong to different trials).
    Small inputs never get that layout by themselves, so it is asked for through the tile-trials setting; the results
    must be the oracle's bits, on evenly spaced and on irregular grids, whole and ragged last tiles, both loops."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=900 + N + M, shift=0.01, mean=0.02).numpy()
    mean = M * 0.03
    grids = [grid_for(lat, K, seed=K + N), np.linspace(0.7 * mean, 1.3 * mean, K, dtype=np.float64).astype(np.float32)]
    lat_d = torch.from_numpy(lat).cuda()
    try:
        api.dc_tune(api.TUNE_TILE_TRIALS, cap)
        for taus in grids:
            ref = oracle.sweep(lat, taus, 0.05, rule=rule)
            res = run_gpu(api, lat_d, torch.from_numpy(taus).cuda(), 0.05, rule=rule)
            compare_sweep(res, ref, f"packed T={T} N={N} M={M} K={K}")
    finally:
        api.dc_tune(api.TUNE_TILE_TRIALS, 0)
    api.dc_device_status()


@pytest.mark.parametrize("rule", [0, 1])
def test_direct_and_table_binning_agree_with_oracle(api, rule):
    """Evenly spaced grids are binned arithmetically, every other grid through the lookup table; both must
    give the oracle's bits.  Grids: exact dyadic steps with samples ON the thresholds, float32 linspace grids
    of awkward ranges, a single threshold, a two-point grid, and a nearly even grid (falls back to the table)."""
    rng = np.random.default_rng(11)
    cases = []
    lat = W.iid_latencies("dyadic", 5, 70, 24, seed=31, hi=8).numpy()
    cases.append((lat, np.arange(48, dtype=np.float32) / 16.0))
    lat = W.iid_latencies("uniform", 4, 300, 36, seed=32, lo=0.0, hi=0.05).numpy()
    cases.append((lat, np.linspace(0.3, 1.1, 129).astype(np.float32)))
    cases.append((lat, np.linspace(0.9, 0.9000305, 64).astype(np.float32)))   # steps of a few ulps
    cases.append((lat, np.linspace(-0.2, 3.0, 7).astype(np.float32)))
    cases.append((lat, np.array([0.7], np.float32)))
    cases.append((lat, np.array([0.5, 0.9], np.float32)))
    g = np.linspace(0.3, 1.1, 200)
    g[1:-1] += rng.uniform(-0.4, 0.4, 198) * (g[1] - g[0])                      # uneven: table
    cases.append((lat, np.sort(g).astype(np.float32)))
    lat = W.iid_latencies("uniform", 3, 2048, 128, seed=33, lo=0.0, hi=0.014).numpy()
    cases.append((lat, np.linspace(0.6 * 0.896, 1.4 * 0.896, 256).astype(np.float32)))
    try:
        for lat, taus in cases:
            ref = oracle.sweep(lat, taus, 0.1, rule=rule)
            lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
            for mode in (1, 2):
                api.dc_tune(api.TUNE_DIRECT_BINS, mode)
                res = run_gpu(api, lat_d, taus_d, 0.1, rule=rule)
                compare_sweep(res, ref, f"(K={len(taus)}, direct bins {'on' if mode == 2 else 'off'})")
    finally:
        api.dc_tune(api.TUNE_DIRECT_BINS, 0)
    api.dc_device_status()


# ---- the start-before-tau rule (timeout looked at between accumulations) ---------------------------

@pytest.mark.parametrize("T,N,M,K", EDGE_SHAPES)
def test_start_before_tau_rule_matches_oracle(api, T, N, M, K):
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=300 + T + N + M, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, seed=K + 1)
    t_comm = 0.0625 + 0.001
    # small shapes are compared with the oracle form that reads a worker's time off the table of finish times
    # (the finish time of the LAST micro-batch it ran), the large ones with the one-pass form
    ref = oracle.sweep(lat, taus, t_comm, rule=1, order="definition" if T * N * M * K < 10 ** 8 else "rows")
    res = run_gpu(api, torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda(), t_comm, rule=1)
    compare_sweep(res, ref, f"rule 1 {(T, N, M, K)}")
    compare_stats(res, ref, N, M, what=f"rule 1 {(T, N, M, K)}")
    api.dc_device_status()


def test_start_before_tau_rule_special_grids(api):
    T, N, M = 6, 37, 24
    lat = W.iid_latencies("dyadic", T, N, M, seed=16, hi=8).numpy()
    lat[:, ::3, ::2] = 0.0
    for taus in (np.arange(40, dtype=np.float32) / 16.0, [-1.0, 0.0], [0.0], [INF], [-INF, INF], [1e30, INF, INF],
                 [0.5] * 7, [-2.0, -1.0, 0.0, 0.125, 0.125, 3.0, INF]):
        taus = np.array(taus, np.float32)
        ref = oracle.sweep(lat, taus, 0.25, rule=1, order="definition")
        res = run_gpu(api, torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda(), 0.25, rule=1)
        compare_sweep(res, ref, f"rule 1 {taus[:4]}")


@pytest.mark.parametrize("name,trials", [("tiny", 1024), ("paper_scale", 2048), ("extrapolation", 256),
                                         ("correlated", 48), ("bandwidth_stress", 48)])
def test_start_before_tau_rule_on_workloads(api, name, trials):
    w = W.WORKLOADS[name].with_trials(trials)
    lat_d = W.fill_latencies(w, "cuda")
    taus = W.make_taus(w)
    res = run_gpu(api, lat_d, torch.from_numpy(taus).cuda(), w.t_comm, rule=1)
    ref = oracle.sweep(lat_d.cpu().numpy(), taus, w.t_comm, rule=1)
    compare_sweep(res, ref, f"rule 1 {name}")
    compare_stats(res, ref, w.N, w.M, what=f"rule 1 {name}")
    # the two rules are tied together: a worker starts at most one micro-batch more than it finishes in time
    res0 = run_gpu(api, lat_d, torch.from_numpy(taus).cuda(), w.t_comm, rule=0)
    assert bool((res.out_done >= res0.out_done).all()) and bool((res.out_done <= res0.out_done + w.N).all())
    assert bool((res.out_step >= res0.out_step).all())
    api.dc_device_status()


@pytest.mark.parametrize("rule", [0, 1])
@pytest.mark.parametrize("T,N,M,K", [(9, 8, 4, 16), (5, 300, 36, 40), (4, 33, 129, 17), (40, 200, 12, 64)])
def test_per_trial_communication_time(api, T, N, M, K, rule):
    """Algorithm 2's T_i^c: one communication time per trial."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=400 + T, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, seed=K + 2)
    tc = np.random.default_rng(T).uniform(0.01, 0.3, T).astype(np.float32)
    ref = oracle.sweep(lat, taus, tc, rule=rule)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    step = torch.empty((T, K), dtype=torch.float32, device="cuda")
    done = torch.empty((T, K), dtype=torch.int32, device="cuda")
    sync = torch.empty((T,), dtype=torch.float32, device="cuda")
    api.dc_simulate_tc(lat_d, taus_d, torch.from_numpy(tc).cuda(), step, done, sync, rule)
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty(2, dtype=torch.float64, device="cuda")
    ws = torch.empty(api.dc_reduce_workspace_bytes(T, K), dtype=torch.uint8, device="cuda")
    api.dc_reduce_trials(step, done, sync, N, M, stats, base, ws)
    torch.cuda.synchronize()
    assert np.array_equal(done.cpu().numpy(), ref.done)
    assert np.array_equal(step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32))
    assert np.array_equal(sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32))
    st = oracle.reduce_trials(ref.step, ref.done, ref.sync, N, M)
    assert np.allclose(stats.cpu().numpy(), st.stats, rtol=RTOL_STATS, atol=0)
    assert np.allclose(base.cpu().numpy(), st.baseline, rtol=RTOL_STATS, atol=0)


def test_closed_form_matches_oracle(api):
    """App. C.2's estimates (Eq. 4/12, 5/10, 11) on the GPU against the oracle's, and the analytic tau*."""
    import math
    for mu, sd, M, N, tc in ((1.0, 0.1, 16, 400, 0.3), (0.675, math.sqrt(0.05), 12, 1000, 0.5), (0.03, 0.004, 64, 2, 0.0),
                             (0.007, 0.0014, 128, 2048, 0.1)):
        taus = np.linspace(0.4 * M * mu, 1.4 * M * mu, 257).astype(np.float32)
        taus_d = torch.from_numpy(taus).cuda()
        out = torch.empty((3, taus.size), dtype=torch.float64, device="cuda")
        sc = torch.empty(1, dtype=torch.float64, device="cuda")
        for mean_T in (-1.0, 1.07 * M * mu):
            ref = oracle.closed_form(mu, sd, M, N, tc, taus, mean_T=mean_T)
            api.dc_closed_form(mu, sd, M, N, tc, taus_d, out, sc, mean_T=mean_T)
            k = torch.empty((), dtype=torch.int32, device="cuda")
            tau_s = torch.empty((), dtype=torch.float32, device="cuda")
            val = torch.empty((), dtype=torch.float64, device="cuda")
            api.dc_argmax_tau(out, taus_d, 2, k, tau_s, val)           # row 2 of the [3,K] matrix
            torch.cuda.synchronize()
            got = out.cpu().numpy()
            assert np.allclose(got[0], ref.done_frac, rtol=1e-9, atol=1e-300)
            assert np.allclose(got[1], ref.step, rtol=1e-12)
            assert np.allclose(got[2], ref.s_eff, rtol=1e-9, atol=1e-300)
            assert abs(float(sc.item()) - ref.mean_T) <= 1e-10 * abs(ref.mean_T)
            assert int(k.item()) == ref.k_star and float(tau_s.item()) == ref.tau_star


@pytest.mark.parametrize("noise", sorted(W.C3_NOISE) + ["b1_delay"])
def test_appendix_workloads_match_oracle(api, noise):
    """The paper's own synthetic settings (App. C.3: 12 accumulations of 0.45 s + eps for every noise law of its two
    tables; App. B.1: the bounded log-normal delay), 200 and 768 workers, both rules: bit for bit against the oracle,
    statistics at 1e-9.  (The normal law can draw a negative eps; the generator keeps latencies >= 0.)"""
    for N in (200, 768):
        w = W.b1_workload(N=N, T=64, K=64) if noise == "b1_delay" else W.c3_workload(noise, N=N, T=64, K=64)
        lat_d = W.fill_latencies(w, "cuda")
        assert float(lat_d.min()) >= 0.0
        taus = W.make_taus(w)
        taus_d = torch.from_numpy(taus).cuda()
        lat = lat_d.cpu().numpy()
        for rule in (0, 1):
            res = run_gpu(api, lat_d, taus_d, w.t_comm, rule=rule)
            ref = oracle.sweep(lat, taus, w.t_comm, rule=rule)
            compare_sweep(res, ref, f"{noise} N={N} rule {rule}")
            compare_stats(res, ref, w.N, w.M, what=f"{noise} N={N} rule {rule}")
    api.dc_device_status()


def test_scale_graph_rows(api):
    """The scale-graph helper: the printed E[T]/E[T_i] values are only a plausibility band (the worker count behind
    them is not printed), so the check on them is loose on purpose."""
    from paper_2306_10598_b200 import scale_graph
    row = scale_graph.scale_row("exponential_0.05", 768, 256, 64, 0.5)
    assert 1.25 < row["E[T]/E[T_i]"] < 1.55                   # paper prints 1.386 for this law
    small = scale_graph.scale_row("exponential_0.05", 8, 256, 64, 0.5)
    assert small["E[T]/E[T_i]"] < row["E[T]/E[T_i]"]           # grows with the number of workers (Sec. 4.2)
    assert row["s_eff"] >= 1.0 and 0.0 <= row["drop_rate"] < 0.5
    assert abs(row["s_eff_closed_form_given_E[T]"] - row["s_eff"]) < 0.1 * row["s_eff"]
    delay = scale_graph.scale_row("b1_delay", 200, 128, 64, 0.5)
    assert delay["E[T]/E[T_i]"] > 1.0 and delay["s_eff"] >= 1.0
    assert set(scale_graph.PAPER_RATIO) == set(W.C3_NOISE)


def test_random_shapes_and_grids(api):
    """Seeded sweep over random shapes, latency laws, grids, both rules and both communication-time forms:
    every tile geometry (16- to 128-byte rows, ragged last column chunk, several passes, plain-load kernel)
    against the oracle, bit for bit."""
    rng = np.random.default_rng(20260601)
    laws = [("shifted_exp", dict(shift=0.01, mean=0.02)), ("uniform", dict(lo=0.0, hi=0.05)), ("dyadic", dict(hi=12)),
            ("exp", dict(rate=30.0))]
    for case in range(70):
        T = int(rng.integers(1, 12))
        N = int(rng.choice([1, 2, 7, 31, 32, 33, 100, 255, 256, 257, 600]))
        M = int(rng.choice([1, 2, 3, 4, 8, 12, 16, 20, 24, 28, 32, 36, 44, 64, 68, 96, 100, 128, 132, 160]))
        K = int(rng.choice([1, 2, 3, 16, 31, 32, 33, 64, 100, 257, 1000]))
        law, prm = laws[int(rng.integers(len(laws)))]
        lat = W.iid_latencies(law, T, N, M, seed=1000 + case, **prm).numpy()
        kind = int(rng.integers(4))
        if kind == 0:
            taus = grid_for(lat, K, seed=case)
        elif kind == 1:                                   # evenly spaced, like the workloads
            tot = float(lat.sum(-1).mean())
            taus = np.linspace(0.5 * tot, 1.5 * tot + 1e-3, K).astype(np.float32)
        elif kind == 2:                                   # geometric: many thresholds share a table cell
            tot = float(lat.sum(-1).max()) + 1e-3
            taus = (tot * np.geomspace(1e-4, 2.0, K)).astype(np.float32)
        else:                                             # few distinct values, heavy duplication
            tot = float(lat.sum(-1).max()) + 1e-3
            taus = np.sort(rng.choice(np.linspace(0, tot, 5), K)).astype(np.float32)
        rule = int(rng.integers(2))
        lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
        step = torch.empty((T, K), dtype=torch.float32, device="cuda")
        done = torch.empty((T, K), dtype=torch.int32, device="cuda")
        sync = torch.empty((T,), dtype=torch.float32, device="cuda")
        if rng.integers(2):
            tc = rng.uniform(0.0, 0.2, T).astype(np.float32)
            api.dc_simulate_tc(lat_d, taus_d, torch.from_numpy(tc).cuda(), step, done, sync, rule)
        else:
            tc = float(np.float32(rng.uniform(0.0, 0.2)))
            api.dc_simulate_ex(lat_d, taus_d, tc, step, done, sync, rule)
        torch.cuda.synchronize()
        ref = oracle.sweep(lat, taus, tc, rule=rule)
        what = f"case {case}: T,N,M,K={T, N, M, K} law={law} grid={kind} rule={rule}"
        assert np.array_equal(done.cpu().numpy(), ref.done), what
        assert np.array_equal(step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32)), what
        assert np.array_equal(sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32)), what
    api.dc_device_status()


def test_flat_kernel_shapes(api):
    """Rows whose length is not a multiple of 4 (flat kernel: one bulk copy per tile, 4-byte shared loads):
    spans that start at every offset modulo 4, a tensor whose size is not a multiple of 4 (its last floats
    are moved by ordinary loads), several tiles per trial, the longest supported row, both rules, and repeated
    runs under different splits of the consumer warps (warps per tile, groups working on different tiles at
    once, ring stages per group), including more groups than a trial has tiles and trials that end mid-ring."""
    cases = [(7, 3, 5, 9), (5, 1, 1, 3), (3, 257, 30, 64), (6, 513, 6, 33), (4, 100, 255, 40), (9, 64, 33, 100),
             (11, 37, 10, 16), (2, 2048, 126, 256), (64, 200, 14, 64), (13, 300, 65, 48), (5, 1000, 127, 32),
             (2, 200, 255, 4096), (2, 300, 126, 3000)]   # the last two: ring and tables compete for shared memory
    splits = [(0, 0, 0), (1, 8, 1), (1, 4, 2), (2, 4, 1), (2, 2, 2), (1, 3, 2), (4, 2, 1), (1, 5, 1), (8, 1, 2)]
    try:
        api.dc_tune(api.TUNE_FLAT_MAX_M, 255)      # rows of 128-255 samples go to the plain-load kernel by default
        for (T, N, M, K) in cases:
            lat = W.iid_latencies("shifted_exp", T, N, M, seed=900 + T + N + M, shift=0.01, mean=0.02).numpy()
            taus = grid_for(lat, K, seed=K + 5)
            lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
            assert api.dc_simulate_plan(lat_d, K) == 2
            for rule in (0, 1):
                ref = oracle.sweep(lat, taus, 0.07, rule=rule)
                for (wt, groups, depth) in splits:
                    if wt and wt * 32 * M * 4 + 32 > 32768 * 3:
                        continue  # such a tile would not fit the shared memory of a block
                    api.dc_tune(api.TUNE_FLAT_TILE_WARPS, wt)
                    api.dc_tune(api.TUNE_FLAT_GROUPS, groups)
                    api.dc_tune(api.TUNE_FLAT_DEPTH, depth)
                    try:
                        res = run_gpu(api, lat_d, taus_d, 0.07, rule=rule)
                    except api.DropComputeError as e:
                        assert e.status == 4 and wt, (e.status, wt, groups, depth)   # a forced split that does not fit
                        continue
                    compare_sweep(res, ref, f"flat {(T, N, M, K)} rule {rule} split {(wt, groups, depth)}")
    finally:
        api.dc_tune(api.TUNE_FLAT_MAX_M, 0)
        api.dc_tune(api.TUNE_FLAT_TILE_WARPS, 0)
        api.dc_tune(api.TUNE_FLAT_GROUPS, 0)
        api.dc_tune(api.TUNE_FLAT_DEPTH, 0)
    api.dc_device_status()


@pytest.mark.parametrize("T,N,M,K", [(3, 600, 257, 64), (2, 300, 301, 17), (5, 33, 514, 256), (2, 1, 999, 5), (40, 7, 258, 1),
                                      (4, 300, 129, 40), (3, 100, 255, 33), (6, 64, 150, 16)])
def test_plain_kernel_shapes(api, T, N, M, K):
    """Rows longer than 127 samples whose length is not a multiple of 4 (plain-load kernel: a warp stages 32 x 32
    pieces of its rows through a tile of its own): several passes per trial, ragged last warp and last chunk, a
    single worker, both rules, dyadic latencies so that running sums land ON thresholds."""
    lat = W.iid_latencies("dyadic", T, N, M, seed=300 + M, hi=6).numpy()
    taus = grid_for(lat, K, seed=K + 2)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    assert api.dc_simulate_plan(lat_d, K) == 1
    for rule in (0, 1):
        ref = oracle.sweep(lat, taus, 0.125, rule=rule)
        res = run_gpu(api, lat_d, taus_d, 0.125, rule=rule)
        compare_sweep(res, ref, f"(rule {rule})")
        compare_stats(res, ref, N, M)
    api.dc_device_status()


@pytest.mark.parametrize("T,N,M,K", [(3, 100000, 4, 40), (200000, 8, 4, 16), (2, 40, 4096, 64), (2, 70, 1030, 33),
                                      (1, 300000, 1, 8), (50000, 1, 32, 5)])
def test_extreme_aspect_ratios(api, T, N, M, K):
    """Very many workers (hundreds of passes per trial), very many trials, very long rows (hundreds of column
    chunks; 1030 is not a multiple of 4 and too long for the flat kernel, so it takes the plain-load one)."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=7000 + K, shift=0.001, mean=0.002).numpy()
    taus = grid_for(lat, K, seed=K + 9)
    for rule in (0, 1):
        ref = oracle.sweep(lat, taus, 0.01, rule=rule)
        res = run_gpu(api, torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda(), 0.01, rule=rule)
        compare_sweep(res, ref, f"{(T, N, M, K)} rule {rule}")
        compare_stats(res, ref, N, M, what=f"{(T, N, M, K)} rule {rule}")
    api.dc_device_status()


@pytest.mark.parametrize("T,N,M,K", [(3, 4096, 32, 64), (1, 20000, 16, 40), (7, 1000, 12, 33), (2, 2048, 126, 50),
                                      (5, 1009, 8, 16), (400, 512, 8, 16), (4, 100, 8, 9)])
def test_split_entry_point_matches(api, T, N, M, K):
    """dc_simulate_split (few trials swept as groups of workers, then merged) gives the bits of dc_simulate_ex
    and of the oracle; with a prime N, few workers or many trials it falls back to the plain call."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=8000 + N, shift=0.005, mean=0.01).numpy()
    taus = grid_for(lat, K, seed=K + 11)
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    wbytes = api.dc_simulate_split_workspace_bytes(T, N, M, K)
    if N == 1009 or N == 100 or T == 400:
        assert wbytes == 0
    else:
        assert wbytes > 0
    ws = torch.empty(wbytes + 256, dtype=torch.uint8, device="cuda") if wbytes else None
    if ws is not None:
        ws = ws[(-ws.data_ptr()) % 256:]
    for rule in (0, 1):
        ref = oracle.sweep(lat, taus, 0.02, rule=rule)
        step = torch.empty((T, K), dtype=torch.float32, device="cuda")
        done = torch.empty((T, K), dtype=torch.int32, device="cuda")
        sync = torch.empty((T,), dtype=torch.float32, device="cuda")
        api.dc_simulate_split(lat_d, taus_d, 0.02, step, done, sync, ws, rule)
        torch.cuda.synchronize()
        assert np.array_equal(done.cpu().numpy(), ref.done), (rule, "done")
        assert np.array_equal(step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32)), (rule, "step")
        assert np.array_equal(sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32)), (rule, "sync")
    if wbytes:
        with pytest.raises(api.DropComputeError) as e:
            api.dc_simulate_split(lat_d, taus_d, 0.02, step, done, sync, None, 0)
        assert e.value.status == 9
    api.dc_device_status()


def test_two_host_threads_on_two_streams(api):
    """Two host threads, each with a stream of its own, sweep different inputs at the same time while the main
    thread keeps changing the expert settings: every result must carry the oracle's bits (the library keeps no
    per-call state and every call works from one consistent copy of the settings)."""
    import threading
    cases = [(40, 200, 32, 64, 0), (25, 300, 36, 40, 1)]
    inputs, refs = [], []
    for i, (T, N, M, K, rule) in enumerate(cases):
        lat = W.iid_latencies("shifted_exp", T, N, M, seed=1200 + i, shift=0.01, mean=0.02).numpy()
        taus = grid_for(lat, K, seed=50 + i)
        inputs.append((torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()))
        refs.append(oracle.sweep(lat, taus, 0.11, rule=rule))
    torch.cuda.synchronize()
    errors = []

    def worker(i):
        try:
            T, N, M, K, rule = cases[i]
            lat_d, taus_d = inputs[i]
            stream = torch.cuda.Stream()
            step = torch.empty((T, K), dtype=torch.float32, device="cuda")
            done = torch.empty((T, K), dtype=torch.int32, device="cuda")
            sync = torch.empty((T,), dtype=torch.float32, device="cuda")
            with torch.cuda.stream(stream):
                for _ in range(40):
                    step.fill_(-1.0)
                    done.fill_(-1)
                    api.dc_simulate_ex(lat_d, taus_d, 0.11, step, done, sync, rule)
                    stream.synchronize()
                    ok = (np.array_equal(done.cpu().numpy(), refs[i].done)
                          and np.array_equal(step.cpu().numpy().view(np.uint32), refs[i].step.view(np.uint32))
                          and np.array_equal(sync.cpu().numpy().view(np.uint32), refs[i].sync.view(np.uint32)))
                    if not ok:
                        errors.append((i, "bits differ"))
                        return
        except Exception as e:  # noqa: BLE001 - reported by the main thread
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(cases))]
    for t in threads:
        t.start()
    try:
        n = 0
        while any(t.is_alive() for t in threads):
            api.dc_tune(api.TUNE_STAGES, (0, 2, 3)[n % 3])
            api.dc_tune(api.TUNE_LANE_COPIES, (0, 1, 2, 4)[n % 4])
            api.dc_tune(api.TUNE_DIRECT_BINS, n % 3)
            n += 1
    finally:
        for t in threads:
            t.join()
        api.dc_tune(api.TUNE_STAGES, 0)
        api.dc_tune(api.TUNE_LANE_COPIES, 0)
        api.dc_tune(api.TUNE_DIRECT_BINS, 0)
    assert not errors, errors
    api.dc_device_status()


@pytest.mark.parametrize("rule", [0, 1])
@pytest.mark.parametrize("T,N,M,K", [(9, 8, 4, 16), (5, 300, 36, 40), (4, 33, 129, 17), (40, 200, 12, 64), (3, 1000, 7, 300),
                                      (6, 1, 5, 3), (2, 70, 16, 4096)])
def test_heterogeneous_workers_match_oracle(api, T, N, M, K, rule):
    """dc_simulate_scaled: worker n against its own thresholds s_n tau_k (App. C.2: workers need not be identical), both
    rules, grids with negative, repeated and infinite thresholds; with all scales one it must give dc_simulate_ex's bits."""
    lat = W.iid_latencies("shifted_exp", T, N, M, seed=600 + T + N, shift=0.01, mean=0.02).numpy()
    taus = grid_for(lat, K, seed=K + 21)
    rng = np.random.default_rng(N + M)
    scale = rng.uniform(0.6, 1.6, N).astype(np.float32)
    scale[rng.integers(N)] = 1.0
    lat_d, taus_d = torch.from_numpy(lat).cuda(), torch.from_numpy(taus).cuda()
    step = torch.empty((T, K), dtype=torch.float32, device="cuda")
    done = torch.empty((T, K), dtype=torch.int32, device="cuda")
    sync = torch.empty((T,), dtype=torch.float32, device="cuda")
    for sc in (scale, np.ones(N, np.float32)):
        ref = oracle.sweep(lat, taus, 0.07, rule=rule, worker_scale=sc,
                           order="definition" if T * N * M * K < 10 ** 7 else "rows")
        step.fill_(-1.0)
        done.fill_(-1)
        api.dc_simulate_scaled(lat_d, taus_d, torch.from_numpy(sc).cuda(), 0.07, step, done, sync, rule)
        torch.cuda.synchronize()
        assert np.array_equal(done.cpu().numpy(), ref.done), "out_done differs"
        assert np.array_equal(step.cpu().numpy().view(np.uint32), ref.step.view(np.uint32)), "out_step differs"
        assert np.array_equal(sync.cpu().numpy().view(np.uint32), ref.sync.view(np.uint32)), "out_sync differs"
    same = run_gpu(api, lat_d, taus_d, 0.07, rule=rule)          # all scales one == the common-threshold entry point
    assert torch.equal(done, same.out_done) and torch.equal(step, same.out_step) and torch.equal(sync, same.out_sync)
    # the statistics and tau* follow from the per-trial outputs as always
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device="cuda")
    base = torch.empty(2, dtype=torch.float64, device="cuda")
    ws = torch.empty(api.dc_reduce_workspace_bytes(T, K), dtype=torch.uint8, device="cuda")
    api.dc_simulate_scaled(lat_d, taus_d, torch.from_numpy(scale).cuda(), 0.07, step, done, sync, rule)
    api.dc_reduce_trials(step, done, sync, N, M, stats, base, ws)
    torch.cuda.synchronize()
    ref = oracle.sweep(lat, taus, 0.07, rule=rule, worker_scale=scale)
    st = oracle.reduce_trials(ref.step, ref.done, ref.sync, N, M)
    assert np.allclose(stats.cpu().numpy(), st.stats, rtol=RTOL_STATS, atol=0, equal_nan=True)
    api.dc_device_status()
