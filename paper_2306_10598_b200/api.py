"""Thin Python binding of the C ABI in ``include/dropcompute.h`` (and of the measurement and tuning aids in
``include/dropcompute_dev.h``).

Argument marshalling only: every function checks dtype/device/contiguity of the torch tensors it is
given, passes their device pointers and the current CUDA stream to the library entry point of the
same name, and raises :class:`DropComputeError` on a non-zero status.  There is no fallback: if
``libdropcompute.so`` is not built this module fails to import.
"""
from __future__ import annotations

import ctypes
import os
from typing import NamedTuple, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdropcompute.so")

DC_MAX_K = 4096
RULE_FINISH_BEFORE_TAU = 0
RULE_START_BEFORE_TAU = 1
STAT_MEAN_STEP, STAT_DONE_FRAC, STAT_THR, STAT_THR_MEAN, STAT_S_EFF = range(5)
NSTATS = 5
STAT_NAMES = ("mean_step", "done_frac", "thr", "thr_mean", "s_eff")

EXPORTS = (
    "dc_simulate", "dc_simulate_ex", "dc_simulate_tc", "dc_simulate_scaled", "dc_simulate_split_workspace_bytes", "dc_simulate_split",
    "dc_reduce_workspace_bytes", "dc_reduce_trials", "dc_reduce_trials_static",
    "dc_argmax_tau", "dc_sweep_device",
    "dc_closed_form", "dc_sweep_host_workspace_bytes", "dc_sweep_host", "dc_check_inputs", "dc_device_status",
    "dc_status_string",
)
DEV_EXPORTS = ("dc_simulate_plan", "dc_tune", "dc_launch_count", "dc_read_probe", "dc_kernel_version")


class DropComputeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2306_10598_b200.build` "
        "(there is no CPU or PyTorch fallback for this library)")

_lib = ctypes.CDLL(LIB_PATH)

_p, _i64, _i32, _f32, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
_lib.dc_simulate.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _f32, _p, _p, _p]
_lib.dc_simulate_ex.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _f32, _p, _p, _p, _i32, _p]
_lib.dc_simulate_tc.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _p, _p, _p, _p, _i32, _p]
_lib.dc_simulate_tc.restype = ctypes.c_int
_lib.dc_simulate_scaled.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _p, _f32, _p, _p, _p, _i32, _p]
_lib.dc_simulate_scaled.restype = ctypes.c_int
_lib.dc_simulate_split_workspace_bytes.argtypes = [_i64, _i64, _i64, _i32]
_lib.dc_simulate_split_workspace_bytes.restype = _sz
_lib.dc_simulate_split.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _f32, _p, _p, _p, _i32, _p, _sz, _p]
_lib.dc_simulate_split.restype = ctypes.c_int
_lib.dc_reduce_workspace_bytes.argtypes = [_i64, _i32]
_lib.dc_reduce_workspace_bytes.restype = _sz
_lib.dc_reduce_trials.argtypes = [_p, _p, _p, _i64, _i32, _i64, _i64, _p, _p, _p, _sz, _p]
_lib.dc_reduce_trials_static.argtypes = [_p, _p, _p, _i64, _i32, _i64, _i64, _p, _p, _p]
_lib.dc_reduce_trials_static.restype = ctypes.c_int
_lib.dc_argmax_tau.argtypes = [_p, _p, _i32, _i32, _p, _p, _p, _p]
_lib.dc_sweep_device.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _f32, _i32, _i32, _p, _p, _p, _p, _p, _p, _p, _p, _p, _sz, _p]
_lib.dc_sweep_host_workspace_bytes.argtypes = [_i64, _i64, _i64, _i32, _i64]
_lib.dc_sweep_host_workspace_bytes.restype = _sz
_lib.dc_sweep_host.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _f32, _i32, _i32, _i64, _p, _p, _p, _p, _p, _sz, _p]
_lib.dc_closed_form.argtypes = [ctypes.c_double, ctypes.c_double, _i64, _i64, ctypes.c_double, ctypes.c_double, _p, _i32, _p, _p, _p]
_lib.dc_closed_form.restype = ctypes.c_int
_lib.dc_check_inputs.argtypes = [_p, _i64, _i64, _i64, _p, _i32, _p, _p, _p]
_lib.dc_device_status.argtypes = [_p]
_lib.dc_read_probe.argtypes = [_p, _i64, _p, _p]
_lib.dc_simulate_plan.argtypes = [_p, _i64, _i64, _i64, _i32]
_lib.dc_tune.argtypes = [_i32, _i32]
_lib.dc_tune.restype = ctypes.c_int
_lib.dc_status_string.argtypes = [ctypes.c_int]
_lib.dc_status_string.restype = ctypes.c_char_p
_lib.dc_kernel_version.argtypes = []
_lib.dc_kernel_version.restype = ctypes.c_char_p
_lib.dc_launch_count.argtypes = [_i32, _i64, _i64, _i64, _i32, _i64]
for _name in ("dc_simulate", "dc_simulate_ex", "dc_reduce_trials", "dc_argmax_tau", "dc_sweep_host", "dc_check_inputs",
              "dc_device_status", "dc_simulate_plan", "dc_launch_count", "dc_sweep_device", "dc_read_probe"):
    getattr(_lib, _name).restype = ctypes.c_int


def dc_kernel_version() -> str:
    return _lib.dc_kernel_version().decode()


def status_string(status: int) -> str:
    return _lib.dc_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise DropComputeError(status, where)


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def dc_simulate(latencies: torch.Tensor, taus: torch.Tensor, t_comm: float,
                out_step: torch.Tensor, out_done: torch.Tensor) -> None:
    """``dc_simulate`` of the C ABI on the current stream.  latencies [T,N,M] fp32, taus [K] fp32,
    out_step [T,K] fp32, out_done [T,K] int32 (all CUDA, contiguous)."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K)
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_simulate(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"), K,
                                float(t_comm), _dev(out_step, torch.float32, "out_step"),
                                _dev(out_done, torch.int32, "out_done"), _stream(latencies)), "dc_simulate")


def dc_simulate_ex(latencies: torch.Tensor, taus: torch.Tensor, t_comm: float, out_step: torch.Tensor,
                   out_done: torch.Tensor, out_sync: Optional[torch.Tensor], rule: int = RULE_FINISH_BEFORE_TAU) -> None:
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K)
    assert out_sync is None or tuple(out_sync.shape) == (T,)
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_simulate_ex(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"),
                                   K, float(t_comm), _dev(out_step, torch.float32, "out_step"),
                                   _dev(out_done, torch.int32, "out_done"),
                                   None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                   int(rule), _stream(latencies)), "dc_simulate_ex")


def dc_simulate_tc(latencies: torch.Tensor, taus: torch.Tensor, t_comm_trials: torch.Tensor, out_step: torch.Tensor,
                   out_done: torch.Tensor, out_sync: Optional[torch.Tensor], rule: int = RULE_FINISH_BEFORE_TAU) -> None:
    """``dc_simulate_tc``: like dc_simulate_ex with one communication time per trial (t_comm_trials [T] fp32)."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K) and tuple(t_comm_trials.shape) == (T,)
    assert out_sync is None or tuple(out_sync.shape) == (T,)
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_simulate_tc(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"),
                                   K, _dev(t_comm_trials, torch.float32, "t_comm_trials"),
                                   _dev(out_step, torch.float32, "out_step"), _dev(out_done, torch.int32, "out_done"),
                                   None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                   int(rule), _stream(latencies)), "dc_simulate_tc")


def dc_simulate_scaled(latencies: torch.Tensor, taus: torch.Tensor, worker_scale: torch.Tensor, t_comm: float,
                       out_step: torch.Tensor, out_done: torch.Tensor, out_sync: Optional[torch.Tensor],
                       rule: int = RULE_FINISH_BEFORE_TAU) -> None:
    """``dc_simulate_scaled``: worker n works against its own thresholds worker_scale[n] * taus[k] (worker_scale [N] fp32)."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K) and tuple(worker_scale.shape) == (N,)
    assert out_sync is None or tuple(out_sync.shape) == (T,)
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_simulate_scaled(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"),
                                       K, _dev(worker_scale, torch.float32, "worker_scale"), float(t_comm),
                                       _dev(out_step, torch.float32, "out_step"), _dev(out_done, torch.int32, "out_done"),
                                       None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                       int(rule), _stream(latencies)), "dc_simulate_scaled")


def dc_simulate_split_workspace_bytes(T: int, N: int, M: int, K: int) -> int:
    return int(_lib.dc_simulate_split_workspace_bytes(T, N, M, K))


def dc_simulate_split(latencies: torch.Tensor, taus: torch.Tensor, t_comm: float, out_step: torch.Tensor,
                      out_done: torch.Tensor, out_sync: Optional[torch.Tensor], workspace: Optional[torch.Tensor],
                      rule: int = RULE_FINISH_BEFORE_TAU) -> None:
    """``dc_simulate_split``: dc_simulate_ex for few trials of many workers (each trial is swept as several
    groups of workers on different blocks and merged).  ``workspace``: CUDA tensor of at least
    dc_simulate_split_workspace_bytes(T, N, M, K) bytes, 256-byte aligned (None when that is 0)."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K)
    assert out_sync is None or tuple(out_sync.shape) == (T,)
    wptr = None if workspace is None else workspace.data_ptr()
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_simulate_split(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"),
                                      K, float(t_comm), _dev(out_step, torch.float32, "out_step"),
                                      _dev(out_done, torch.int32, "out_done"),
                                      None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                      int(rule), wptr, wbytes, _stream(latencies)), "dc_simulate_split")


def dc_reduce_workspace_bytes(T: int, K: int) -> int:
    return int(_lib.dc_reduce_workspace_bytes(T, K))


def dc_reduce_trials(out_step: torch.Tensor, out_done: torch.Tensor, out_sync: Optional[torch.Tensor], N: int, M: int,
                     stats: torch.Tensor, baseline: torch.Tensor, workspace: torch.Tensor) -> None:
    """stats [NSTATS,K] fp64, baseline [2] fp64, workspace: any CUDA tensor of at least
    dc_reduce_workspace_bytes(T,K) bytes."""
    T, K = out_step.shape
    assert tuple(stats.shape) == (NSTATS, K) and tuple(baseline.shape) == (2,)
    if not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous CUDA tensor")
    with torch.cuda.device(out_step.device):
        _check(_lib.dc_reduce_trials(_dev(out_step, torch.float32, "out_step"), _dev(out_done, torch.int32, "out_done"),
                                     None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                     T, K, int(N), int(M), _dev(stats, torch.float64, "stats"),
                                     _dev(baseline, torch.float64, "baseline"), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream(out_step)), "dc_reduce_trials")


STATIC_MAX_K = 1024


def dc_reduce_trials_static(out_step: torch.Tensor, out_done: torch.Tensor, out_sync: Optional[torch.Tensor], N: int,
                            M: int, stats: torch.Tensor, baseline: torch.Tensor) -> None:
    """``dc_reduce_trials_static``: the trial statistics without a workspace argument, for callers that may
    not allocate device memory (the partial sums go to an array built into the library; K <= STATIC_MAX_K).
    This wrapper allocates nothing either: it only passes the pointers of the tensors it is given.  Calls on
    one device share that array, so do not run two of them concurrently on different streams."""
    T, K = out_step.shape
    assert tuple(stats.shape) == (NSTATS, K) and tuple(baseline.shape) == (2,)
    with torch.cuda.device(out_step.device):
        _check(_lib.dc_reduce_trials_static(_dev(out_step, torch.float32, "out_step"), _dev(out_done, torch.int32, "out_done"),
                                            None if out_sync is None else _dev(out_sync, torch.float32, "out_sync"),
                                            T, K, int(N), int(M), _dev(stats, torch.float64, "stats"),
                                            _dev(baseline, torch.float64, "baseline"), _stream(out_step)),
               "dc_reduce_trials_static")


def dc_argmax_tau(stats: torch.Tensor, taus: torch.Tensor, objective: int, out_k: torch.Tensor, out_tau: torch.Tensor,
                  out_value: torch.Tensor) -> None:
    K = taus.shape[0]
    with torch.cuda.device(stats.device):
        _check(_lib.dc_argmax_tau(_dev(stats, torch.float64, "stats"), _dev(taus, torch.float32, "taus"), K, int(objective),
                                  _dev(out_k, torch.int32, "out_k"), _dev(out_tau, torch.float32, "out_tau"),
                                  _dev(out_value, torch.float64, "out_value"), _stream(stats)), "dc_argmax_tau")


def dc_closed_form(mu: float, sigma: float, M: int, N: int, t_comm: float, taus: torch.Tensor, out: torch.Tensor,
                   scalars: torch.Tensor, mean_T: float = -1.0) -> None:
    """``dc_closed_form``: App. C.2's estimates on the grid.  out [3,K] fp64 (E[M~]/M, step, E[S_eff]),
    scalars [1] fp64 (E[T]); mean_T >= 0 plugs in a measured E[T]."""
    K = taus.shape[0]
    assert tuple(out.shape) == (3, K) and scalars.numel() >= 1
    with torch.cuda.device(taus.device):
        _check(_lib.dc_closed_form(float(mu), float(sigma), int(M), int(N), float(t_comm), float(mean_T),
                                   _dev(taus, torch.float32, "taus"), K, _dev(out, torch.float64, "out"),
                                   _dev(scalars, torch.float64, "scalars"), _stream(taus)), "dc_closed_form")


def dc_check_inputs(latencies: torch.Tensor, taus: torch.Tensor) -> None:
    """Synchronous data-precondition check; raises DropComputeError (DC_ERR_LATENCIES / DC_ERR_TAUS)."""
    T, N, M = latencies.shape
    counters = torch.empty(2, dtype=torch.int64, device=latencies.device)
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_check_inputs(_dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"),
                                    taus.shape[0], counters.data_ptr(), None, _stream(latencies)), "dc_check_inputs")


def dc_read_probe(data: torch.Tensor, sink: torch.Tensor) -> None:
    """Enqueues a plain read-only pass over `data` (a measurement aid; see the header)."""
    with torch.cuda.device(data.device):
        _check(_lib.dc_read_probe(_dev(data, torch.float32, "data"), data.numel(), _dev(sink, torch.float32, "sink"),
                                  _stream(data)), "dc_read_probe")


def dc_device_status() -> int:
    """Reads and clears the device's expired-wait mask; raises if any wait expired."""
    flags = ctypes.c_uint32(0)
    rc = _lib.dc_device_status(ctypes.byref(flags))
    _check(rc, f"dc_device_status (flags {flags.value:#x})")
    return int(flags.value)


def dc_simulate_plan(latencies: torch.Tensor, K: int) -> int:
    T, N, M = latencies.shape
    return int(_lib.dc_simulate_plan(latencies.data_ptr(), T, N, M, K))


def dc_sweep_host_workspace_bytes(T: int, N: int, M: int, K: int, chunk_trials: int) -> int:
    return int(_lib.dc_sweep_host_workspace_bytes(T, N, M, K, chunk_trials))


class HostSweep(NamedTuple):
    stats: torch.Tensor      # [NSTATS,K] fp64, host
    baseline: torch.Tensor   # [2] fp64, host
    k_star: int
    tau_star: float


def dc_sweep_host(latencies_host: torch.Tensor, taus_host: torch.Tensor, t_comm: float, workspace: torch.Tensor,
                  chunk_trials: int, rule: int = RULE_FINISH_BEFORE_TAU, objective: int = STAT_S_EFF,
                  stats_out: Optional[torch.Tensor] = None, baseline_out: Optional[torch.Tensor] = None) -> HostSweep:
    """``dc_sweep_host``: latencies and thresholds in HOST memory (pin them for speed), results in
    host memory; synchronous.  ``workspace`` is a CUDA byte tensor from dc_sweep_host_workspace_bytes."""
    for t, dt, nm in ((latencies_host, torch.float32, "latencies_host"), (taus_host, torch.float32, "taus_host")):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise TypeError(f"{nm} must be a contiguous host {dt} tensor")
    T, N, M = latencies_host.shape
    K = taus_host.shape[0]
    stats = stats_out if stats_out is not None else torch.empty((NSTATS, K), dtype=torch.float64)
    base = baseline_out if baseline_out is not None else torch.empty((2,), dtype=torch.float64)
    k_star = ctypes.c_int32(-1)
    tau_star = ctypes.c_float(float("nan"))
    with torch.cuda.device(workspace.device):
        _check(_lib.dc_sweep_host(latencies_host.data_ptr(), T, N, M, taus_host.data_ptr(), K, float(t_comm), int(rule),
                                  int(objective), int(chunk_trials), stats.data_ptr(), base.data_ptr(),
                                  ctypes.addressof(k_star), ctypes.addressof(tau_star), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(),
                                  torch.cuda.current_stream(workspace.device).cuda_stream), "dc_sweep_host")
    return HostSweep(stats, base, int(k_star.value), float(tau_star.value))


TUNE_STAGES, TUNE_LANE_COPIES, TUNE_WARP_GROUPS, TUNE_BOX_FLOATS, TUNE_BATCH_LOOKUPS, TUNE_DIRECT_BINS = 1, 2, 3, 4, 5, 6
TUNE_FLAT_TILE_WARPS, TUNE_FLAT_GROUPS, TUNE_FLAT_DEPTH, TUNE_FLAT_MAX_M = 7, 8, 9, 11
TUNE_LEAN_LOOP, TUNE_TILE_TRIALS, TUNE_WHOLE_LINES, TUNE_EVEN_GRID, TUNE_L2_PROMOTION = 12, 13, 14, 15, 16


def dc_tune(key: int, value: int) -> None:
    _check(_lib.dc_tune(int(key), int(value)), "dc_tune")


ENTRY_SIMULATE, ENTRY_SIMULATE_SPLIT, ENTRY_REDUCE_TRIALS, ENTRY_ARGMAX_TAU, ENTRY_SWEEP_DEVICE, ENTRY_SWEEP_HOST = range(6)


def dc_launch_count(entry_point: int, T: int, N: int, M: int, K: int, chunk_trials: int = 0) -> int:
    """Kernels one successful call of an entry point enqueues for this shape (``dc_launch_count``)."""
    n = int(_lib.dc_launch_count(int(entry_point), T, N, M, K, int(chunk_trials)))
    if n < 0:
        raise DropComputeError(-n, "dc_launch_count")
    return n


# --- convenience wrapper (allocation + the three calls); still nothing but calls into the library ---------------

class SweepResult(NamedTuple):
    out_step: torch.Tensor   # [T,K] fp32
    out_done: torch.Tensor   # [T,K] int32
    out_sync: torch.Tensor   # [T] fp32
    stats: torch.Tensor      # [NSTATS,K] fp64
    baseline: torch.Tensor   # [2] fp64
    k_star: torch.Tensor     # int32 scalar (device)
    tau_star: torch.Tensor   # fp32 scalar (device)
    value: torch.Tensor      # fp64 scalar (device)


def dc_sweep_device(latencies: torch.Tensor, taus: torch.Tensor, t_comm: float, rule: int, objective: int,
                    out_step: torch.Tensor, out_done: torch.Tensor, out_sync: torch.Tensor, stats: torch.Tensor,
                    baseline: torch.Tensor, out_k: torch.Tensor, out_tau: torch.Tensor, out_value: torch.Tensor,
                    workspace: torch.Tensor) -> None:
    """dc_simulate_ex + dc_reduce_trials + dc_argmax_tau enqueued by one call into the library."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    assert tuple(out_step.shape) == (T, K) and tuple(out_done.shape) == (T, K) and tuple(out_sync.shape) == (T,)
    assert tuple(stats.shape) == (NSTATS, K) and baseline.numel() == 2
    with torch.cuda.device(latencies.device):
        _check(_lib.dc_sweep_device(
            _dev(latencies, torch.float32, "latencies"), T, N, M, _dev(taus, torch.float32, "taus"), K, float(t_comm),
            int(rule), int(objective), _dev(out_step, torch.float32, "out_step"), _dev(out_done, torch.int32, "out_done"),
            _dev(out_sync, torch.float32, "out_sync"), _dev(stats, torch.float64, "stats"),
            _dev(baseline, torch.float64, "baseline"), _dev(out_k, torch.int32, "out_k"),
            _dev(out_tau, torch.float32, "out_tau"), _dev(out_value, torch.float64, "out_value"),
            _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(latencies)), "dc_sweep_device")


def sweep(latencies: torch.Tensor, taus: torch.Tensor, t_comm: float, rule: int = RULE_FINISH_BEFORE_TAU,
          objective: int = STAT_S_EFF) -> SweepResult:
    """Allocates the outputs with torch and runs dc_simulate_ex, dc_reduce_trials and dc_argmax_tau."""
    T, N, M = latencies.shape
    K = taus.shape[0]
    dev = latencies.device
    out_step = torch.empty((T, K), dtype=torch.float32, device=dev)
    out_done = torch.empty((T, K), dtype=torch.int32, device=dev)
    out_sync = torch.empty((T,), dtype=torch.float32, device=dev)
    stats = torch.empty((NSTATS, K), dtype=torch.float64, device=dev)
    baseline = torch.empty((2,), dtype=torch.float64, device=dev)
    ws = torch.empty((max(8, dc_reduce_workspace_bytes(T, K)),), dtype=torch.uint8, device=dev)
    k_star = torch.empty((), dtype=torch.int32, device=dev)
    tau_star = torch.empty((), dtype=torch.float32, device=dev)
    value = torch.empty((), dtype=torch.float64, device=dev)
    dc_simulate_ex(latencies, taus, t_comm, out_step, out_done, out_sync, rule)
    dc_reduce_trials(out_step, out_done, out_sync, N, M, stats, baseline, ws)
    dc_argmax_tau(stats, taus, objective, out_k=k_star, out_tau=tau_star, out_value=value)
    return SweepResult(out_step, out_done, out_sync, stats, baseline, k_star, tau_star, value)
