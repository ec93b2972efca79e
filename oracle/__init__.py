"""CPU oracle for the DropCompute threshold sweep.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
this package.  It compiles ``dc_oracle.c`` with gcc on first use (for the CPU
it is running on) and exposes the C functions on numpy arrays.  It imports
nothing from the CUDA package and the CUDA package imports nothing from here.

Paper passages each function follows are cited in ``dc_oracle.c``.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import platform
import subprocess
from typing import NamedTuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dc_oracle.c")
NSTATS = 5
STAT_NAMES = ("mean_step", "done_frac", "thr", "thr_mean", "s_eff")
_lib = None


def _host_tag() -> str:
    """A short tag for this host's CPU so a library built with -march=native
    on one machine is never loaded on another."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as f:
        src = f.read()
    h = hashlib.sha1(flags.encode() + platform.machine().encode() + src).hexdigest()[:12]
    return h


def lib_path() -> str:
    return os.path.join(_HERE, f"libdc_oracle.{_host_tag()}.so")


def build(force: bool = False, source: str | None = None, out: str | None = None) -> str:
    """Compile the oracle.  ``source``/``out`` let a test compile a deliberately
    altered copy (mutation checks) without touching the real one."""
    src = source or _SRC
    dst = out or lib_path()
    if not force and os.path.exists(dst) and os.path.getmtime(dst) >= os.path.getmtime(src):
        return dst
    tmp = dst + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=native", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", tmp, src, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, dst)
    return dst


def _bind(lib):
    i64, i32, f32 = ctypes.c_int64, ctypes.c_int, ctypes.c_float
    p = ctypes.c_void_p
    for name in ("dco_sweep_definition", "dco_sweep_rows"):
        fn = getattr(lib, name)
        fn.argtypes = [p, i64, i64, i64, p, i64, f32, p, i32, p, p, p, p]
        fn.restype = i32
    lib.dco_reduce_trials.argtypes = [p, p, p, i64, i64, i64, i64, p, p]
    lib.dco_reduce_trials.restype = i32
    lib.dco_argmax.argtypes = [p, i64]
    lib.dco_argmax.restype = i64
    lib.dco_s_eff_fractional.argtypes = [p, i64, i64, i64, p, i64, f32, p, p]
    lib.dco_s_eff_fractional.restype = i32
    f64 = ctypes.c_double
    lib.dco_closed_form.argtypes = [f64, f64, i64, i64, f64, f64, p, i64, p, p]
    lib.dco_closed_form.restype = i32
    lib.dco_bailey_mean_max.argtypes = [f64, f64, i64, i64]
    lib.dco_bailey_mean_max.restype = f64
    return lib


def load(path: str | None = None):
    global _lib
    if path is not None:
        return _bind(ctypes.CDLL(path))
    if _lib is None:
        _lib = _bind(ctypes.CDLL(build()))
    return _lib


def num_threads() -> int:
    """Threads the row-order sweep uses (OpenMP's default: OMP_NUM_THREADS or all cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        try:
            return max(1, int(env.split(",")[0]))
        except ValueError:
            pass
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


class Sweep(NamedTuple):
    step: np.ndarray  # [T,K] float32
    done: np.ndarray  # [T,K] int32
    sync: np.ndarray  # [T]   float32


class Stats(NamedTuple):
    stats: np.ndarray     # [NSTATS,K] float64, rows in STAT_NAMES order
    baseline: np.ndarray  # [2] float64: mean_sync, thr_sync


def _f32c(a, ndim):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.ndim == ndim
    return a


def sweep(lat, taus, t_comm: float, rule: int = 0, order: str = "rows", lib=None, worker_scale=None) -> Sweep:
    """Per-(iteration, tau) step time and completed count.

    ``order='definition'`` writes out each iteration's table of finish times and reads every quantity off
    it, one threshold at a time (Sec. 4.3's definitions as they stand);
    ``order='rows'`` reads every sample once (same predicate, same integers).
    ``t_comm`` is one number, or an array of T numbers (Algorithm 2's per-iteration T_i^c).
    ``worker_scale``: None, or N positive numbers s_n: worker n works against its own threshold s_n * tau_k."""
    lib = lib or load()
    lat = _f32c(lat, 3)
    taus = _f32c(taus, 1)
    T, N, M = lat.shape
    K = taus.shape[0]
    step = np.empty((T, K), np.float32)
    done = np.empty((T, K), np.int32)
    sync = np.empty((T,), np.float32)
    fn = {"definition": lib.dco_sweep_definition, "rows": lib.dco_sweep_rows}[order]
    tc_vec = None
    if np.ndim(t_comm) > 0:
        tc_vec = np.ascontiguousarray(t_comm, dtype=np.float32)
        assert tc_vec.shape == (T,)
    sc = None
    if worker_scale is not None:
        sc = np.ascontiguousarray(worker_scale, dtype=np.float32)
        assert sc.shape == (N,)
    rc = fn(lat.ctypes.data, T, N, M, taus.ctypes.data, K, np.float32(0.0 if tc_vec is not None else t_comm),
            None if tc_vec is None else tc_vec.ctypes.data, rule, None if sc is None else sc.ctypes.data,
            step.ctypes.data, done.ctypes.data, sync.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle sweep failed with status {rc}")
    return Sweep(step, done, sync)


def reduce_trials(step, done, sync, N: int, M: int, lib=None) -> Stats:
    lib = lib or load()
    step = _f32c(step, 2)
    done = np.ascontiguousarray(done, dtype=np.int32)
    sync = _f32c(sync, 1)
    T, K = step.shape
    assert done.shape == (T, K) and sync.shape == (T,)
    stats = np.empty((NSTATS, K), np.float64)
    base = np.empty((2,), np.float64)
    rc = lib.dco_reduce_trials(step.ctypes.data, done.ctypes.data, sync.ctypes.data, T, K, N, M,
                               stats.ctypes.data, base.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle reduce failed with status {rc}")
    return Stats(stats, base)


def argmax(objective, lib=None) -> int:
    lib = lib or load()
    obj = np.ascontiguousarray(objective, dtype=np.float64)
    return int(lib.dco_argmax(obj.ctypes.data, obj.shape[0]))


def s_eff_fractional(lat, taus, t_comm: float, lib=None):
    """S_eff(tau) and its first maximum with M~ accumulated as a floating-point mean over workers (Sec. 4.3's
    (1/N) sum_n form) instead of the integer count used everywhere else."""
    lib = lib or load()
    lat = _f32c(lat, 3)
    taus = _f32c(taus, 1)
    T, N, M = lat.shape
    K = taus.shape[0]
    s_eff = np.empty((K,), np.float64)
    k_star = ctypes.c_int64(-1)
    rc = lib.dco_s_eff_fractional(lat.ctypes.data, T, N, M, taus.ctypes.data, K, np.float32(t_comm),
                            s_eff.ctypes.data, ctypes.byref(k_star))
    if rc != 0:
        raise ValueError(f"oracle s_eff_fractional failed with status {rc}")
    return s_eff, int(k_star.value)


class ClosedForm(NamedTuple):
    done_frac: np.ndarray  # [K] E[M~]/M                      (Eq. 5)
    step: np.ndarray       # [K] min(tau, E[T]) + T^c
    s_eff: np.ndarray      # [K] E[S_eff]                      (Eq. 11)
    mean_T: float          # E[T] used (Eq. 4/12, or the value passed in)
    k_star: int
    tau_star: float


def closed_form(mu: float, sigma: float, M: int, N: int, t_comm: float, taus, mean_T: float = -1.0, lib=None) -> ClosedForm:
    """App. C.2's closed forms on a threshold grid; ``mean_T >= 0`` plugs in a measured E[T]."""
    lib = lib or load()
    taus = _f32c(taus, 1)
    K = taus.shape[0]
    out = np.empty((3, K), np.float64)
    sc = np.empty((3,), np.float64)
    rc = lib.dco_closed_form(mu, sigma, M, N, t_comm, mean_T, taus.ctypes.data, K, out.ctypes.data, sc.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle closed_form failed with status {rc}")
    return ClosedForm(out[0], out[1], out[2], float(sc[0]), int(sc[1]), float(sc[2]))


def bailey_mean_max(mu: float, sigma: float, M: int, N: int, lib=None) -> float:
    lib = lib or load()
    return float(lib.dco_bailey_mean_max(mu, sigma, M, N))
