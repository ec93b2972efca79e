"""The C-ABI library loads without a GPU, exports every function the header declares, and turns
host-visible argument errors into status codes before touching CUDA (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dropcompute.h")
DEV_HEADER = os.path.join(ROOT, "include", "dropcompute_dev.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2306_10598_b200 import build
    build.build_library()
    from paper_2306_10598_b200 import api
    return api._lib


def declared_functions(header=HEADER):
    with open(header) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(dc_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert "dc_simulate" in names and "dc_reduce_trials" in names and "dc_argmax_tau" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in dropcompute.h but not exported"
    from paper_2306_10598_b200 import api
    assert sorted(api.EXPORTS) == names, "the Python binding must list exactly the header's functions"
    # the measurement and tuning aids live in a header of their own, outside the product interface
    dev = declared_functions(DEV_HEADER)
    assert sorted(api.DEV_EXPORTS) == dev and not set(dev) & set(names)
    for n in dev:
        assert hasattr(lib, n), f"{n} is declared in dropcompute_dev.h but not exported"
    for n in ("dc_tune", "dc_read_probe", "dc_kernel_version", "dc_launch_count"):
        assert n in dev and n not in names


def test_argument_errors_need_no_gpu(lib):
    A = 0x10000  # a made-up aligned address: validation fails before anything is dereferenced
    f = ctypes.c_float(0.1)
    # null pointers
    assert lib.dc_simulate(None, 1, 1, 1, A, 1, f, A, A, None) == 1
    assert lib.dc_simulate(A, 1, 1, 1, None, 1, f, A, A, None) == 1
    assert lib.dc_simulate(A, 1, 1, 1, A, 1, f, None, A, None) == 1
    assert lib.dc_simulate(A, 1, 1, 1, A, 1, f, A, None, None) == 1
    # shapes
    for T, N, M, K in ((0, 1, 1, 1), (1, 0, 1, 1), (1, 1, -3, 1), (1, 1, 1, 0)):
        assert lib.dc_simulate(A, T, N, M, A, K, f, A, A, None) == 2
    # ranges: K beyond the maximum, N*M beyond int32
    assert lib.dc_simulate(A, 1, 1, 1, A, 4097, f, A, A, None) == 4
    assert lib.dc_simulate(A, 1, 1 << 20, 1 << 12, A, 1, f, A, A, None) == 4
    # alignment
    assert lib.dc_simulate(A + 2, 1, 1, 1, A, 1, f, A, A, None) == 3
    assert lib.dc_simulate(A, 1, 1, 1, A + 1, 1, f, A, A, None) == 3
    # unknown rule
    assert lib.dc_simulate_ex(A, 1, 1, 1, A, 1, f, A, A, None, 5, None) == 7
    # reduce / argmax
    assert lib.dc_reduce_trials(None, A, A, 1, 1, 1, 1, A, A, A, 1 << 20, None) == 1
    assert lib.dc_reduce_trials(A, A, A, 1, 1, 1, 1, A, A, None, 0, None) == 9
    assert lib.dc_reduce_trials(A, A, A, 100, 8, 1, 1, A, A, A, 8, None) == 9
    assert lib.dc_argmax_tau(A, A, 4, 1, A, A, A, None) == 7      # done_frac is not an objective
    assert lib.dc_argmax_tau(A, A, 0, 4, A, A, A, None) == 2
    assert lib.dc_simulate_plan(A, 4, 8, 12, 3) == 0
    assert lib.dc_simulate_plan(A, 4, 8, 13, 3) == 2
    assert lib.dc_simulate_plan(A, 4, 8, 301, 3) == 1
    assert lib.dc_simulate_plan(A, 4, 8, 127, 3) == 2 and lib.dc_simulate_plan(A, 4, 8, 129, 3) == 1
    assert lib.dc_simulate_plan(A + 4, 4, 8, 12, 3) == 2
    assert lib.dc_simulate_plan(A + 4, 4, 8, 300, 3) == 1
    assert lib.dc_simulate_plan(A, 4, 8, 12, 5000) == -4
    # the later entry points
    assert lib.dc_simulate_tc(A, 1, 1, 1, A, 1, None, A, A, None, 0, None) == 1          # per-trial times missing
    assert lib.dc_simulate_tc(A, 1, 1, 1, A, 1, A + 2, A, A, None, 0, None) == 3
    assert lib.dc_simulate_scaled(A, 1, 1, 1, A, 1, None, f, A, A, None, 0, None) == 1      # per-worker scales missing
    assert lib.dc_simulate_scaled(A, 1, 1, 1, A, 1, A + 2, f, A, A, None, 0, None) == 3
    assert lib.dc_simulate_scaled(A, 1, 1, 1, A, 1, A, f, A, A, None, 3, None) == 7
    assert lib.dc_reduce_trials_static(A, A, A, 4, 1025, 1, 1, A, A, None) == 4           # beyond the built-in scratch
    assert lib.dc_reduce_trials_static(A, A, A, 0, 4, 1, 1, A, A, None) == 2
    d = ctypes.c_double
    assert lib.dc_closed_form(d(1.0), d(0.1), 4, 1, d(0.1), d(-1.0), A, 4, A, A, None) == 2   # needs N >= 2
    assert lib.dc_closed_form(d(1.0), d(0.0), 4, 8, d(0.1), d(-1.0), A, 4, A, A, None) == 4   # sigma must be > 0
    assert lib.dc_closed_form(d(1.0), d(0.1), 4, 8, d(0.1), d(-1.0), None, 4, A, A, None) == 1
    # tuning knobs: unknown keys and values are refused, 0 always restores the default
    assert lib.dc_tune(1, 9) == 7 and lib.dc_tune(2, 3) == 7 and lib.dc_tune(99, 0) == 7
    for key in (1, 2, 3, 4, 5):
        assert lib.dc_tune(key, 0) == 0
    assert lib.dc_kernel_version().startswith(b"sweep-")
    from paper_2306_10598_b200 import build
    assert lib.dc_kernel_version() == b"sweep-" + build.source_hash().encode()   # the tag follows the sources
    # sizes that would overflow N*M are refused, not multiplied
    assert lib.dc_reduce_trials(A, A, A, 4, 4, 1 << 62, 1 << 62, A, A, A, 1 << 20, None) == 4
    assert lib.dc_reduce_trials_static(A, A, A, 4, 4, 1 << 62, 4, A, A, None) == 4
    # launch counts are a pure function of the shape
    assert lib.dc_launch_count(0, 5, 5, 5, 5, 0) == 1 and lib.dc_launch_count(2, 5, 5, 5, 5, 0) == 2
    assert lib.dc_launch_count(3, 5, 5, 5, 5, 0) == 1 and lib.dc_launch_count(4, 5, 5, 5, 5, 0) == 4
    assert lib.dc_launch_count(5, 10, 5, 5, 5, 3) == 4 + 3 and lib.dc_launch_count(5, 10, 5, 5, 5, 0) == -2
    assert lib.dc_launch_count(9, 5, 5, 5, 5, 0) == -7 and lib.dc_launch_count(0, 0, 5, 5, 5, 0) == -2


def test_two_host_threads_and_the_tuning_knobs(lib):
    """The library is called from two host threads at once while a third keeps changing the expert settings:
    every call must come back with the status its own arguments deserve (argument errors need no GPU; with valid
    arguments a call ends with DC_ERR_CUDA on a machine without a GPU and DC_OK on one with)."""
    import threading
    A = 0x10000
    f = ctypes.c_float(0.1)
    stop = threading.Event()
    bad = []

    def tuner():
        i = 0
        while not stop.is_set():
            for key, vals in ((1, (0, 2, 3, 4)), (2, (0, 1, 2, 4)), (3, (0, 1, 2)), (5, (0, 1, 2)), (6, (0, 1, 2)), (11, (0, 200))):
                if lib.dc_tune(key, vals[i % len(vals)]) != 0:
                    bad.append(("tune", key))
            if lib.dc_tune(99, 0) != 7:
                bad.append(("tune", 99))
            i += 1

    def caller(seed):
        for i in range(3000):
            j = (i + seed) % 5
            if j == 0 and lib.dc_simulate(None, 1, 1, 1, A, 1, f, A, A, None) != 1:
                bad.append(("null", i))
            if j == 1 and lib.dc_simulate(A, 1, 1, 1, A, 4097, f, A, A, None) != 4:
                bad.append(("range", i))
            if j == 2 and lib.dc_simulate_ex(A, 1, 1, 1, A, 1, f, A, A, None, 5, None) != 7:
                bad.append(("rule", i))
            if j == 3 and lib.dc_simulate_plan(A, 4, 8, 129 + (i % 2) * 72, 3) not in (1, 2):
                bad.append(("plan", i))
            if j == 4 and lib.dc_reduce_trials(A, A, A, 100, 8, 1, 1, A, A, A, 8, None) != 9:
                bad.append(("workspace", i))

    threads = [threading.Thread(target=tuner)] + [threading.Thread(target=caller, args=(s,)) for s in (0, 2)]
    for t in threads:
        t.start()
    for t in threads[1:]:
        t.join()
    stop.set()
    threads[0].join()
    for key in (1, 2, 3, 5, 6, 11):
        assert lib.dc_tune(key, 0) == 0
    assert not bad, bad[:5]


def test_workspace_sizes(lib):
    from paper_2306_10598_b200 import api
    assert api.dc_reduce_workspace_bytes(0, 4) == 0
    for T, K in ((1, 1), (31, 7), (33, 16), (32768, 256), (5000, 4096)):
        b = api.dc_reduce_workspace_bytes(T, K)
        chunks = min(64, -(-T // 32))
        rows = -(-T // chunks)
        chunks = -(-T // rows)
        assert b == 8 * (chunks * 4 * K + chunks)
    assert api.dc_sweep_host_workspace_bytes(8, 4, 4, 2, 0) == 0
    assert api.dc_sweep_host_workspace_bytes(1024, 8, 4, 16, 4096) == api.dc_sweep_host_workspace_bytes(1024, 8, 4, 16, 1024)
    assert api.status_string(0) == "ok" and "NULL" in api.status_string(1)
