"""Plant one plausible mistake at a time in a COPY of the oracle's C source (on the CPU, never in
the CUDA path) and require that the pins notice it.  This is what shows the pins are sharp enough
to trust the oracle as the reference for the GPU parity tests."""
import os

import pytest

import oracle
import pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "dc_oracle.c")

# (name, [(old, new, expected_occurrences)])
MUTANTS = [
    ("non_strict_compare", [("completed += (f[m] < tau) ? 1 : 0;", "completed += (f[m] <= tau) ? 1 : 0;", 1),
                            ("cnt[k] += (elapsed < taus[k]) ? 1 : 0;", "cnt[k] += (elapsed <= taus[k]) ? 1 : 0;", 1)]),
    ("last_worker_not_max", [("slowest_full = fmaxf(slowest_full, finish[n * M + (M - 1)]);", "slowest_full = finish[n * M + (M - 1)];", 1),
                             ("slowest_full = fmaxf(slowest_full, elapsed);", "slowest_full = elapsed;", 2)]),
    ("double_accumulator", [("float elapsed = 0.0f;", "double elapsed = 0.0;", 4)]),
    ("no_min_with_tau", [("(fminf(tau, slowest_full) + tc)", "(tau + tc)", 1),
                         ("(fminf(taus[k], slowest_full) + tc)", "(taus[k] + tc)", 1)]),
    ("sync_without_comm", [("out_sync[i] = slowest_full + tc;", "out_sync[i] = slowest_full;", 2)]),
    ("step_without_comm", [("(fminf(tau, slowest_full) + tc)", "(fminf(tau, slowest_full))", 1),
                           ("(fminf(taus[k], slowest_full) + tc)", "(fminf(taus[k], slowest_full))", 1)]),
    ("transposed_layout", [("const float *row = lat + (i * N + n) * M;", "const float *row = lat + (i * M + n) * N;", 4)]),
    ("skips_first_microbatch", [("elapsed = elapsed + row[m];\n                finish[n * M + m] = elapsed;",
                                 "if (m > 0) elapsed = elapsed + row[m];\n                finish[n * M + m] = elapsed;", 1),
                                ("for (int64_t m = 0; m < M; ++m) {\n                    if (rule == 0) {",
                                 "for (int64_t m = 1; m < M; ++m) {\n                    if (rule == 0) {", 1)]),
    ("exclusive_prefix_rule0", [("elapsed = elapsed + row[m];\n                finish[n * M + m] = elapsed;",
                                 "finish[n * M + m] = elapsed;\n                elapsed = elapsed + row[m];", 1),
                                ("elapsed = elapsed + row[m];\n                        for (int64_t k = 0; k < K; ++k) cnt[k] += (elapsed < taus[k]) ? 1 : 0;",
                                 "for (int64_t k = 0; k < K; ++k) cnt[k] += (elapsed < taus[k]) ? 1 : 0;\n                        elapsed = elapsed + row[m];", 1)]),
    ("speedup_forgets_workers", [("(dn / NM)", "(dn / (double)M)", 1)]),
    ("speedup_inverted_ratio", [("((double)sync[i] / st)", "(st / (double)sync[i])", 1)]),
    ("thr_mean_is_ratio_of_means", [("sum_ratio / (double)T", "((double)sum_done / sum_step)", 1)]),
    ("argmax_takes_last", [("v > objective[best]", "v >= objective[best]", 1)]),
    ("comm_time_of_wrong_iteration", [("t_comm_per_iter ? t_comm_per_iter[i] : t_comm", "t_comm_per_iter ? t_comm_per_iter[0] : t_comm", 2)]),
    ("bailey_weights_swapped", [("(1.0 - g) * dco_phi_inv(1.0 - 1.0 / (double)N) + g * dco_phi_inv(", "g * dco_phi_inv(1.0 - 1.0 / (double)N) + (1.0 - g) * dco_phi_inv(", 1)]),
    ("eq5_variance_not_scaled_by_m", [("sqrt((double)m * sigma * sigma)", "sqrt(sigma * sigma)", 1)]),
    ("eq11_numerator_without_comm", [("* (ET + t_comm) / step", "* ET / step", 1)]),
    ("rule1_inclusive", [("const float start = (m == 0) ? 0.0f : f[m - 1];", "const float start = f[m];", 2),
                         ("if (start < taus[k]) {", "if (elapsed < taus[k]) {", 1)]),
    ("rule1_time_is_start_of_last", [("last_run >= 0 ? f[last_run] : 0.0f", "last_run > 0 ? f[last_run - 1] : 0.0f", 2),
                                     ("wlast[k] = elapsed;", "wlast[k] = start;", 2)]),
    ("scale_of_the_wrong_worker", [("worker_scale[n] * taus[k]", "worker_scale[0] * taus[k]", 2)]),
    ("scaled_worker_time_ignores_its_threshold", [("worker_time = fminf(own_tau, f[M - 1]);", "worker_time = f[M - 1];", 1),
                                                  ("(rule == 0) ? fminf(own[k], elapsed) : wlast[k]", "(rule == 0) ? elapsed : wlast[k]", 1)]),
    ("scaled_step_starts_from_zero", [("slowest = (n == 0) ? worker_time : fmaxf(slowest, worker_time);", "slowest = fmaxf(slowest, worker_time);", 1),
                                      ("wmax[k] = (n == 0) ? worker_time : fmaxf(wmax[k], worker_time);", "wmax[k] = fmaxf(wmax[k], worker_time);", 1)]),
    ("rule1_last_worker_not_max", [("slowest_cut = fmaxf(slowest_cut, last_run >= 0 ? f[last_run] : 0.0f);",
                                    "slowest_cut = last_run >= 0 ? f[last_run] : 0.0f;", 1),
                                   ("wmax[k] = fmaxf(wmax[k], wlast[k]);", "wmax[k] = wlast[k];", 1)]),
]


@pytest.mark.parametrize("name,edits", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, edits):
    with open(SRC) as f:
        src = f.read()
    for old, new, count in edits:
        assert src.count(old) == count, f"mutation site for {name} not found {count}x: {old!r}"
        src = src.replace(old, new)
    c = tmp_path / f"{name}.c"
    c.write_text(src)
    so = str(tmp_path / f"{name}.so")
    oracle.build(force=True, source=str(c), out=so)
    lib = oracle.load(so)
    caught = []
    for order in ("rows", "definition"):
        missed = True
        for pin in pins.FAST_PINS:
            try:
                pin(lib, order=order)
            except AssertionError:
                missed = False
                caught.append((order, pin.__name__))
                break
        assert not missed, f"no pin noticed mutant {name} in order {order}"


def test_swapped_bailey_weights_die_on_the_quadrature_pin(tmp_path):
    """Eq. 4's two weights exchanged: the pin that notices must be the one that compares with the exact
    E[max] from Eq. 3's integral, not a retyped copy of the formula."""
    with open(SRC) as f:
        src = f.read()
    old, new, count = dict((m[0], m[1]) for m in MUTANTS)["bailey_weights_swapped"][0]
    assert src.count(old) == count
    c = tmp_path / "bailey.c"
    c.write_text(src.replace(old, new))
    so = str(tmp_path / "bailey.so")
    oracle.build(force=True, source=str(c), out=so)
    with pytest.raises(AssertionError):
        pins.pin_bailey_against_quadrature(oracle.load(so))
    pins.pin_bailey_against_quadrature(oracle.load())
