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
    ("non_strict_compare", [("if (Tin < tau) done += 1;", "if (Tin <= tau) done += 1;", 1),
                            ("cnt[k] += (Tin < taus[k]) ? 1 : 0;", "cnt[k] += (Tin <= taus[k]) ? 1 : 0;", 1)]),
    ("last_worker_not_max", [("Ti = fmaxf(Ti, Tin);", "Ti = Tin;", 3)]),
    ("double_accumulator", [("float Tin = 0.0f;", "double Tin = 0.0;", 3)]),
    ("no_min_with_tau", [("out_step[i * K + k] = fminf(tau, Ti) + tc;", "out_step[i * K + k] = tau + tc;", 1),
                         ("(fminf(taus[k], Ti) + tc)", "(taus[k] + tc)", 1)]),
    ("sync_without_comm", [("out_sync[i] = Ti + tc;", "out_sync[i] = Ti;", 2)]),
    ("step_without_comm", [("out_step[i * K + k] = fminf(tau, Ti) + tc;", "out_step[i * K + k] = fminf(tau, Ti);", 1),
                           ("(fminf(taus[k], Ti) + tc)", "(fminf(taus[k], Ti))", 1)]),
    ("transposed_layout", [("const float *t = lat + (i * N + n) * M;", "const float *t = lat + (i * M + n) * N;", 2)]),
    ("skips_first_microbatch", [("for (int64_t m = 0; m < M; ++m) {\n                    if (rule == 0) {",
                                 "for (int64_t m = 1; m < M; ++m) {\n                    if (rule == 0) {", 2)]),
    ("exclusive_prefix_rule0", [("Tin = Tin + t[m];\n                        if (Tin < tau) done += 1;",
                                 "if (Tin < tau) done += 1;\n                        Tin = Tin + t[m];", 1),
                                ("Tin = Tin + t[m];\n                        for (int64_t k = 0; k < K; ++k) cnt[k] += (Tin < taus[k]) ? 1 : 0;",
                                 "for (int64_t k = 0; k < K; ++k) cnt[k] += (Tin < taus[k]) ? 1 : 0;\n                        Tin = Tin + t[m];", 1)]),
    ("speedup_forgets_workers", [("(dn / NM)", "(dn / (double)M)", 1)]),
    ("speedup_inverted_ratio", [("((double)sync[i] / st)", "(st / (double)sync[i])", 1)]),
    ("thr_mean_is_ratio_of_means", [("sum_ratio / (double)T", "((double)sum_done / sum_step)", 1)]),
    ("argmax_takes_last", [("v > objective[best]", "v >= objective[best]", 1)]),
    ("comm_time_of_wrong_iteration", [("t_comm_per_iter ? t_comm_per_iter[i] : t_comm", "t_comm_per_iter ? t_comm_per_iter[0] : t_comm", 2)]),
    ("bailey_weights_swapped", [("(1.0 - g) * dco_phi_inv(1.0 - 1.0 / (double)N) + g * dco_phi_inv(", "g * dco_phi_inv(1.0 - 1.0 / (double)N) + (1.0 - g) * dco_phi_inv(", 1)]),
    ("eq5_variance_not_scaled_by_m", [("sqrt((double)m * sigma * sigma)", "sqrt(sigma * sigma)", 1)]),
    ("eq11_numerator_without_comm", [("* (ET + t_comm) / step", "* ET / step", 1)]),
    ("rule1_inclusive", [("if (before < taus[k]) {", "if (Tin < taus[k]) {", 1),
                         ("if (Tin < tau) {\n                            done += 1;", "if (Tin + t[m] < tau) {\n                            done += 1;", 1)]),
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
    for order in ("rows", "literal"):
        missed = True
        for pin in pins.FAST_PINS:
            try:
                pin(lib, order=order)
            except AssertionError:
                missed = False
                caught.append((order, pin.__name__))
                break
        assert not missed, f"no pin noticed mutant {name} in order {order}"
