"""The battery of checks that pins the CPU oracle to things other than itself.

Each ``pin_*`` takes a loaded oracle library (the real one, or a deliberately
altered copy in the mutation test) and raises AssertionError when the library
disagrees with what the paper and the mathematics fix.  Citations name the
paper's sections/equations/algorithms.
"""
from __future__ import annotations

import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import scipy.integrate
import scipy.stats

import oracle
from paper_2306_10598_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
INF = np.float32(np.inf)


def _np(t):
    return t.numpy() if hasattr(t, "numpy") else np.asarray(t)


def _stats(lib, lat, taus, t_comm, rule=0, order="rows", worker_scale=None):
    lat = _np(lat)
    T, N, M = lat.shape
    sw = oracle.sweep(lat, taus, t_comm, rule=rule, order=order, lib=lib, worker_scale=worker_scale)
    st = oracle.reduce_trials(sw.step, sw.done, sw.sync, N, M, lib=lib)
    return sw, st


# --- closed forms ------------------------------------------------------------

def pin_exp_max_harmonic(lib, order="rows"):
    """Sec. 4.2 / Eq. 3 special case: the max of N iid Exp(rate) has mean H_N / rate.
    M = 1, tau = infinity, T^c = 0."""
    for N, rate, T, seed in ((8, 2.0, 40000, 1), (200, 5.0, 20000, 2)):
        lat = W.iid_latencies("exp", T, N, 1, seed, rate=rate)
        sw, st = _stats(lib, lat, np.array([INF]), 0.0, order=order)
        H = sum(1.0 / i for i in range(1, N + 1))
        sd = math.sqrt(sum(1.0 / (i * rate) ** 2 for i in range(1, N + 1)))
        assert abs(st.baseline[0] - H / rate) <= 5 * sd / math.sqrt(T), (N, st.baseline[0], H / rate)
        # tau = infinity: everything completed, step is the plain synchronous max
        assert (sw.done == N).all() and (sw.step[:, 0] == sw.sync).all()
        assert abs(st.stats[0, 0] - st.baseline[0]) <= 1e-12 * st.baseline[0]
        assert np.array_equal(sw.sync, _np(lat).max(axis=(1, 2)))


def _emax_normal(N, mu, sd):
    f = lambda x: x * N * scipy.stats.norm.pdf(x, mu, sd) * scipy.stats.norm.cdf(x, mu, sd) ** (N - 1)
    v, _ = scipy.integrate.quad(f, mu - 12 * sd, mu + 12 * sd, epsabs=1e-13, epsrel=1e-12)
    return v


def pin_normal_max_quadrature(lib, order="rows"):
    """Eq. 3: f_T = N f F^(N-1).  E[max of N normals] by quadrature; N = 2 is mu + sd/sqrt(pi).
    With M micro-batches a worker's time is N(M mu, M sd^2) (sum of normals), so the same
    integral pins running sum and max together."""
    assert abs(_emax_normal(2, 1.0, 0.1) - (1.0 + 0.1 / math.sqrt(math.pi))) < 1e-10
    mu, sd = 1.0, 0.1
    for N, M, T, seed in ((2, 1, 60000, 3), (3, 1, 60000, 4), (5, 4, 40000, 5), (8, 9, 40000, 6)):
        lat = W.iid_latencies("normal", T, N, M, seed, mu=mu, sd=sd)
        sw, st = _stats(lib, lat, np.array([INF]), 0.25, order=order)
        want = _emax_normal(N, M * mu, math.sqrt(M) * sd) + 0.25
        tol = 5 * math.sqrt(M) * sd / math.sqrt(T) + 1e-6
        assert abs(st.baseline[0] - want) <= tol, (N, M, st.baseline[0], want)


def pin_done_frac_normal_eq5(lib, order="rows"):
    """Eq. 5 is exact when micro-batch latencies are iid normal:
    E[M~(tau)] = sum_m Phi((tau - m mu)/sqrt(m sd^2))."""
    mu, sd, N, M, T = 1.0, 0.15, 6, 8, 20000
    lat = W.iid_latencies("normal", T, N, M, 7, mu=mu, sd=sd)
    taus = np.linspace(3.0, 9.0, 13).astype(np.float32)
    sw, st = _stats(lib, lat, taus, 0.5, order=order)
    per_trial = sw.done.astype(np.float64) / (N * M)
    for k, tau in enumerate(taus.astype(np.float64)):
        want = sum(scipy.stats.norm.cdf((tau - m * mu) / (sd * math.sqrt(m))) for m in range(1, M + 1)) / M
        se = per_trial[:, k].std(ddof=1) / math.sqrt(T)
        assert abs(st.stats[1, k] - want) <= 5 * se + 2e-6, (k, st.stats[1, k], want, se)


def pin_done_frac_erlang(lib, order="rows"):
    """E[M~(tau)] = sum_m P(T_n^(m) < tau) (App. C.2); for c + Exp(mean b) micro-batches
    T_n^(m) - m c is Erlang(m, b)."""
    c, b, N, M, T = 0.1, 0.02, 8, 4, 30000
    lat = W.iid_latencies("shifted_exp", T, N, M, 8, shift=c, mean=b)
    taus = np.linspace(0.2, 0.6, 16).astype(np.float32)
    sw, st = _stats(lib, lat, taus, 0.05, order=order)
    per_trial = sw.done.astype(np.float64) / (N * M)
    for k, tau in enumerate(taus.astype(np.float64)):
        want = sum(scipy.stats.gamma.cdf(tau - m * c, a=m, scale=b) for m in range(1, M + 1)) / M
        se = per_trial[:, k].std(ddof=1) / math.sqrt(T)
        assert abs(st.stats[1, k] - want) <= 5 * se + 2e-6, (k, st.stats[1, k], want, se)


def pin_start_rule_memoryless(lib, order="rows"):
    """The start-before-tau rule (Limitations paragraph) on iid Exp(rate) micro-batches, one worker, more
    micro-batches than can start before the largest threshold.  Micro-batch m starts iff the m-fold sum before it is
    < tau, so the number started is 1 + (arrivals of a Poisson process of that rate before tau): mean 1 + rate*tau;
    and the worker's time is the first arrival at or after tau, which by memorylessness is tau + Exp(rate):
    mean tau + 1/rate, standard deviation 1/rate, always >= tau."""
    rate, M, T = 20.0, 64, 40000
    lat = W.iid_latencies("exp", T, 1, M, 17, rate=rate)
    taus = np.array([0.05, 0.2, 0.55, 1.0], np.float32)   # rate*tau up to 20, far below M = 64 micro-batches
    t_comm = 0.25
    sw, st = _stats(lib, lat, taus, t_comm, rule=1, order=order)
    assert (sw.step >= taus[None, :] + np.float32(t_comm) - 1e-6).all()
    for k, tau in enumerate(taus.astype(np.float64)):
        started = sw.done[:, k].astype(np.float64)
        want_n = 1.0 + rate * tau
        assert abs(started.mean() - want_n) <= 5 * math.sqrt(rate * tau / T) + 1e-9, (k, started.mean(), want_n)
        assert abs(started.var(ddof=1) - rate * tau) <= 0.05 * rate * tau + 0.02, (k, started.var(ddof=1))
        want_step = tau + 1.0 / rate + t_comm
        assert abs(st.stats[0, k] - want_step) <= 5 * (1.0 / rate) / math.sqrt(T), (k, st.stats[0, k], want_step)
        over = sw.step[:, k].astype(np.float64) - t_comm - tau
        assert abs(over.std(ddof=1) - 1.0 / rate) <= 0.03 / rate, (k, over.std(ddof=1))
    # the paper's rule on the same samples counts one fewer micro-batch whenever a threshold is crossed
    sw0, _ = _stats(lib, lat, taus, t_comm, rule=0, order=order)
    assert np.array_equal(sw.done, np.minimum(sw0.done + 1, M))


# --- exhaustive enumeration in rational arithmetic -----------------------------

def _enumerate_exact(values, N, M, taus, t_comm, rule):
    """All len(values)^(N*M) equally likely outcomes; returns exact per-outcome and mean quantities
    written directly from Sec. 4.3 / Eq. 6 (not from Algorithm 2's loops)."""
    outcomes = list(itertools.product(values, repeat=N * M))
    done, step, sync = [], [], []
    for o in outcomes:
        rows = [o[n * M:(n + 1) * M] for n in range(N)]
        finish = [list(itertools.accumulate(r)) for r in rows]           # T_n^(m)
        Tmax = max(f[-1] for f in finish)
        d_row, s_row = [], []
        for tau in taus:
            if rule == 0:
                d = sum(1 for f in finish for x in f if x < tau)
                s = min(tau, Tmax) + t_comm
            else:
                d, w = 0, Fraction(0)
                for f in finish:
                    start = [Fraction(0)] + f[:-1]
                    ran = [x for b, x in zip(start, f) if b < tau]
                    d += len(ran)
                    if ran:
                        w = max(w, ran[-1])
                s = w + t_comm
            d_row.append(d)
            s_row.append(s)
        done.append(d_row)
        step.append(s_row)
        sync.append(Tmax + t_comm)
    return outcomes, done, step, sync


def pin_enumeration(lib, order="rows"):
    """Tiny dyadic law {1/4, 1/2}: feeding every outcome once as the trials makes trial means exact
    expectations; thresholds include reachable sums (ties test '<' versus '<=')."""
    vals = [Fraction(1, 4), Fraction(1, 2)]
    t_comm = Fraction(1, 8)
    for (N, M), rule in itertools.product(((2, 3), (3, 2), (1, 4), (2, 2)), (0, 1)):
        taus = [Fraction(1, 8), Fraction(1, 4), Fraction(1, 2), Fraction(3, 4), Fraction(1), Fraction(5, 4),
                Fraction(3, 2), Fraction(7, 4), Fraction(2), Fraction(4)]
        outcomes, done, step, sync = _enumerate_exact(vals, N, M, taus, t_comm, rule)
        T = len(outcomes)
        lat = np.array([[float(x) for x in o] for o in outcomes], np.float32).reshape(T, N, M)
        taus_f = np.array([float(t) for t in taus], np.float32)
        sw, st = _stats(lib, lat, taus_f, float(t_comm), rule=rule, order=order)
        assert np.array_equal(sw.done, np.array(done, np.int32)), (N, M, rule)
        assert np.array_equal(sw.step, np.array([[float(x) for x in r] for r in step], np.float32)), (N, M, rule)
        assert np.array_equal(sw.sync, np.array([float(x) for x in sync], np.float32))
        NM = N * M
        for k in range(len(taus)):
            sd = sum(Fraction(d[k]) for d in done)
            ss = sum(s[k] for s in step)
            want = [ss / T, sd / (T * NM), sd / ss,
                    sum(Fraction(d[k]) / s[k] for d, s in zip(done, step)) / T,
                    sum((y / s[k]) * Fraction(d[k], NM) for d, s, y in zip(done, step, sync)) / T]
            for r in range(5):
                assert abs(st.stats[r, k] - float(want[r])) <= 1e-13 * max(1.0, abs(float(want[r]))), (N, M, rule, r, k)
        assert abs(st.baseline[0] - float(sum(sync) / T)) <= 1e-13
        assert abs(st.baseline[1] - float(Fraction(T * NM) / sum(sync))) <= 1e-12
        if rule == 0:
            exact_seff = [sum((y / s[k]) * Fraction(d[k], NM) for d, s, y in zip(done, step, sync)) / T
                          for k in range(len(taus))]
            k_first = max(range(len(taus)), key=lambda k: (exact_seff[k], -k))
            assert oracle.argmax(st.stats[4], lib=lib) == k_first


# --- hand-worked example and rounding order ------------------------------------

def _fr(x):
    return float(Fraction(x))


def pin_hand_example(lib, order="rows"):
    with open(os.path.join(GOLDEN, "alg2_hand_example.json")) as f:
        g = json.load(f)
    lat = np.array([[[_fr(x) for x in row] for row in it] for it in g["latencies"]], np.float32)
    taus = np.array([_fr(x) for x in g["taus"]], np.float32)
    tc = _fr(g["t_comm"])
    for rule in (0, 1):
        sw, st = _stats(lib, lat, taus, tc, rule=rule, order=order)
        want = g[f"rule{rule}"]
        assert np.array_equal(sw.done, np.array(want["done"], np.int32)), rule
        assert np.array_equal(sw.step, np.array([[_fr(x) for x in r] for r in want["step"]], np.float32)), rule
        assert np.array_equal(sw.sync, np.array([_fr(x) for x in g["sync"]], np.float32))
        if rule == 0:
            for r, name in enumerate(oracle.STAT_NAMES):
                ref = np.array([_fr(x) for x in want[name]])
                assert np.allclose(st.stats[r], ref, rtol=1e-14, atol=0), name
            assert oracle.argmax(st.stats[4], lib=lib) == want["k_star"]
            assert abs(st.baseline[0] - _fr(want["mean_sync"])) < 1e-15
            assert abs(st.baseline[1] - _fr(want["thr_sync"])) < 1e-14
            s_eff, k_star = oracle.s_eff_fractional(lat, taus, tc, lib=lib)
            assert np.allclose(s_eff, st.stats[4], rtol=1e-14) and k_star == want["k_star"]


def pin_per_iteration_comm(lib, order="rows"):
    """Algorithm 2 takes the communication time per iteration (T_i^c).  A vector of equal values is the
    scalar case bit for bit; with different values the hand-worked example changes only through
    min(tau, T_i) + T_i^c and (T_i + T_i^c) / (...), recomputed here in rational arithmetic."""
    with open(os.path.join(GOLDEN, "alg2_hand_example.json")) as f:
        g = json.load(f)
    lat = np.array([[[_fr(x) for x in row] for row in it] for it in g["latencies"]], np.float32)
    taus_q = [Fraction(x) for x in g["taus"]]
    taus = np.array([float(x) for x in taus_q], np.float32)
    T, N, M = lat.shape
    same = oracle.sweep(lat, taus, np.full(T, 0.25, np.float32), order=order, lib=lib)
    scal = oracle.sweep(lat, taus, 0.25, order=order, lib=lib)
    assert np.array_equal(same.step, scal.step) and np.array_equal(same.sync, scal.sync) and np.array_equal(same.done, scal.done)
    tc = [Fraction(1, 8), Fraction(1, 2), Fraction(1, 4)]
    tmax = [Fraction(x) - Fraction(g["t_comm"]) for x in g["sync"]]          # the example's T_i
    sw = oracle.sweep(lat, taus, np.array([float(x) for x in tc], np.float32), order=order, lib=lib)
    st = oracle.reduce_trials(sw.step, sw.done, sw.sync, N, M, lib=lib)
    done = g["rule0"]["done"]
    want_step = [[min(tau, tmax[i]) + tc[i] for tau in taus_q] for i in range(T)]
    assert np.array_equal(sw.step, np.array([[float(x) for x in r] for r in want_step], np.float32))
    assert np.array_equal(sw.sync, np.array([float(tmax[i] + tc[i]) for i in range(T)], np.float32))
    assert np.array_equal(sw.done, np.array(done, np.int32))
    for k in range(len(taus_q)):
        s_eff = sum((tmax[i] + tc[i]) / want_step[i][k] * Fraction(done[i][k], N * M) for i in range(T)) / T
        assert abs(st.stats[4, k] - float(s_eff)) <= 1e-14


def pin_fp32_left_to_right(lib, order="rows"):
    """The running sum is binary32 with one rounding per addition, taken m = 1..M in order
    (Algorithm 2's inner loop; the precision is a reading taken where the paper is silent)."""
    e = 2.0 ** -24
    nxt = np.float32(1.0 + 2.0 ** -23)
    # 1 + 2^-24 ties to even = 1, three times over: the sum never leaves 1.0
    lat = np.array([[[1.0, e, e, e]]], np.float32)
    sw = oracle.sweep(lat, np.array([1.0, nxt, INF], np.float32), 0.0, order=order, lib=lib)
    assert sw.done.tolist() == [[0, 4, 4]] and sw.sync[0] == np.float32(1.0)
    # same addends, the large one last: 3*2^-24 is exact, then 1 + 1.5 ulp ties to even = 1 + 2^-22
    lat = np.array([[[e, e, e, 1.0]]], np.float32)
    sw = oracle.sweep(lat, np.array([1.0, nxt, INF], np.float32), 0.0, order=order, lib=lib)
    assert sw.sync[0] == np.float32(1.0 + 2.0 ** -22) and sw.done.tolist() == [[3, 3, 4]]
    # cumulative sum in binary32 from numpy on random data (advisory third opinion)
    lat = _np(W.iid_latencies("uniform", 50, 7, 33, 9, lo=0.001, hi=0.3))
    P = np.cumsum(lat, axis=-1, dtype=np.float32)
    taus = np.sort(np.random.default_rng(0).uniform(0.0, 6.0, 40)).astype(np.float32)
    sw = oracle.sweep(lat, taus, 0.125, order=order, lib=lib)
    assert np.array_equal(sw.done, (P[..., None] < taus).sum(axis=(1, 2)).astype(np.int32))
    assert np.array_equal(sw.sync, P[..., -1].max(axis=1) + np.float32(0.125))


def pin_m1_sort(lib, order="rows"):
    """M = 1: the completed count at tau is the rank of tau among the sorted worker times and
    the synchronous time is their maximum (textbook routines on the same fp32 data)."""
    lat = _np(W.iid_latencies("uniform", 300, 37, 1, 10, lo=0.0, hi=1.0))
    taus = np.concatenate([np.linspace(-0.1, 1.1, 25), lat[0, :5, 0]]).astype(np.float32)
    taus.sort()
    sw = oracle.sweep(lat, taus, 0.5, order=order, lib=lib)
    for t in range(lat.shape[0]):
        s = np.sort(lat[t, :, 0])
        assert np.array_equal(sw.done[t], np.searchsorted(s, taus, side="left").astype(np.int32))
        assert sw.sync[t] == s[-1] + np.float32(0.5)
        assert np.array_equal(sw.step[t], np.minimum(taus, s[-1]) + np.float32(0.5))


# --- invariants ---------------------------------------------------------------------

def pin_invariants(lib, order="rows"):
    rng = np.random.default_rng(11)
    for (T, N, M), law in (((40, 9, 12), "shifted_exp"), ((25, 33, 5), "dyadic"), ((10, 1, 1), "uniform")):
        p = dict(shift=0.1, mean=0.05) if law == "shifted_exp" else dict(hi=40) if law == "dyadic" else dict(lo=0, hi=1)
        lat = _np(W.iid_latencies(law, T, N, M, 12, **p))
        tot = lat.sum(-1).max()
        taus = np.sort(rng.uniform(-0.2, 1.3 * tot, 23)).astype(np.float32)
        taus = np.concatenate([taus, [taus[5], INF]]).astype(np.float32)
        taus.sort()
        K = taus.shape[0]
        tc = np.float32(0.3)
        for rule in (0, 1):
            sw = oracle.sweep(lat, taus, tc, rule=rule, order=order, lib=lib)
            assert (np.diff(sw.done.astype(np.int64), axis=1) >= 0).all()
            assert (np.diff(sw.step, axis=1) >= 0).all()
            assert (sw.done >= 0).all() and (sw.done <= N * M).all()
            P = np.cumsum(lat, axis=-1, dtype=np.float32)
            tmax = P[..., -1].max(axis=1)
            above = taus[None, :] > tmax[:, None]
            assert (sw.done[above] == N * M).all()
            assert (sw.step[above] == np.broadcast_to(sw.sync[:, None], (T, K))[above]).all()
            assert (sw.step[:, -1] == sw.sync).all() and (sw.done[:, -1] == N * M).all()  # tau = inf
            if rule == 0:
                assert (sw.step <= (taus[None, :] + tc)).all()
            else:
                # step <= tau + the micro-batch that was running when tau passed
                nonneg = taus >= 0
                assert (sw.step[:, nonneg] <= (taus[None, nonneg] + lat.max() + tc) * (1 + 1e-6)).all()
            assert (sw.step[:, taus >= 0] >= tc).all()
            # per-worker decisions: each worker as its own one-worker trial
            per = oracle.sweep(lat.reshape(T * N, 1, M), taus, tc, rule=rule, order=order, lib=lib)
            assert np.array_equal(per.done.reshape(T, N, K).sum(1), sw.done)
            assert (per.done <= M).all()
            assert np.array_equal(per.step.reshape(T, N, K).max(1), sw.step)
            if rule == 1:
                base = oracle.sweep(lat.reshape(T * N, 1, M), taus, tc, rule=0, order=order, lib=lib)
                want = np.where(taus[None, :] > 0, np.minimum(M, base.done + 1), 0)
                assert np.array_equal(per.done, want.astype(np.int32))
            # permuting workers changes nothing; permuting trials permutes rows
            pw = rng.permutation(N)
            pt = rng.permutation(T)
            sw2 = oracle.sweep(lat[:, pw][pt], taus, tc, rule=rule, order=order, lib=lib)
            assert np.array_equal(sw2.done, sw.done[pt]) and np.array_equal(sw2.step, sw.step[pt])
            assert np.array_equal(sw2.sync, sw.sync[pt])
            # dropping columns of the grid leaves the others unchanged
            sub = oracle.sweep(lat, taus[3:-1], tc, rule=rule, order=order, lib=lib)
            assert np.array_equal(sub.done, sw.done[:, 3:-1]) and np.array_equal(sub.step, sw.step[:, 3:-1])


def pin_argmax(lib, order="rows"):
    nan = float("nan")
    assert oracle.argmax([1.0, 3.0, 3.0, 2.0], lib=lib) == 1
    assert oracle.argmax([nan, 1.0, nan, 1.0], lib=lib) == 1
    assert oracle.argmax([nan, nan], lib=lib) == -1
    assert oracle.argmax([-1.0], lib=lib) == 0
    assert oracle.argmax([0.5, nan, 0.7, 0.7], lib=lib) == 2


def pin_definition_equals_rows(lib, order=None):
    rng = np.random.default_rng(13)
    for T, N, M, K in ((7, 5, 9, 11), (3, 1, 1, 1), (4, 17, 2, 30), (2, 3, 40, 6)):
        lat = _np(W.iid_latencies("shifted_exp", T, N, M, 14, shift=0.05, mean=0.03))
        taus = np.sort(rng.uniform(0, 1.2 * lat.sum(-1).max(), K)).astype(np.float32)
        for rule in (0, 1):
            a = oracle.sweep(lat, taus, 0.07, rule=rule, order="definition", lib=lib)
            b = oracle.sweep(lat, taus, 0.07, rule=rule, order="rows", lib=lib)
            assert np.array_equal(a.done, b.done) and np.array_equal(a.step, b.step) and np.array_equal(a.sync, b.sync)
        s_eff, k_star = oracle.s_eff_fractional(lat, taus, 0.07, lib=lib)
        sw0 = oracle.sweep(lat, taus, 0.07, rule=0, order="rows", lib=lib)
        st = oracle.reduce_trials(sw0.step, sw0.done, sw0.sync, N, M, lib=lib)
        assert np.allclose(s_eff, st.stats[4], rtol=1e-12, atol=0)
        assert k_star == oracle.argmax(st.stats[4], lib=lib)
    # neither form assumes that running sums grow: with negative "latencies" (outside the simulator's
    # contract, inside the definitions') they still agree, under both rules
    lat = _np(W.iid_latencies("normal", 6, 4, 7, 19, mu=0.02, sd=0.05))
    assert (lat < 0).any()
    taus = np.sort(rng.uniform(-0.1, 0.4, 9)).astype(np.float32)
    for rule in (0, 1):
        a = oracle.sweep(lat, taus, 0.07, rule=rule, order="definition", lib=lib)
        b = oracle.sweep(lat, taus, 0.07, rule=rule, order="rows", lib=lib)
        assert np.array_equal(a.done, b.done) and np.array_equal(a.step, b.step) and np.array_equal(a.sync, b.sync)


def pin_independence_and_bailey(lib, order="rows"):
    """Loose plausibility: E[M~ T] is close to E[M~] E[T] for many workers (App. C.2), and the
    Bailey approximation (Eq. 4) lands within a few percent of the simulated E[T] for normal totals."""
    mu, sd, N, M, T = 0.025, 0.004, 400, 16, 400
    lat = W.iid_latencies("normal", T, N, M, 15, mu=mu, sd=sd)
    tau = np.array([M * mu * 1.02], np.float32)
    sw, st = _stats(lib, lat, tau, 0.0, order=order)
    mt = sw.done[:, 0] / N
    tm = sw.sync.astype(np.float64)
    assert abs((mt * tm).mean() - mt.mean() * tm.mean()) <= 0.01 * mt.mean() * tm.mean()
    g = 0.5772156649015329
    z = (1 - g) * scipy.stats.norm.ppf(1 - 1 / N) + g * scipy.stats.norm.ppf(1 - 1 / (math.e * N))
    bailey = math.sqrt(M) * sd * z + M * mu
    assert abs(st.baseline[0] - bailey) <= 0.03 * bailey


def pin_bailey_against_quadrature(lib, order="rows"):
    """Eq. 4 approximates E[max of N standard normals]; Eq. 3 gives that expectation exactly as the integral of
    x N f F^(N-1).  The approximation lies ABOVE the exact value by less than one percent for N >= 100 and comes
    closer as N grows (0.92 %, 0.56 %, 0.35 %, 0.23 % at N = 100, 400, 2048, 10000), whereas exchanging its two
    weights puts it about one percent BELOW: a one-sided band tells the two apart.  mu and sigma scale it."""
    prev = None
    for N in (100, 400, 2048, 10000):
        exact = _emax_normal(N, 0.0, 1.0)
        z = oracle.bailey_mean_max(0.0, 1.0, 1, N, lib=lib)
        assert exact < z < 1.01 * exact, (N, z, exact)
        if prev is not None:
            assert z / exact < prev, (N, z / exact, prev)
        prev = z / exact
    # sqrt(M sigma^2) z + M mu
    z = oracle.bailey_mean_max(0.0, 1.0, 1, 400, lib=lib)
    assert abs(oracle.bailey_mean_max(0.5, 0.2, 9, 400, lib=lib) - (0.6 * z + 4.5)) <= 1e-12


def pin_worker_scales(lib, order="rows"):
    """Heterogeneous workers (App. C.2: workers may differ): worker n works against its own threshold s_n tau_k, its
    time is min{s_n tau_k, T_n} (Sec. 4.3, per worker) and the step is the slowest worker's time plus T^c.
    Exhaustive enumeration in rational arithmetic with dyadic scales (every product exact), the all-ones case equal
    to the common-threshold code bit for bit, and a worker whose latencies and scale are both doubled keeps its
    decisions."""
    vals = [Fraction(1, 4), Fraction(1, 2)]
    t_comm = Fraction(1, 8)
    taus = [Fraction(-1, 4), Fraction(1, 8), Fraction(1, 4), Fraction(1, 2), Fraction(3, 4), Fraction(1), Fraction(3, 2), Fraction(4)]
    for (N, M, scales), rule in itertools.product((((2, 3, (Fraction(1), Fraction(1, 2)))), (3, 2, (Fraction(2), Fraction(1), Fraction(1, 2))),
                                                   (1, 3, (Fraction(1, 2),))), (0, 1)):
        outcomes = list(itertools.product(vals, repeat=N * M))
        T = len(outcomes)
        want_done, want_step = [], []
        for o in outcomes:
            finish = [list(itertools.accumulate(o[n * M:(n + 1) * M])) for n in range(N)]
            d_row, s_row = [], []
            for tau in taus:
                d, times = 0, []
                for n, f in enumerate(finish):
                    own = scales[n] * tau
                    if rule == 0:
                        d += sum(1 for x in f if x < own)
                        times.append(min(own, f[-1]))
                    else:
                        start = [Fraction(0)] + f[:-1]
                        ran = [x for b, x in zip(start, f) if b < own]
                        d += len(ran)
                        times.append(ran[-1] if ran else Fraction(0))
                d_row.append(d)
                s_row.append(max(times) + t_comm)
            want_done.append(d_row)
            want_step.append(s_row)
        lat = np.array([[float(x) for x in o] for o in outcomes], np.float32).reshape(T, N, M)
        taus_f = np.array([float(t) for t in taus], np.float32)
        sc = np.array([float(x) for x in scales], np.float32)
        sw = oracle.sweep(lat, taus_f, float(t_comm), rule=rule, order=order, lib=lib, worker_scale=sc)
        assert np.array_equal(sw.done, np.array(want_done, np.int32)), (N, M, rule)
        assert np.array_equal(sw.step, np.array([[float(x) for x in r] for r in want_step], np.float32)), (N, M, rule)
    # all scales one: the common-threshold results, bit for bit; and the synchronous time never depends on the scales
    rng = np.random.default_rng(23)
    lat = _np(W.iid_latencies("shifted_exp", 9, 7, 6, 24, shift=0.05, mean=0.03))
    taus_f = np.sort(rng.uniform(-0.1, 1.2 * lat.sum(-1).max(), 13)).astype(np.float32)
    for rule in (0, 1):
        a = oracle.sweep(lat, taus_f, 0.07, rule=rule, order=order, lib=lib)
        b = oracle.sweep(lat, taus_f, 0.07, rule=rule, order=order, lib=lib, worker_scale=np.ones(7, np.float32))
        assert np.array_equal(a.done, b.done) and np.array_equal(a.step, b.step) and np.array_equal(a.sync, b.sync)
        # worker 3 twice as slow and given twice the threshold: its own decisions do not change (powers of two are exact)
        sc = rng.uniform(0.5, 1.5, 7).astype(np.float32)
        one = oracle.sweep(lat[:, 3:4], taus_f, 0.07, rule=rule, order=order, lib=lib, worker_scale=sc[3:4])
        lat2, sc2 = lat.copy(), sc.copy()
        lat2[:, 3] *= 2.0
        sc2[3] *= 2.0
        two = oracle.sweep(lat2[:, 3:4], taus_f, 0.07, rule=rule, order=order, lib=lib, worker_scale=sc2[3:4])
        assert np.array_equal(one.done, two.done)
        c = oracle.sweep(lat, taus_f, 0.07, rule=rule, order=order, lib=lib, worker_scale=sc)
        assert np.array_equal(c.sync, a.sync)
        # the counts are the sum of the workers' own counts
        per = sum(oracle.sweep(lat[:, n:n + 1], taus_f, 0.07, rule=rule, order=order, lib=lib, worker_scale=sc[n:n + 1]).done
                  for n in range(7))
        assert np.array_equal(per, c.done)


def pin_closed_form(lib, order="rows"):
    """App. C.2: Phi and Phi^-1 against scipy, Eq. 4/12, Eq. 5/10, Eq. 11 and the analytic tau*; then the
    closed forms against the simulator itself where they are exact (normal micro-batches: Eq. 5) or good
    to a few percent (Bailey's E[max])."""
    g = 0.5772156649015329
    for mu, sd, M, N in ((1.0, 0.1, 16, 400), (0.675, math.sqrt(0.05), 12, 1000), (0.03, 0.004, 64, 2)):
        z = (1 - g) * scipy.stats.norm.ppf(1 - 1 / N) + g * scipy.stats.norm.ppf(1 - 1 / (math.e * N))
        want = math.sqrt(M) * sd * z + M * mu
        assert abs(oracle.bailey_mean_max(mu, sd, M, N, lib=lib) - want) <= 1e-12 * want
        taus = np.linspace(0.4 * M * mu, 1.4 * M * mu, 41).astype(np.float32)
        tc = 0.3 * mu
        cf = oracle.closed_form(mu, sd, M, N, tc, taus, lib=lib)
        assert abs(cf.mean_T - want) <= 1e-12 * want
        t64 = taus.astype(np.float64)
        em = sum(scipy.stats.norm.cdf((t64 - m * mu) / (sd * math.sqrt(m))) for m in range(1, M + 1)) / M
        assert np.allclose(cf.done_frac, em, rtol=1e-12, atol=1e-15)
        assert np.allclose(cf.step, np.minimum(t64, want) + tc, rtol=1e-14)
        assert np.allclose(cf.s_eff, em * (want + tc) / (np.minimum(t64, want) + tc), rtol=1e-12)
        assert cf.k_star == int(np.argmax(cf.s_eff)) and cf.tau_star == float(taus[cf.k_star])
        # a threshold far above everything: nothing dropped, no speedup
        far = oracle.closed_form(mu, sd, M, N, tc, np.array([100 * M * mu], np.float32), lib=lib)
        assert abs(far.s_eff[0] - 1.0) < 1e-12 and abs(far.done_frac[0] - 1.0) < 1e-12
        # a measured E[T] replaces Eq. 12
        given = oracle.closed_form(mu, sd, M, N, tc, taus, mean_T=1.1 * want, lib=lib)
        assert given.mean_T == 1.1 * want and np.allclose(given.done_frac, cf.done_frac, rtol=0, atol=0)
        assert np.allclose(given.s_eff, em * (1.1 * want + tc) / (np.minimum(t64, 1.1 * want) + tc), rtol=1e-12)
    # against the simulator: normal micro-batches, many workers
    mu, sd, N, M, T = 0.025, 0.004, 300, 16, 500
    lat = W.iid_latencies("normal", T, N, M, 21, mu=mu, sd=sd)
    taus = np.linspace(0.8 * M * mu, 1.3 * M * mu, 11).astype(np.float32)
    sw, st = _stats(lib, lat, taus, 0.05, order=order)
    cf = oracle.closed_form(mu, sd, M, N, 0.05, taus, lib=lib)
    assert np.allclose(st.stats[1], cf.done_frac, rtol=0, atol=2e-3)                    # Eq. 5 is exact here
    assert abs(st.baseline[0] - 0.05 - cf.mean_T) <= 0.03 * cf.mean_T                   # Bailey: a few percent
    given = oracle.closed_form(mu, sd, M, N, 0.05, taus, mean_T=st.baseline[0] - 0.05, lib=lib)
    assert np.allclose(st.stats[4], given.s_eff, rtol=0.02)                             # Eq. 11 with measured E[T]


ALL_PINS = (
    pin_exp_max_harmonic, pin_normal_max_quadrature, pin_done_frac_normal_eq5, pin_done_frac_erlang,
    pin_enumeration, pin_hand_example, pin_per_iteration_comm, pin_fp32_left_to_right, pin_m1_sort, pin_invariants, pin_argmax,
    pin_definition_equals_rows, pin_independence_and_bailey, pin_bailey_against_quadrature, pin_closed_form,
    pin_start_rule_memoryless, pin_worker_scales,
)
# a quick subset that still kills every planted mistake (used by the mutation test)
FAST_PINS = (pin_worker_scales, pin_hand_example, pin_per_iteration_comm, pin_enumeration, pin_fp32_left_to_right, pin_m1_sort, pin_argmax,
             pin_bailey_against_quadrature, pin_closed_form, pin_invariants, pin_exp_max_harmonic)
