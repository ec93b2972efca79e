/*
 * CPU oracle for the DropCompute threshold sweep.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the simulator computes.  It
 * exists so that tests, the smoke check and the benchmark's CPU-baseline leg
 * can compare the CUDA library against it.  Nothing in the product path may
 * include, link or call it, and it shares no code with the CUDA sources.
 *
 * What is stated here (paper: DropCompute, arXiv 2306.10598):
 *   - Sec. 4.3: a worker's finish times T_n^{(m)} (inclusive running sums), the
 *     completed micro-batches M~ (those with T_n^{(m)} < tau, strict) and the
 *     DropCompute step time min{tau, T} + T^c with T = max_n T_n^{(M)}.
 *   - Algorithm 2, App. C.1 (the automatic choice of tau): what it evaluates per
 *     candidate tau and measured iteration (the quantities above), the
 *     per-iteration speedup S_i(tau), its mean S_eff(tau), and tau* = arg max.
 *   - Sec. 4.4, Eq. 6: effective speedup and throughput N*M~ / (min{tau,T}+T^c).
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   - samples, running sums, comparisons and step times are IEEE binary32;
 *     one rounding per addition, micro-batches strictly in the order m=1..M;
 *   - M~ is kept as the integer number of completed micro-batches summed over
 *     workers (the paper averages over workers in floating point; the integer
 *     count divided once at the end is the same number in exact arithmetic);
 *   - T^c is given per iteration as in Algorithm 2, or as one scalar used for all iterations;
 *   - statistics over iterations are binary64;
 *   - argmax takes the first maximum and never selects a NaN.
 *
 * Heterogeneous workers (App. C.2 remarks that workers may differ, each with its own mu_n, sigma_n): optionally
 * worker n works against its own threshold s_n * tau_k (one binary32 product) instead of the common tau_k; its time
 * is then min{s_n tau_k, T_n} and the step takes the maximum of those over workers.  With all s_n = 1 this is the
 * common-threshold case bit for bit.
 *
 * rule 0 is the paper's (a micro-batch counts iff it FINISHES before tau).
 * rule 1 is the variant described in the paper's Limitations paragraph, where
 * the timeout is only looked at between accumulations: a micro-batch is run
 * iff it STARTS before tau, and a worker's time is the finish time of the
 * last micro-batch it ran.
 *
 * Pins (tests/test_oracle_pins.py and friends): harmonic-number mean of the
 * max of exponentials, quadrature of Eq. 3 for normals (which also bounds
 * Eq. 4's approximation from one side), Eq. 5 (exact for
 * normal micro-batches), Erlang CDF for shifted exponentials, exhaustive
 * enumeration of tiny dyadic laws in rational arithmetic, a hand-worked
 * example, M=1 against sort/searchsorted, invariants, and mutation checks.
 * Parity unpinned: none of the paper's printed E[T]/E[T_i] table values pins
 * this code firmly (the worker count behind them is not printed); they are
 * used as a loose plausibility band only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DCO_NSTATS 5 /* mean_step, done_frac, thr, thr_mean, s_eff */

/* ---------------------------------------------------------------------------
 * The per-(iteration, tau) quantities straight from their definitions in Sec. 4.3.
 * For every iteration the table of finish times T_n^{(m)} = sum_{j<=m} t_n^{(j)}
 * is written out first; everything else is read off that table, one threshold
 * at a time:
 *   completed micro-batches   N * M~(tau) = #{(n,m) : T_n^{(m)} < tau}
 *   slowest worker            T = max_n T_n^{(M)}
 *   step time                 min{tau, T} + T^c
 * This is also what Algorithm 2 (App. C.1) evaluates for each candidate tau.
 *   lat      [T,N,M] binary32, m fastest
 *   taus     [K]
 *   out_step [T,K]  step time
 *   out_done [T,K]  N * M~_i(tau) as an integer
 *   out_sync [T]    T_i + T^c   (the tau = infinity step time)
 *   t_comm_per_iter [T] or NULL: Algorithm 2's input T_i^c, one value per iteration; when this is
 *                   NULL the one scalar t_comm is used for every iteration.
 * rule 1 (Limitations paragraph): micro-batch m starts at T_n^{(m-1)} (0 for the first) and is run
 * iff that is < tau; the worker's time is the finish time of the last micro-batch it ran, and the
 * step time is the slowest worker's time plus T^c.
 * ------------------------------------------------------------------------- */
int dco_sweep_definition(const float *lat, int64_t T, int64_t N, int64_t M,
                         const float *taus, int64_t K, float t_comm, const float *t_comm_per_iter, int rule,
                         const float *worker_scale, float *out_step, int32_t *out_done, float *out_sync)
{
    if (!lat || !taus || !out_step || !out_done || !out_sync) return 1;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return 2;
    if (rule != 0 && rule != 1) return 7;
    float *finish = (float *)malloc((size_t)N * (size_t)M * sizeof(float));
    if (!finish) return 6;
    for (int64_t i = 0; i < T; ++i) {
        const float tc = t_comm_per_iter ? t_comm_per_iter[i] : t_comm;
        /* finish times: binary32, one rounding per addition, micro-batches in order */
        for (int64_t n = 0; n < N; ++n) {
            const float *row = lat + (i * N + n) * M;
            float elapsed = 0.0f;
            for (int64_t m = 0; m < M; ++m) {
                elapsed = elapsed + row[m];
                finish[n * M + m] = elapsed;
            }
        }
        float slowest_full = 0.0f; /* T = max_n T_n^{(M)} */
        for (int64_t n = 0; n < N; ++n) slowest_full = fmaxf(slowest_full, finish[n * M + (M - 1)]);
        out_sync[i] = slowest_full + tc;
        for (int64_t k = 0; k < K && worker_scale; ++k) {
            /* heterogeneous workers: worker n works against its own threshold s_n * tau_k (one binary32 product) */
            int64_t completed = 0;
            float slowest = 0.0f; /* max_n of the worker's time under its threshold */
            for (int64_t n = 0; n < N; ++n) {
                const float *f = finish + n * M;
                const float own_tau = worker_scale[n] * taus[k];
                float worker_time;
                if (rule == 0) {
                    for (int64_t m = 0; m < M; ++m) completed += (f[m] < own_tau) ? 1 : 0;
                    worker_time = fminf(own_tau, f[M - 1]); /* min{tau, T_n} of Sec. 4.3, per worker */
                } else {
                    int64_t last_run = -1;
                    for (int64_t m = 0; m < M; ++m) {
                        const float start = (m == 0) ? 0.0f : f[m - 1];
                        if (start < own_tau) {
                            completed += 1;
                            last_run = m;
                        }
                    }
                    worker_time = last_run >= 0 ? f[last_run] : 0.0f;
                }
                slowest = (n == 0) ? worker_time : fmaxf(slowest, worker_time);
            }
            out_done[i * K + k] = (int32_t)completed;
            out_step[i * K + k] = slowest + tc;
        }
        for (int64_t k = 0; k < K && !worker_scale; ++k) {
            const float tau = taus[k];
            int64_t completed = 0;
            float slowest_cut = 0.0f; /* rule 1: max_n (finish time of the last micro-batch worker n ran) */
            for (int64_t n = 0; n < N; ++n) {
                const float *f = finish + n * M;
                if (rule == 0) {
                    for (int64_t m = 0; m < M; ++m) completed += (f[m] < tau) ? 1 : 0;
                } else {
                    int64_t last_run = -1;
                    for (int64_t m = 0; m < M; ++m) {
                        const float start = (m == 0) ? 0.0f : f[m - 1];
                        if (start < tau) {
                            completed += 1;
                            last_run = m;
                        }
                    }
                    slowest_cut = fmaxf(slowest_cut, last_run >= 0 ? f[last_run] : 0.0f);
                }
            }
            out_done[i * K + k] = (int32_t)completed;
            out_step[i * K + k] = (rule == 0) ? (fminf(tau, slowest_full) + tc) : (slowest_cut + tc);
        }
    }
    free(finish);
    return 0;
}

/* ---------------------------------------------------------------------------
 * The same quantities in one pass over the samples: iteration, worker,
 * micro-batch, tau.  The predicate evaluated for every (i,n,m,k) is the same
 * and the counts are integers, so no output bit can differ from the form
 * above; this one reads the samples once and is used on large inputs.
 * Under rule 1 each worker keeps, per threshold, the finish time of the last
 * micro-batch it ran; the step takes the maximum of those over workers.
 * Iterations are independent and are spread over OpenMP threads.
 * ------------------------------------------------------------------------- */
int dco_sweep_rows(const float *lat, int64_t T, int64_t N, int64_t M,
                   const float *taus, int64_t K, float t_comm, const float *t_comm_per_iter, int rule,
                   const float *worker_scale, float *out_step, int32_t *out_done, float *out_sync)
{
    if (!lat || !taus || !out_step || !out_done || !out_sync) return 1;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return 2;
    if (rule != 0 && rule != 1) return 7;
    int failed = 0;
#pragma omp parallel
    {
        int64_t *cnt = (int64_t *)malloc((size_t)K * sizeof(int64_t));
        float *wmax = (float *)malloc((size_t)K * sizeof(float));   /* rule 1: slowest worker's time per threshold */
        float *wlast = (float *)malloc((size_t)K * sizeof(float));  /* rule 1: this worker's time per threshold */
        float *own = (float *)malloc((size_t)K * sizeof(float));    /* heterogeneous workers: this worker's thresholds */
        if (!cnt || !wmax || !wlast || !own) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < T; ++i) {
            if (!cnt || !wmax || !wlast || !own) continue;
            const float tc = t_comm_per_iter ? t_comm_per_iter[i] : t_comm;
            float slowest_full = 0.0f;
            for (int64_t k = 0; k < K; ++k) { cnt[k] = 0; wmax[k] = 0.0f; }
            for (int64_t n = 0; n < N && worker_scale; ++n) {
                /* heterogeneous workers: worker n against its own thresholds s_n * tau_k; wmax[k] collects the
                 * maximum over workers of each worker's time under its threshold (both rules) */
                const float *row = lat + (i * N + n) * M;
                float elapsed = 0.0f;
                for (int64_t k = 0; k < K; ++k) { own[k] = worker_scale[n] * taus[k]; wlast[k] = 0.0f; }
                for (int64_t m = 0; m < M; ++m) {
                    const float start = elapsed;
                    elapsed = elapsed + row[m];
                    for (int64_t k = 0; k < K; ++k) {
                        if (rule == 0) {
                            cnt[k] += (elapsed < own[k]) ? 1 : 0;
                        } else if (start < own[k]) {
                            cnt[k] += 1;
                            wlast[k] = elapsed;
                        }
                    }
                }
                slowest_full = fmaxf(slowest_full, elapsed);
                for (int64_t k = 0; k < K; ++k) {
                    const float worker_time = (rule == 0) ? fminf(own[k], elapsed) : wlast[k];
                    wmax[k] = (n == 0) ? worker_time : fmaxf(wmax[k], worker_time);
                }
            }
            for (int64_t n = 0; n < N && !worker_scale; ++n) {
                const float *row = lat + (i * N + n) * M;
                float elapsed = 0.0f;
                if (rule == 1) for (int64_t k = 0; k < K; ++k) wlast[k] = 0.0f;
                for (int64_t m = 0; m < M; ++m) {
                    if (rule == 0) {
                        elapsed = elapsed + row[m];
                        for (int64_t k = 0; k < K; ++k) cnt[k] += (elapsed < taus[k]) ? 1 : 0;
                    } else {
                        const float start = elapsed;
                        elapsed = elapsed + row[m];
                        for (int64_t k = 0; k < K; ++k) {
                            if (start < taus[k]) {
                                cnt[k] += 1;
                                wlast[k] = elapsed;
                            }
                        }
                    }
                }
                slowest_full = fmaxf(slowest_full, elapsed);
                if (rule == 1) for (int64_t k = 0; k < K; ++k) wmax[k] = fmaxf(wmax[k], wlast[k]);
            }
            out_sync[i] = slowest_full + tc;
            for (int64_t k = 0; k < K; ++k) {
                if (worker_scale)
                    out_step[i * K + k] = wmax[k] + tc;
                else
                    out_step[i * K + k] = (rule == 0) ? (fminf(taus[k], slowest_full) + tc) : (wmax[k] + tc);
                out_done[i * K + k] = (int32_t)cnt[k];
            }
        }
        free(cnt);
        free(wmax);
        free(wlast);
        free(own);
    }
    return failed ? 6 : 0;
}

/* ---------------------------------------------------------------------------
 * Reduction over iterations, binary64 (Algorithm 2: S_i(tau) and its mean;
 * Eq. 6; Sec. 4.4 throughput).  For every tau_k:
 *   stats[0][k] mean_step  = (1/T) sum_i step[i,k]
 *   stats[1][k] done_frac  = sum_i done[i,k] / (T*N*M)
 *   stats[2][k] thr        = sum_i done[i,k] / sum_i step[i,k]      micro-batches per second
 *   stats[3][k] thr_mean   = (1/T) sum_i done[i,k]/step[i,k]
 *   stats[4][k] s_eff      = (1/T) sum_i (sync[i]/step[i,k]) * done[i,k]/(N*M)
 * baseline[0] mean_sync = (1/T) sum_i sync[i];  baseline[1] thr_sync = T*N*M / sum_i sync[i].
 * ------------------------------------------------------------------------- */
int dco_reduce_trials(const float *step, const int32_t *done, const float *sync,
                      int64_t T, int64_t K, int64_t N, int64_t M,
                      double *stats, double *baseline)
{
    if (!step || !done || !sync || !stats || !baseline) return 1;
    if (T <= 0 || K <= 0 || N <= 0 || M <= 0) return 2;
    const double NM = (double)N * (double)M;
    for (int64_t k = 0; k < K; ++k) {
        double sum_step = 0.0, sum_ratio = 0.0, sum_S = 0.0;
        int64_t sum_done = 0;
        for (int64_t i = 0; i < T; ++i) {
            const double st = (double)step[i * K + k];
            const double dn = (double)done[i * K + k];
            sum_step += st;
            sum_done += done[i * K + k];
            sum_ratio += dn / st;
            sum_S += ((double)sync[i] / st) * (dn / NM);
        }
        stats[0 * K + k] = sum_step / (double)T;
        stats[1 * K + k] = (double)sum_done / ((double)T * NM);
        stats[2 * K + k] = (double)sum_done / sum_step;
        stats[3 * K + k] = sum_ratio / (double)T;
        stats[4 * K + k] = sum_S / (double)T;
    }
    double sum_sync = 0.0;
    for (int64_t i = 0; i < T; ++i) sum_sync += (double)sync[i];
    baseline[0] = sum_sync / (double)T;
    baseline[1] = ((double)T * NM) / sum_sync;
    return 0;
}

/* tau* = argmax_tau objective(tau): first index attaining the maximum; a NaN
 * never wins; returns -1 if every entry is NaN. */
int64_t dco_argmax(const double *objective, int64_t K)
{
    int64_t best = -1;
    for (int64_t k = 0; k < K; ++k) {
        const double v = objective[k];
        if (v != v) continue;
        if (best < 0 || v > objective[best]) best = k;
    }
    return best;
}

/* ---------------------------------------------------------------------------
 * S_eff(tau) with M~ taken as a floating-point mean over workers, the way
 * Sec. 4.3 writes it: M~_i(tau) = (1/N) sum_n c_n, c_n = #{m : T_n^{(m)} < tau},
 * accumulated in binary64 one worker at a time; then Eq. 6 per iteration,
 *   S_i(tau) = (M~_i / M) * (T_i + T^c) / (min{tau, T_i} + T^c),
 * the mean over iterations, and the first maximum.  Exists only so that a test can
 * show that keeping N * M~ as an integer (the reading used everywhere else in this
 * file) gives the same S_eff and the same tau*.
 * ------------------------------------------------------------------------- */
int dco_s_eff_fractional(const float *lat, int64_t T, int64_t N, int64_t M,
                         const float *taus, int64_t K, float t_comm,
                         double *s_eff, int64_t *k_star)
{
    if (!lat || !taus || !s_eff || !k_star) return 1;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return 2;
    float *total = (float *)malloc((size_t)N * sizeof(float));
    int64_t *c = (int64_t *)malloc((size_t)N * sizeof(int64_t));
    if (!total || !c) { free(total); free(c); return 6; }
    for (int64_t k = 0; k < K; ++k) s_eff[k] = 0.0;
    for (int64_t i = 0; i < T; ++i) {
        for (int64_t k = 0; k < K; ++k) {
            const float tau = taus[k];
            for (int64_t n = 0; n < N; ++n) {
                const float *row = lat + (i * N + n) * M;
                float elapsed = 0.0f;
                c[n] = 0;
                for (int64_t m = 0; m < M; ++m) {
                    elapsed = elapsed + row[m];
                    c[n] += (elapsed < tau) ? 1 : 0;
                }
                total[n] = elapsed;
            }
            double m_tilde = 0.0;
            float slowest = 0.0f;
            for (int64_t n = 0; n < N; ++n) {
                m_tilde += (double)c[n] / (double)N;
                slowest = fmaxf(slowest, total[n]);
            }
            const double sync_time = (double)(slowest + t_comm);
            const double drop_time = (double)(fminf(tau, slowest) + t_comm);
            s_eff[k] += (m_tilde / (double)M) * (sync_time / drop_time);
        }
    }
    for (int64_t k = 0; k < K; ++k) s_eff[k] /= (double)T;
    free(total);
    free(c);
    *k_star = dco_argmax(s_eff, K);
    return 0;
}

/* ===========================================================================
 * Closed-form companion (App. C.2): what the paper derives from the mean mu and
 * variance sigma^2 of one micro-batch latency alone.
 *
 *   Phi        standard normal CDF, here 0.5 erfc(-x / sqrt 2)
 *   Phi^-1     its inverse; libm has none, so it is found by bisection on Phi
 *   Eq. 4 / 12 E[T] ~ sqrt(M sigma^2) ((1-g) Phi^-1(1 - 1/N) + g Phi^-1(1 - 1/(e N))) + M mu,
 *              g the Euler-Mascheroni constant.  Eq. 12 as printed also adds T^c; here T
 *              never contains T^c (the paper adds it separately in Eq. 6, Eq. 11 and Algorithm 2).
 *   Eq. 5 / 10 E[M~(tau)] ~ sum_{m=1..M} Phi((tau - m mu) / sqrt(m sigma^2))
 *   Eq. 11     E[S_eff(tau)] ~ (E[M~]/M) (E[T] + T^c) / (min(tau, E[T]) + T^c)     (numerator as in Eq. 6)
 *   tau*       arg max over the grid of Eq. 11 (first maximum)
 * mean_T >= 0 replaces Eq. 12 by a measured E[T] (the paper's 'analytical given E[T]' curve).
 * out[0][k] = E[M~]/M, out[1][k] = min(tau_k, E[T]) + T^c, out[2][k] = E[S_eff];  scalars = E[T], k*, tau*.
 * =========================================================================== */
static double dco_phi(double x) { return 0.5 * erfc(-x / sqrt(2.0)); }

static double dco_phi_inv(double p)
{
    if (!(p > 0.0)) return -INFINITY;
    if (!(p < 1.0)) return INFINITY;
    double lo = -40.0, hi = 40.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (dco_phi(mid) < p) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

double dco_bailey_mean_max(double mu, double sigma, int64_t M, int64_t N)
{
    const double g = 0.57721566490153286061;
    const double z = (1.0 - g) * dco_phi_inv(1.0 - 1.0 / (double)N) + g * dco_phi_inv(1.0 - 1.0 / (exp(1.0) * (double)N));
    return sqrt((double)M * sigma * sigma) * z + (double)M * mu;
}

int dco_closed_form(double mu, double sigma, int64_t M, int64_t N, double t_comm, double mean_T,
                    const float *taus, int64_t K, double *out, double *scalars)
{
    if (!taus || !out || !scalars) return 1;
    if (M <= 0 || N < 2 || K <= 0) return 2;
    if (!(sigma > 0.0)) return 4;
    const double ET = (mean_T >= 0.0) ? mean_T : dco_bailey_mean_max(mu, sigma, M, N);
    for (int64_t k = 0; k < K; ++k) {
        const double tau = (double)taus[k];
        double em = 0.0;
        for (int64_t m = 1; m <= M; ++m) em += dco_phi((tau - (double)m * mu) / sqrt((double)m * sigma * sigma));
        const double step = fmin(tau, ET) + t_comm;
        out[0 * K + k] = em / (double)M;
        out[1 * K + k] = step;
        out[2 * K + k] = (em / (double)M) * (ET + t_comm) / step;
    }
    const int64_t ks = dco_argmax(out + 2 * K, K);
    scalars[0] = ET;
    scalars[1] = (double)ks;
    scalars[2] = ks >= 0 ? (double)taus[ks] : NAN;
    return 0;
}
