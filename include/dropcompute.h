/*
 * dropcompute.h — C ABI of the DropCompute threshold-sweep simulator for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, on one GPU, the Monte-Carlo model behind the paper's automatic choice of
 * the compute threshold tau (DropCompute, arXiv 2306.10598: Algorithm 2 in App. C.1, built from
 * the completed-micro-batch count M~ and the step time min{tau,T}+T^c of Sec. 4.3 and the effective
 * speedup of Eq. 6).
 *
 * Conventions
 *   T  trials (the paper's iterations i = 1..I)        N  data-parallel workers n
 *   M  micro-batches (gradient accumulations) m        K  candidate thresholds tau_k
 *   t_comm  the serial latency T^c of one step (all-reduce etc.), one scalar for all trials
 *   latencies[t][n][m] = t_{i,n}^{(m)}: seconds worker n spent on micro-batch m in trial t
 *
 * Every pointer argument says whether it is a DEVICE or a HOST pointer.  The library never
 * allocates or frees device memory, keeps no per-call state (any number of host threads may call it
 * at the same time, on the same or different streams and devices; what it caches per device or per
 * process -- device properties, kernel attributes, the expert settings of dropcompute_dev.h -- is
 * guarded by locks, and a call works from one consistent copy of the settings taken when it
 * starts), and never synchronises the device unless the function says so: work is enqueued on `stream` (a cudaStream_t passed as void*; NULL
 * is the default stream) and the call returns.  Buffers belong to the caller and must stay valid
 * until the enqueued work has run.  Outputs are overwritten, never accumulated into.
 *
 * Errors.  Every function returns a dc_status.  Anything the host can see (null pointers, sizes
 * out of range, misalignment, unknown enum values, too small a workspace) returns an error code
 * and enqueues nothing.  Properties of the DATA (latencies finite and >= 0, thresholds sorted and
 * not NaN) cannot be seen without reading device memory; they are preconditions.  When they are
 * violated every kernel still stays inside its buffers and terminates, but the numbers are
 * unspecified.  dc_check_inputs() verifies them synchronously for callers who want that.
 * The kernels never trap.  Their internal waits on asynchronous copies are bounded; should one
 * ever expire, the kernel records it and carries on to completion, and dc_device_status()
 * reports it.
 */
#ifndef DROPCOMPUTE_H_
#define DROPCOMPUTE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DC_OK = 0,
    DC_ERR_NULL = 1,        /* a required pointer is NULL */
    DC_ERR_SHAPE = 2,       /* T, N, M or K is not positive */
    DC_ERR_ALIGN = 3,       /* a pointer is not aligned as documented */
    DC_ERR_RANGE = 4,       /* a size exceeds what the library supports (see DC_MAX_K, N*M <= INT32_MAX) */
    DC_ERR_TAUS = 5,        /* dc_check_inputs: thresholds not non-decreasing, or NaN */
    DC_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed (launch, copy, tensor-map encode) */
    DC_ERR_UNSUPPORTED = 7, /* unknown rule / objective */
    DC_ERR_LATENCIES = 8,   /* dc_check_inputs: a latency is negative, NaN or infinite */
    DC_ERR_WORKSPACE = 9,   /* workspace pointer NULL, misaligned or too small */
    DC_ERR_DEVICE = 10      /* dc_device_status: a bounded wait inside a kernel expired */
} dc_status;

/* Largest number of thresholds one call accepts. */
#define DC_MAX_K 4096

/* Completion rule. */
#define DC_RULE_FINISH_BEFORE_TAU 0 /* Algorithm 2 / Sec. 4.3: micro-batch m counts iff T_n^{(m)} < tau */
#define DC_RULE_START_BEFORE_TAU 1  /* Limitations paragraph: the timeout is looked at between
                                       accumulations, so m is run iff T_n^{(m-1)} < tau */

/* Rows of the statistics matrix written by dc_reduce_trials and read by dc_argmax_tau. */
#define DC_STAT_MEAN_STEP 0 /* E[step time](tau)                         = mean_t step[t,k]                 */
#define DC_STAT_DONE_FRAC 1 /* completed fraction E[M~]/M                = sum_t done[t,k] / (T*N*M)        */
#define DC_STAT_THR 2       /* throughput, micro-batches per second     = sum_t done[t,k] / sum_t step[t,k] */
#define DC_STAT_THR_MEAN 3  /* mean per-trial throughput                 = mean_t done[t,k]/step[t,k]       */
#define DC_STAT_S_EFF 4     /* Algorithm 2's S_eff(tau) = mean_t (sync[t]/step[t,k]) * done[t,k]/(N*M)      */
#define DC_NSTATS 5

/*
 * dc_simulate — one pass of the threshold sweep (Algorithm 2's loops over i, n, m for all tau at
 * once; Sec. 4.3).  For every trial t and threshold k:
 *
 *   P_{t,n,m}      = fl32(P_{t,n,m-1} + latencies[t][n][m]),  P_{t,n,-1} = +0     (strictly m = 0..M-1)
 *   out_done[t][k] = #{ (n,m) : P_{t,n,m} < taus[k] }          (= N * M~_t(tau_k); strict '<', fp32)
 *   out_step[t][k] = fl32( fminf(taus[k], max_n P_{t,n,M-1}) + t_comm )   (= min{tau,T} + T^c)
 *
 *   latencies  DEVICE, [T][N][M] fp32, contiguous, m fastest; finite, >= 0 and small enough that a worker's M
 *              latencies add up to a finite fp32 number; 4-byte aligned.  A 16-byte aligned
 *              pointer with M a multiple of 4 takes the fastest (tiled) kernel; every other case takes the flat
 *              kernel when M <= 127 and the plain-load kernel beyond (roughly 0.3-0.7 and 0.4-0.6 of the tiled
 *              kernel's rate); see dc_simulate_plan
 *   T, N, M    > 0, N*M <= INT32_MAX
 *   taus       DEVICE, [K] fp32, non-decreasing, no NaN; +infinity is allowed (gives the
 *              synchronous baseline); 4-byte aligned.  1 <= K <= DC_MAX_K
 *   out_step   DEVICE, [T][K] fp32        out_done   DEVICE, [T][K] int32
 *   stream     cudaStream_t
 *
 * The result does not depend on the launch configuration or on scheduling: counts are integers
 * and the maximum is exact, so two calls on the same input give the same bits.
 */
int dc_simulate(const float *latencies, int64_t T, int64_t N, int64_t M,
                const float *taus, int32_t K, float t_comm,
                float *out_step, int32_t *out_done, void *stream);

/*
 * dc_simulate_ex — dc_simulate plus the tau = infinity baseline and the choice of completion rule.
 *
 *   out_sync   DEVICE, [T] fp32 or NULL:  out_sync[t] = fl32( max_n P_{t,n,M-1} + t_comm )
 *              (the plain synchronous step time T + T^c of Sec. 4.2 / 4.4)
 *   rule       DC_RULE_FINISH_BEFORE_TAU: as dc_simulate.
 *              DC_RULE_START_BEFORE_TAU:  out_done[t][k] = #{(n,m): P_{t,n,m-1} < taus[k]} and
 *              out_step[t][k] = fl32( max_n W_n + t_comm ), W_n = P_{t,n,s-1} with s the number of
 *              micro-batches worker n ran (W_n = 0 if none).
 */
int dc_simulate_ex(const float *latencies, int64_t T, int64_t N, int64_t M,
                   const float *taus, int32_t K, float t_comm,
                   float *out_step, int32_t *out_done, float *out_sync,
                   int32_t rule, void *stream);

/*
 * dc_simulate_tc — dc_simulate_ex with one communication time per trial (Algorithm 2, input T_i^c: the
 * algorithm takes a measured value for every iteration):
 *   t_comm_trials  DEVICE, [T] fp32; trial t uses t_comm_trials[t] wherever dc_simulate_ex uses t_comm.
 * Everything else as dc_simulate_ex.  dc_reduce_trials needs no change: it works from out_step and out_sync.
 */
int dc_simulate_tc(const float *latencies, int64_t T, int64_t N, int64_t M,
                   const float *taus, int32_t K, const float *t_comm_trials,
                   float *out_step, int32_t *out_done, float *out_sync,
                   int32_t rule, void *stream);

/*
 * dc_simulate_scaled — dc_simulate_ex for workers that are not identical (App. C.2 remarks that each worker may have
 * its own mu_n, sigma_n): worker n works against its own thresholds
 *
 *   theta[n][k] = fl32( worker_scale[n] * taus[k] )          (one fp32 product; worker_scale[n] > 0, finite)
 *
 * instead of the common taus[k].  With DC_RULE_FINISH_BEFORE_TAU:
 *   out_done[t][k] = #{ (n,m) : P_{t,n,m} < theta[n][k] }
 *   out_step[t][k] = fl32( max_n fminf(theta[n][k], P_{t,n,M-1}) + t_comm )     (Sec. 4.3's min{tau, T_n}, per worker)
 * and with DC_RULE_START_BEFORE_TAU micro-batch m of worker n is run iff P_{t,n,m-1} < theta[n][k], W_n is the finish
 * time of the last one it ran and out_step[t][k] = fl32( max_n W_n + t_comm ).  out_sync as in dc_simulate_ex (it does not
 * depend on the scales).  worker_scale = all ones gives dc_simulate_ex's results bit for bit.
 *   worker_scale  DEVICE, [N] fp32, 4-byte aligned
 * Everything else as dc_simulate_ex; dc_reduce_trials and dc_argmax_tau work on the outputs unchanged.  A plain kernel
 * (ordinary loads, one block per trial, a cursor per row): 0.9-2.1 TB/s on the workloads here, a sixth to a third of
 * dc_simulate_ex's rate.
 */
int dc_simulate_scaled(const float *latencies, int64_t T, int64_t N, int64_t M,
                       const float *taus, int32_t K, const float *worker_scale, float t_comm,
                       float *out_step, int32_t *out_done, float *out_sync,
                       int32_t rule, void *stream);

/*
 * dc_simulate_split — dc_simulate_ex for FEW trials of MANY workers.  The sweep kernels give a whole trial to
 * one thread block, so fewer trials than about twice the number of SMs leave most of the GPU idle.  This entry
 * point sweeps every trial as G groups of N/G workers (G a divisor of N chosen by the library; no data is
 * moved) and then merges the groups: counts add, step times and the synchronous time are maxima.  Results are
 * bit-identical to dc_simulate_ex.  When nothing would be gained (enough trials, N < 128, or N has no suitable
 * divisor) it simply calls dc_simulate_ex and needs no workspace.
 *   workspace  DEVICE scratch, 256-byte aligned, at least dc_simulate_split_workspace_bytes(T, N, M, K) bytes
 *              (0 when no split is used; sizes refer to the current device).  Contents unspecified afterwards.
 * Other arguments as dc_simulate_ex.
 */
size_t dc_simulate_split_workspace_bytes(int64_t T, int64_t N, int64_t M, int32_t K);
int dc_simulate_split(const float *latencies, int64_t T, int64_t N, int64_t M,
                      const float *taus, int32_t K, float t_comm,
                      float *out_step, int32_t *out_done, float *out_sync, int32_t rule,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * dc_reduce_trials — statistics over trials in fp64 (Algorithm 2: S_i(tau) and S_eff(tau); Eq. 6;
 * Sec. 4.4 throughput).  Sums run over trials in a fixed order that depends only on (T, K), so the
 * result is reproducible bit for bit.
 *
 *   out_step, out_done   DEVICE, as written by dc_simulate
 *   out_sync             DEVICE [T] or NULL.  With NULL, row DC_STAT_S_EFF and both baseline
 *                        entries are NaN.
 *   stats      DEVICE, [DC_NSTATS][K] fp64, rows as DC_STAT_* above
 *   baseline   DEVICE, [2] fp64: mean_t sync[t]  and  T*N*M / sum_t sync[t]  (micro-batches per second
 *              without DropCompute)
 *   workspace  DEVICE scratch of at least dc_reduce_workspace_bytes(T, K) bytes, 8-byte aligned.
 *              Contents on entry are ignored; contents on return are unspecified.  Two calls that may
 *              overlap on the device need different workspaces.
 */
size_t dc_reduce_workspace_bytes(int64_t T, int32_t K);
int dc_reduce_trials(const float *out_step, const int32_t *out_done, const float *out_sync,
                     int64_t T, int32_t K, int64_t N, int64_t M,
                     double *stats, double *baseline,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * dc_reduce_trials_static — the same statistics as dc_reduce_trials, for a caller that cannot hand over a
 * workspace.  (The paper has no counterpart to this entry point; it exists for deployment only.)
 *
 * Who needs it: code that runs where device memory may not be requested any more — a plug-in inside a
 * serving or training process whose memory pool already owns the whole GPU (a fresh cudaMalloc there fails
 * or forces the pool to shrink), or a latency-critical loop in which an allocation would stall the device.
 * Such a caller still owns its inputs and outputs, but has nowhere to put the partial sums of the two-phase
 * reduction.  Here they live in an array that is part of the library image: DC_STATIC_SCRATCH_BYTES bytes of
 * device memory that every GPU holds from the moment it loads this library until the process ends.
 *
 * Same arguments, results and error codes as dc_reduce_trials without the workspace pair, plus:
 *   K <= DC_STATIC_MAX_K, otherwise DC_ERR_RANGE (the array is sized for that many thresholds; use
 *   dc_reduce_trials with your own workspace beyond it).  T is not limited.
 * The call allocates and frees nothing, neither directly nor through a library routine.  (What the CUDA runtime
 * itself does when a device first uses this library is outside the call's control: the library image, the array
 * included, is made resident on that device at the first call of any entry point there.)
 * The first call on each device looks up the array's device address (one runtime query, cached); make that
 * first call outside any stream capture.
 * All calls on a device share the one array.  Nothing in it has to be cleared between calls — each call
 * overwrites every partial sum before reading it, so what an earlier call left behind is never seen — but
 * two calls that may run at the same time on one device (different streams) would overwrite each other's
 * partial sums: serialise them, or give the concurrent ones a workspace through dc_reduce_trials.
 */
#define DC_STATIC_MAX_K 1024
#define DC_STATIC_SCRATCH_BYTES (64 * (4 * DC_STATIC_MAX_K + 1) * 8) /* 2 097 664 bytes per GPU */
int dc_reduce_trials_static(const float *out_step, const int32_t *out_done, const float *out_sync,
                            int64_t T, int32_t K, int64_t N, int64_t M,
                            double *stats, double *baseline, void *stream);

/*
 * dc_argmax_tau — tau* = argmax_tau objective(tau) (last line of Algorithm 2).
 *
 *   stats      DEVICE, [DC_NSTATS][K] from dc_reduce_trials      taus  DEVICE [K]
 *   objective  DC_STAT_S_EFF (Algorithm 2's own), DC_STAT_THR or DC_STAT_THR_MEAN
 *   out_k      DEVICE int32: first index attaining the maximum; NaN entries never win; -1 if all are NaN
 *   out_tau    DEVICE fp32: taus[out_k] (NaN if out_k = -1)       out_value  DEVICE fp64 (NaN if -1)
 */
int dc_argmax_tau(const double *stats, const float *taus, int32_t K, int32_t objective,
                  int32_t *out_k, float *out_tau, double *out_value, void *stream);

/*
 * dc_sweep_device — Algorithm 2 from samples to tau* in one host call, everything resident on the DEVICE:
 * enqueues dc_simulate_ex, dc_reduce_trials and dc_argmax_tau on `stream`, in that order, with the arguments
 * documented there (out_sync is required here).  Host-visible errors of any of the three are reported before
 * anything is enqueued.  workspace as for dc_reduce_trials (dc_reduce_workspace_bytes(T, K) bytes).
 * Like the three calls it stands for, it only enqueues kernels: once it has been called normally on a device it
 * can be recorded in a CUDA stream capture and replayed, which pays off on inputs small enough to be bound by
 * launch latency.
 */
int dc_sweep_device(const float *latencies, int64_t T, int64_t N, int64_t M,
                    const float *taus, int32_t K, float t_comm, int32_t rule, int32_t objective,
                    float *out_step, int32_t *out_done, float *out_sync,
                    double *stats, double *baseline, int32_t *out_k, float *out_tau, double *out_value,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * dc_closed_form — the paper's analytical estimates (App. C.2) on a threshold grid, from the mean `mu` and
 * standard deviation `sigma` of ONE micro-batch latency, for comparison with the simulation (Fig. 3):
 *   out[0][k] = E[M~(tau_k)] / M        = (1/M) sum_{m=1..M} Phi((tau_k - m mu) / sqrt(m sigma^2))     (Eq. 5 / 10)
 *   out[1][k] = min(tau_k, E[T]) + t_comm
 *   out[2][k] = E[S_eff(tau_k)]         = out[0][k] (E[T] + t_comm) / out[1][k]                        (Eq. 11; numerator as in Eq. 6)
 *   scalars[0] = E[T] = sqrt(M sigma^2) ((1-g) Phi^-1(1 - 1/N) + g Phi^-1(1 - 1/(e N))) + M mu         (Eq. 4 / 12,
 *                g = Euler-Mascheroni; T does not contain t_comm), or mean_T itself when mean_T >= 0 (the
 *                'analytical given E[T]' variant: pass the simulated mean_sync - t_comm).
 * The analytic tau* is dc_argmax_tau over row 2 (pass `out` as stats with objective 2 — row 2 of a [3][K] matrix).
 *   taus  DEVICE [K] fp32      out  DEVICE [3][K] fp64      scalars  DEVICE [1] fp64      M >= 1, N >= 2, sigma > 0
 */
int dc_closed_form(double mu, double sigma, int64_t M, int64_t N, double t_comm, double mean_T,
                   const float *taus, int32_t K, double *out, double *scalars, void *stream);

/*
 * dc_sweep_host — the whole path for a caller whose samples live in HOST memory: copies the
 * latencies to the device in chunks of whole trials (overlapped with the kernels), runs
 * dc_simulate_ex, dc_reduce_trials and dc_argmax_tau, copies the results back and waits for them.
 * SYNCHRONOUS: returns when the host outputs are written.
 *
 *   latencies_host  HOST [T][N][M] fp32 (page-locked memory makes the copies asynchronous and fast)
 *   taus_host       HOST [K]
 *   stats_host      HOST [DC_NSTATS][K] fp64      baseline_host  HOST [2] fp64
 *   k_star_host     HOST int32                    tau_star_host  HOST fp32
 *   workspace       DEVICE scratch, at least dc_sweep_host_workspace_bytes(T,N,M,K, chunk_trials)
 *                   bytes, 1024-byte aligned.  chunk_trials >= 1 is how many trials travel per copy;
 *                   two chunks are resident at a time.
 *   rule, objective as above
 */
size_t dc_sweep_host_workspace_bytes(int64_t T, int64_t N, int64_t M, int32_t K, int64_t chunk_trials);
int dc_sweep_host(const float *latencies_host, int64_t T, int64_t N, int64_t M,
                  const float *taus_host, int32_t K, float t_comm, int32_t rule, int32_t objective,
                  int64_t chunk_trials,
                  double *stats_host, double *baseline_host, int32_t *k_star_host, float *tau_star_host,
                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * dc_check_inputs — SYNCHRONOUS check of the data preconditions of dc_simulate on `stream`:
 * returns DC_ERR_LATENCIES if any latency is negative, NaN or infinite or a worker's latencies add up
 * (left to right, in fp32) to infinity, DC_ERR_TAUS if the grid is not non-decreasing or holds a NaN,
 * DC_OK otherwise.  report_host (HOST, [2] int64, may be NULL) receives the number of bad latencies
 * plus overflowing rows, and the number of bad thresholds.
 *   counters  DEVICE scratch, [2] int64 (16 bytes, 8-byte aligned)
 */
int dc_check_inputs(const float *latencies, int64_t T, int64_t N, int64_t M,
                    const float *taus, int32_t K,
                    int64_t *counters, int64_t *report_host, void *stream);

/*
 * dc_device_status — SYNCHRONOUS.  Reads and clears the current device's record of expired waits.
 * Returns DC_OK if none expired since the last call, DC_ERR_DEVICE otherwise; *flags_host (HOST,
 * may be NULL) receives the raw bit mask (bit 0: a load never arrived, bit 1: a buffer was never
 * released).
 */
int dc_device_status(uint32_t *flags_host);

const char *dc_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* DROPCOMPUTE_H_ */
