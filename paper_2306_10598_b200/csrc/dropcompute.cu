// DropCompute threshold-sweep simulator for sm_100a: kernels and the C ABI declared in
// include/dropcompute.h.
//
// What is computed (paper: DropCompute, arXiv 2306.10598): Algorithm 2 (App. C.1) evaluates, for
// every candidate threshold tau and every measured iteration, each worker's running compute time
// T_{i,n} (micro-batch by micro-batch), the number of micro-batches whose running time is below
// tau (the M~ of Sec. 4.3), the slowest worker's time T_i, the step time min(tau,T_i)+T^c and the
// effective speedup S_i(tau) (Eq. 6); then it averages over iterations and takes the arg-max.
//
// How it is computed here.  The running sum does not depend on tau, so the samples are read ONCE.
// A thread owns one worker's row of M latencies and adds them strictly left to right in fp32.
// Because latencies are >= 0 the running sum P never decreases, and because the thresholds are
// sorted, [P < tau_k] <=> k >= j(P) with j(P) = #{k : tau_k <= P}.  So each sample falls into one
// bin j in [0,K] and done[t][k] is the prefix sum of the bin counts.  j(P) comes from a lookup
// table over equal cells of the threshold range, or for evenly spaced thresholds from one
// multiply-add, and is then settled by comparing P with the thresholds themselves, so the bins
// are exact.  Whole groups of samples that every lane of a warp still has below the first
// threshold are counted in a register.  Bin counts go to integer histograms in shared memory,
// which a dedicated warp sums, prefix-scans and writes out per trial while the other warps are
// already on the next trial.  One block owns a whole trial at a time (all N workers), so no
// global atomics and no scratch memory are needed and every result is an integer sum or an exact
// maximum: bit-reproducible.  The start-before-tau variant of the rule (the paper's Limitations
// paragraph) needs, besides the count, the largest finish time per bin and a prefix maximum.
//
// Data movement.  The kernel is bound by the one read of latencies[T][N][M] from HBM.  Tiles of
// (rows x up to 128 bytes of each row) are brought into shared memory by the TMA unit
// (cp.async.bulk.tensor, 3-D tensor map over [T][N][M]) through a ring of stages guarded by
// mbarriers; a dedicated producer warp issues the copies and the other warps consume.  The
// hardware swizzle (128/64/32-byte modes) makes "lane r reads 16 bytes of row r" free of
// shared-memory bank conflicts.  Rows past N in a trial's last pass and columns past M are
// out-of-bounds coordinates of the tensor map: they are zero-filled by the TMA unit and cost no
// HBM traffic.  Rows whose length is not a multiple of 4 floats cannot be described by a tensor
// map; they come in as plain bulk copies of whole rows (dc_sweep_flat) or, failing that, by
// ordinary loads (dc_sweep_plain).
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <mutex>
#include <stdint.h>
#include <string.h>

#include "dropcompute.h"

namespace {

// ------------------------------------------------------------------------------------------
// constants
// ------------------------------------------------------------------------------------------
constexpr int kMaxRowsPerPass = 256;          // rows (threads) of one trial handled per pass; also the TMA box limit
constexpr int kMaxStages = 8;
constexpr int kStageBudgetBytes = 96 * 1024;  // shared memory spent on the ring of stages per block
constexpr int kHistBudgetBytes = 32 * 1024;   // shared memory spent on per-warp histograms per block
constexpr uint32_t kWaitLimit = 1u << 22;     // polls of one mbarrier wait before giving up (roughly a second)
constexpr int kReduceChunksMax = 64;          // partial sums per threshold in dc_reduce_trials
constexpr int kConsumerBarrier = 1;           // named barrier used by the consumer warps
constexpr int kFlatMaxM = 255;                // longest row the flat kernel takes (32 rows of it fill a stage)
constexpr int kLutCellsMax = 4096;            // cells of the bin lookup table (4 per threshold up to this)

constexpr uint32_t kErrLoadNeverArrived = 1u;
constexpr uint32_t kErrStageNeverFreed = 2u;

__device__ unsigned int g_wait_expired = 0;   // bit mask of expired waits on this device

struct SweepParams {
    const float *lat;
    const float *taus;
    float *out_step;
    int32_t *out_done;
    float *out_sync;   // may be null
    long long T;
    int N, M, K;
    float t_comm;
    const float *t_comm_vec;  // per-trial T^c, or null: t_comm for every trial
    int passes;        // passes over a trial's workers
    int rows;          // workers per pass (box height for the tiled kernel, blockDim.x for the plain one)
    int chunks;        // column chunks per row
    int bw;            // floats of a row per chunk (box width)
    int nq_last;       // 16-byte quads of a row in the last chunk
    int pitch;         // shared-memory bytes per row in a stage
    int swz_mask;      // 7 / 3 / 1 / 0 for the 128 / 64 / 32-byte swizzle / none
    int stages;
    int stage_bytes;   // multiple of 1024
    int hist_copies;   // histogram copies in shared memory
    int hist_stride;   // ints per copy (>= K + 1)
    int lane_copies;   // tiled kernel: copies per warp (lane l uses copy l % lane_copies); power of two
    int warp_groups;   // tiled kernel: warp w uses the copies of group w % warp_groups
    int lut_cells;     // tiled kernel: cells of the bin lookup table (the table has lut_cells + 1 entries)
    int rule;          // DC_RULE_*
    int aux_copies;    // rule 1: copies of the per-bin finish-time maxima, one per histogram copy (0 for rule 0)
    int batch_lookups; // tiled kernel: 1 = look up a whole group's bins before updating the histogram
    int nbuf;          // histogram / maxima buffers: 2 in the tiled kernel (filled and drained in turn), 1 in the plain one
    int one;           // always 1; a value the compiler cannot see, used to tie a stage release to a warp vote
    int flat_groups;   // flat kernel: groups of consumer warps working on different tiles at the same time
    int tile_warps;    // flat kernel: warps per group (rows / 32)
    int direct_bins;   // staged kernels: 1 = bin evenly spaced thresholds arithmetically instead of through the table
    int short_launch;  // host only: under 1 GiB of latencies (see simulate_impl)
    int epi_vec;       // staged kernels: the epilogue warp may take four bins per lane with 16-byte accesses
                       // (K a multiple of 4, out_step / out_done 16-byte aligned, hist_stride a multiple of 4)
};

// ------------------------------------------------------------------------------------------
// small PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_count(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  If the limit is reached the fact is recorded and the caller carries on, so that
// every thread still reaches every barrier and the kernel ends (its results are then garbage and
// dc_device_status() says so).
__device__ __forceinline__ void mbar_wait(uint64_t *bar, uint32_t parity, uint32_t err_bit)
{
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (it > 64) __nanosleep(128);
    }
    atomicOr(&g_wait_expired, err_bit);
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(smem_addr(bar))
        : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Start-before-tau rule.  Micro-batch m is run iff the time before it, P_{m-1}, is < tau_k, and a worker's time
// W_n(k) is the finish time of the last micro-batch it ran (0 if it ran none).  Running sums never decrease, so
// W_n(k) is also the LARGEST finish time among the micro-batches the worker ran, and the step's compute time is
//     max_n W_n(k) = max { P_{n,m} : P_{n,m-1} < tau_k }            (all micro-batches any worker started).
// With j(x) = #{k' : tau_k' <= x} (the bin of x), P_{m-1} < tau_k  <=>  j(P_{m-1}) <= k.  So each micro-batch
// makes two POINT updates at the bin a = j(P_{m-1}) of the time before it,
//     hist[a] += 1   and   fmax[a] = max(fmax[a], P_m),
// and the epilogue turns them into done[t][k] (prefix sum of hist) and max_n W_n(k) (prefix maximum of fmax).
// Non-negative floats order like their bit patterns, so the integer atomicMax is an exact float maximum.
__device__ __forceinline__ void raise_max(float *slot, float V)
{
    atomicMax(reinterpret_cast<int *>(slot), __float_as_int(V));
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_inclusive_max_scan(float v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v = fmaxf(v, u);
    }
    return v;
}
__device__ __forceinline__ int warp_inclusive_scan(int v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// ------------------------------------------------------------------------------------------
// End of a trial: all `nthr` participating threads call this with their largest row total.
// Sums the histogram copies, prefix-scans the bins into done[t][k] (M~ * N of Sec. 4.3), takes
// T = max_n T_n, writes step[t][k] = min(tau_k, T) + T^c and sync[t] = T + T^c, and clears the
// histograms for the next trial.
// ------------------------------------------------------------------------------------------
// Rule 1 (start-before-tau): step[t][k] = max_n W_n(k) + T^c = (prefix maximum of fmax[] up to bin k) + T^c.
__device__ __forceinline__ void trial_epilogue(const SweepParams &p, long long t, float rowmax, int tid, int nthr,
                                               int barrier_id, const float *tau_s, int *hist, float *smax, int *wtot,
                                               float *fmax, float *wmx)
{
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int K = p.K, H = p.hist_copies, HS = p.hist_stride;
    const bool rule1 = p.rule == DC_RULE_START_BEFORE_TAU;
    const float t_comm = p.t_comm_vec ? p.t_comm_vec[t] : p.t_comm;
    rowmax = warp_max(rowmax);
    if (lane == 0) smax[warp] = rowmax;
    named_barrier(barrier_id, nthr);  // all histogram updates and smax[] visible

    float Tmax = 0.0f;
    for (int w = 0; w < nwarps; ++w) Tmax = fmaxf(Tmax, smax[w]);

    const int ipt = (K + nthr - 1) / nthr;  // bins per thread (consecutive)
    const int b0 = min(K, tid * ipt), b1 = min(K, b0 + ipt);
    int tot = 0;
    float fm = 0.0f;
    for (int b = b0; b < b1; ++b) {
        for (int c = 0; c < H; ++c) {
            tot += hist[c * HS + b];
            if (rule1) fm = fmaxf(fm, fmax[c * HS + b]);
        }
    }
    const int incl = warp_inclusive_scan(tot, lane);
    if (lane == 31) wtot[warp] = incl;
    float fm_incl = 0.0f;
    if (rule1) {
        fm_incl = warp_inclusive_max_scan(fm, lane);
        if (lane == 31) wmx[warp] = fm_incl;
    }
    named_barrier(barrier_id, nthr);

    int run = incl - tot;
    for (int w = 0; w < warp; ++w) run += wtot[w];
    float fm_run = 0.0f;  // maximum of fmax[] over all bins before b0
    if (rule1) {
        const float up = __shfl_up_sync(0xffffffffu, fm_incl, 1);
        if (lane > 0) fm_run = up;
        for (int w = 0; w < warp; ++w) fm_run = fmaxf(fm_run, wmx[w]);
    }
    float *step_row = p.out_step + t * K;
    int32_t *done_row = p.out_done + t * K;
    for (int b = b0; b < b1; ++b) {
        int h = 0;
        for (int c = 0; c < H; ++c) {
            h += hist[c * HS + b];
            hist[c * HS + b] = 0;
            if (rule1) {
                fm_run = fmaxf(fm_run, fmax[c * HS + b]);
                fmax[c * HS + b] = 0.0f;
            }
        }
        run += h;
        done_row[b] = run;
        step_row[b] = __fadd_rn(rule1 ? fm_run : fminf(tau_s[b], Tmax), t_comm);
    }
    for (int c = tid; c < H; c += nthr) {  // the bins of samples at or above the last threshold
        hist[c * HS + K] = 0;
        if (HS > K + 1) hist[c * HS + K + 1] = 0;
        if (rule1) {
            fmax[c * HS + K] = 0.0f;
            if (HS > K + 1) fmax[c * HS + K + 1] = 0.0f;
        }
    }
    if (tid == 0 && p.out_sync != nullptr) p.out_sync[t] = __fadd_rn(Tmax, t_comm);
    named_barrier(barrier_id, nthr);  // histograms cleared, smax/wtot free again
}

// Shared-memory carve-up common to both kernels (after the stages of the tiled kernel).
struct SmemTail {
    float *tau_s;
    int *hist;
    float *smax;
    int *wtot;
    int *meta;           // [0] lookup table has at most one finite threshold per cell, [1..2] lo, scale (as bits),
                         // [3] the thresholds are evenly spaced enough for direct binning, [4..5] its scale, shift
    unsigned short *lut; // lut_cells + 1 entries (tiled kernel only)
    float *wmx;          // rule 1, plain kernel: warp totals of the prefix-maximum scan
    float *fmax;         // rule 1: [nbuf][hist_copies][hist_stride], laid out like hist: largest finish time among
                         // the micro-batches whose start time lies in the bin
};
__device__ __forceinline__ SmemTail carve_tail(unsigned char *base, const SweepParams &p)
{
    SmemTail s;
    s.tau_s = reinterpret_cast<float *>(base);
    s.hist = reinterpret_cast<int *>(s.tau_s + ((p.K + 4) & ~3));  // K + 1 thresholds, padded to 16 bytes
    s.smax = reinterpret_cast<float *>(s.hist + p.nbuf * p.hist_copies * p.hist_stride);
    s.wtot = reinterpret_cast<int *>(s.smax + 32);
    s.meta = s.wtot + 32;
    s.lut = reinterpret_cast<unsigned short *>(s.meta + 8);
    s.wmx = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(s.lut) +
                                      (((size_t)(p.lut_cells + 1) * sizeof(unsigned short) + 15) & ~(size_t)15));
    s.fmax = s.wmx + 32;
    return s;
}
// hist_copies and fmax_copies count all buffers (nbuf times the copies of one buffer)
__host__ __device__ inline size_t tail_bytes(int K, int hist_copies, int hist_stride, int lut_cells, int fmax_copies)
{
    return sizeof(float) * (size_t)((K + 4) & ~3) + sizeof(int) * (size_t)hist_copies * hist_stride + 72 * sizeof(int) +
           (((size_t)(lut_cells + 1) * sizeof(unsigned short) + 15) & ~(size_t)15) + 32 * sizeof(float) +
           sizeof(float) * (size_t)fmax_copies * hist_stride;
}

__device__ __forceinline__ void load_thresholds(const SweepParams &p, const SmemTail &s, int tid, int nthr)
{
    for (int k = tid; k < p.K; k += nthr) s.tau_s[k] = p.taus[k];
    if (tid == 0) s.tau_s[p.K] = __int_as_float(0x7f800000);  // +inf sentinel
    for (int i = tid; i < p.nbuf * p.hist_copies * p.hist_stride; i += nthr) s.hist[i] = 0;
    for (int i = tid; i < p.nbuf * p.aux_copies * p.hist_stride; i += nthr) s.fmax[i] = 0.0f;
}

// ------------------------------------------------------------------------------------------
// Bin lookup for the tiled kernel.  A running sum P falls into bin j(P) = #{k : tau_k <= P}.
// The range [lo, hi] of the finite thresholds is cut into C equal cells; cell(x) is a monotone
// function of x evaluated with the SAME two fp32 operations for thresholds and samples, so
//   lut[c] = #{k : tau_k = -inf or cell(tau_k) < c}  <=  j(P)  for every P with cell(P) = c,
// and j(P) is reached from lut[c] by comparing P with the real thresholds (one compare when no
// cell holds two finite thresholds, which is the case for evenly spaced grids).  The table only
// proposes where to start; the comparisons with tau_k decide, so the bins are exact.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned lut_cell(float x, float lo, float scale, unsigned C)
{
    return min(__float2uint_rz(__fmul_rn(__fsub_rn(x, lo), scale)), C);  // negative and NaN -> 0, huge -> C
}

// Direct binning for evenly spaced thresholds, without the table.  dcell(x) = min(uint(x * dscale + dshift), K) with
// dscale = (K-1) / (tau_{K-1} - tau_0) and dshift = 0.5 - tau_0 * dscale puts tau_k in the middle of cell k.  It is
// used only if dcell(tau_k) == k holds for EVERY k (checked below with the same instruction sequence).  dcell is
// monotone (one fused multiply-add, one truncation, one minimum), hence for a sample P with c = dcell(P):
// k < c gives dcell(tau_k) < dcell(P), so tau_k < P; k > c gives tau_k > P; and tau_c is compared directly:
//     j(P) = c + [P >= tau_c]        (tau_K = +inf)
__device__ __forceinline__ unsigned direct_cell(float x, float dscale, float dshift, unsigned K)
{
    return min(__float2uint_rz(__fmaf_rn(x, dscale, dshift)), K);  // negative and NaN -> 0, huge -> K
}
__device__ __forceinline__ unsigned direct_offset(float P, float dscale, float dshift, unsigned K, const unsigned char *tau_b)
{
    unsigned off = 4u * direct_cell(P, dscale, dshift, K);
    off += (P >= *reinterpret_cast<const float *>(tau_b + off)) ? 4u : 0u;
    return off;
}

// All threads of the block; tau_s[0..K] is loaded (tau_s[K] = +inf).  Ends with __syncthreads().
__device__ __forceinline__ void build_lut(const SweepParams &p, const SmemTail &s, int tid, int nthr)
{
    const int K = p.K;
    const unsigned C = (unsigned)p.lut_cells;
    const float ninf = __int_as_float(0xff800000), pinf = __int_as_float(0x7f800000);
    if (tid == 0) {
        int klo = 0, khi = K - 1;
        while (klo < K && !(s.tau_s[klo] > ninf)) ++klo;
        while (khi >= 0 && !(s.tau_s[khi] < pinf)) --khi;
        float lo = 0.0f, scale = 0.0f;
        if (klo <= khi) {
            lo = s.tau_s[klo];
            const float range = __fsub_rn(s.tau_s[khi], lo);
            if (range > 0.0f && range < pinf) scale = __fdiv_rn((float)C, range);
            if (!(scale < pinf)) scale = 0.0f;
        }
        s.meta[0] = 1;
        s.meta[1] = __float_as_int(lo);
        s.meta[2] = __float_as_int(scale);
        // direct binning: all thresholds finite, checked cell by cell after the barrier
        float dscale = 0.0f;
        const bool finite = (klo == 0 && khi == K - 1);
        if (finite && K > 1) {
            const float range = __fsub_rn(s.tau_s[K - 1], s.tau_s[0]);
            if (range > 0.0f && range < pinf) dscale = __fdiv_rn((float)(K - 1), range);
            if (!(dscale < pinf)) dscale = 0.0f;
        }
        const float dshift = finite ? __fmaf_rn(-s.tau_s[0], dscale, 0.5f) : 0.0f;
        s.meta[3] = (finite && dshift == dshift && fabsf(dshift) < pinf) ? 1 : 0;
        s.meta[4] = __float_as_int(dscale);
        s.meta[5] = __float_as_int(dshift);
    }
    for (unsigned c = tid; c <= C; c += nthr) s.lut[c] = 0;
    __syncthreads();
    const float lo = __int_as_float(s.meta[1]), scale = __int_as_float(s.meta[2]);
    // extended cell of threshold k: -1 for -inf, C+1 for +inf / NaN / the virtual entry k = K
    auto cx = [&](int k) -> int {
        if (k >= K) return (int)C + 1;
        const float x = s.tau_s[k];
        if (x == ninf) return -1;
        if (!(x < pinf)) return (int)C + 1;
        return (int)lut_cell(x, lo, scale, C);
    };
    for (int k = tid; k <= K; k += nthr) {
        const int prev = (k == 0) ? -1 : cx(k - 1);
        const int cur = cx(k);
        const int last = min(cur, (int)C);
        for (int c = prev + 1; c <= last; ++c) s.lut[c] = (unsigned short)(4 * k);  // byte offset of the smallest k with cx(k) >= c
        if (k > 0 && k < K && cur == prev && cur >= 0 && cur <= (int)C) s.meta[0] = 0;  // two finite thresholds share a cell
        if (k < K && direct_cell(s.tau_s[k], __int_as_float(s.meta[4]), __int_as_float(s.meta[5]), (unsigned)K) != (unsigned)k)
            s.meta[3] = 0;  // threshold k is not in cell k: no direct binning
    }
    __syncthreads();
}

// Bins one running sum (tiled kernel): adds 1 to bin j(P) of this thread's histogram copy.  The table
// entry and `off` are BYTE offsets (4 j) into the threshold array and the histogram.  Bins 0..K+1 exist
// (K: at or above the last threshold, K+1: only reachable by P = +inf); the epilogue reads 0..K-1.
// ONE = the table guarantees at most one threshold to step over.
template <bool ONE>
__device__ __forceinline__ unsigned bin_offset(float P, float lo, float scale, unsigned C, const unsigned short *lut,
                                               const unsigned char *tau_b, unsigned K4)
{
    unsigned off = lut[lut_cell(P, lo, scale, C)];
    off += (P >= *reinterpret_cast<const float *>(tau_b + off)) ? 4u : 0u;  // tau_s[K] = +inf
    if (!ONE) {
        while (off < K4 && P >= *reinterpret_cast<const float *>(tau_b + off)) off += 4u;
    }
    return off;
}
template <bool ONE>
__device__ __forceinline__ void bin_sample(float P, float lo, float scale, unsigned C, const unsigned short *lut,
                                           const unsigned char *tau_b, unsigned K4, unsigned char *hist_b)
{
    atomicAdd(reinterpret_cast<int *>(hist_b + bin_offset<ONE>(P, lo, scale, C, lut, tau_b, K4)), 1);
}
// Start-before-tau rule: micro-batch m with finish time P.  The time before it lies in bin `prev` (byte
// offset): that bin's count goes up by one and its finish-time maximum is raised to P (see raise_max);
// fmax_delta is the byte distance from a histogram entry to the maximum of the same bin and copy.
// Bin 0 is kept in the thread's registers (cnt0, fin0) and added once per trial: when a straggler lane sends its
// warp through this path the other lanes are typically all still in bin 0 and would pile up on one entry.  (The
// same test in the finish-before-tau path measured slower there, so that path adds unconditionally.)
__device__ __forceinline__ void start_rule_update(float P, unsigned prev, unsigned char *hist_b, unsigned fmax_delta,
                                                  int &cnt0, float &fin0)
{
    if (prev != 0u) {
        atomicAdd(reinterpret_cast<int *>(hist_b + prev), 1);
        atomicMax(reinterpret_cast<int *>(hist_b + fmax_delta + prev), __float_as_int(P));
    } else {
        ++cnt0;
        fin0 = fmaxf(fin0, P);
    }
}

// ------------------------------------------------------------------------------------------
// What a consumer thread does with one chunk of its row (up to 4*NQ samples held in registers), shared by
// the tiled and the flat kernel.  `ns` samples of the chunk exist (the same number for all threads; missing
// ones hold zeros, so the running sum stays put over them and they are never counted).
// ------------------------------------------------------------------------------------------
struct BinCtx {
    float lut_lo, lut_scale;
    unsigned C;
    const unsigned short *lut;
    const unsigned char *tau_b;
    unsigned K4;
    bool one;                 // the table guarantees at most one threshold to step over
    float dscale, dshift;     // direct binning (only used when the grid qualifies)
    unsigned K;
    float tau_first, tau_last;
    uint32_t arrive_one;      // always 1, opaque to the compiler (ties a stage release to a warp vote)
};

// The binning context of a block, from the tables build_lut() left in shared memory.
__device__ __forceinline__ BinCtx make_bin_ctx(const SweepParams &p, const SmemTail &s)
{
    BinCtx c;
    c.lut_lo = __int_as_float(s.meta[1]);
    c.lut_scale = __int_as_float(s.meta[2]);
    c.C = (unsigned)p.lut_cells;
    c.lut = s.lut;
    c.tau_b = reinterpret_cast<const unsigned char *>(s.tau_s);
    c.K4 = 4u * (unsigned)p.K;
    c.one = s.meta[0] != 0;
    c.dscale = __int_as_float(s.meta[4]);
    c.dshift = __int_as_float(s.meta[5]);
    c.K = (unsigned)p.K;
    c.tau_first = s.tau_s[0];
    c.tau_last = s.tau_s[p.K - 1];
    c.arrive_one = (uint32_t)p.one;
    return c;
}
// Start-before-tau rule: the bin (byte offset) of a running time of 0, where every row starts.
__device__ __forceinline__ unsigned bin_of_zero(const BinCtx &c)
{
    return bin_offset<false>(0.0f, c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4);
}

template <int NQ>
__device__ __forceinline__ float &sample_ref(float4 (&v)[NQ], int e)
{
    float4 &q = v[e >> 2];
    switch (e & 3) {
    case 0: return q.x;
    case 1: return q.y;
    case 2: return q.z;
    default: return q.w;
    }
}

// Rule 1 keeps, besides the count of bin-0 samples (cnt0), the largest finish time among them (fin0), and the bin
// `prev` (byte offset) of the running time before the next micro-batch.
// DIRECT = evenly spaced thresholds binned arithmetically (direct_offset) instead of through the table.
template <int NQ, int RULE, bool BATCH, bool DIRECT>
__device__ __forceinline__ void consume_chunk(float4 (&v)[NQ], int ns, bool valid, int lane, const BinCtx &c,
                                              unsigned char *hist_b, unsigned fmax_delta, float &P, unsigned &prev,
                                              int &cnt0, float &fin0, uint64_t *release_bar)
{
    constexpr int GS = NQ >= 2 ? 8 : 4;  // samples per group
    // Running sums of the whole chunk, in place.
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        P = __fadd_rn(P, v[q].x); v[q].x = P;
        P = __fadd_rn(P, v[q].y); v[q].y = P;
        P = __fadd_rn(P, v[q].z); v[q].z = P;
        P = __fadd_rn(P, v[q].w); v[q].w = P;
    }
    // Whole chunk still below the first threshold for every lane of the warp?  The vote needs every lane's last
    // running sum, i.e. every shared-memory read of the stage by this warp has returned; the stage is released
    // only after it, and the count operand of the arrive depends on the vote (arrive_one is 1), so the release
    // cannot move ahead of the reads.
    const bool chunk_low = __all_sync(0xffffffffu, !valid || P < c.tau_first);
    if (release_bar != nullptr && lane == 0) mbar_arrive_count(release_bar, chunk_low ? 1u : c.arrive_one);
    if (chunk_low) {
        // (rule 1: the times before these micro-batches are below the first threshold too, and a positive first
        // threshold puts them, like a time of 0, into bin 0)
        if (valid) {
            cnt0 += ns;
            if (RULE == 1) fin0 = fmaxf(fin0, P);
        }
        return;
    }
#pragma unroll
    for (int g = 0; g < 4 * NQ; g += GS) {
        const int gs = min(GS, ns - g);  // samples of this group that exist (same for all threads)
        if (gs > 0) {
            const float pend = sample_ref(v, g + GS - 1);  // running sum after the group
            if (__all_sync(0xffffffffu, !valid || pend < c.tau_first)) {
                if (valid) {
                    cnt0 += gs;
                    if (RULE == 1) fin0 = fmaxf(fin0, pend);
                }
            } else if (RULE == 1) {
                // Every lane already at or above the last threshold before the group: none of its micro-batches
                // is started under any threshold.
                if (!__all_sync(0xffffffffu, !valid || prev >= c.K4)) {
                    if (valid) {
                        if (c.one && gs == GS) {
                            unsigned off[GS];
                            if (DIRECT) {
#pragma unroll
                                for (int e = 0; e < GS; ++e) off[e] = direct_offset(sample_ref(v, g + e), c.dscale, c.dshift, c.K, c.tau_b);
                            } else {
#pragma unroll
                                for (int e = 0; e < GS; ++e)
                                    off[e] = bin_offset<true>(sample_ref(v, g + e), c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4);
                            }
#pragma unroll
                            for (int e = 0; e < GS; ++e) {
                                start_rule_update(sample_ref(v, g + e), prev, hist_b, fmax_delta, cnt0, fin0);
                                prev = off[e];
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < GS; ++e) {
                                if (e < gs) {
                                    const float Pe = sample_ref(v, g + e);
                                    start_rule_update(Pe, prev, hist_b, fmax_delta, cnt0, fin0);
                                    prev = c.one ? bin_offset<true>(Pe, c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4)
                                                 : bin_offset<false>(Pe, c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4);
                                }
                            }
                        }
                    }
                }
            } else if (!__all_sync(0xffffffffu, !valid || sample_ref(v, g) >= c.tau_last)) {
                if (valid) {
                    if (c.one && gs == GS) {  // the common case, no per-sample predicates
                        if (BATCH) {
                            // all table and threshold reads of the group first (independent chains that
                            // overlap), then the histogram updates: lower latency per group
                            unsigned off[GS];
                            if (DIRECT) {
#pragma unroll
                                for (int e = 0; e < GS; ++e) off[e] = direct_offset(sample_ref(v, g + e), c.dscale, c.dshift, c.K, c.tau_b);
                            } else {
#pragma unroll
                                for (int e = 0; e < GS; ++e)
                                    off[e] = bin_offset<true>(sample_ref(v, g + e), c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4);
                            }
#pragma unroll
                            for (int e = 0; e < GS; ++e) atomicAdd(reinterpret_cast<int *>(hist_b + off[e]), 1);
                        } else if (DIRECT) {
#pragma unroll
                            for (int e = 0; e < GS; ++e)
                                atomicAdd(reinterpret_cast<int *>(hist_b + direct_offset(sample_ref(v, g + e), c.dscale, c.dshift, c.K, c.tau_b)), 1);
                        } else {
#pragma unroll
                            for (int e = 0; e < GS; ++e)
                                bin_sample<true>(sample_ref(v, g + e), c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4, hist_b);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < GS; ++e) {
                            if (e < gs) {
                                if (c.one)
                                    bin_sample<true>(sample_ref(v, g + e), c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4, hist_b);
                                else
                                    bin_sample<false>(sample_ref(v, g + e), c.lut_lo, c.lut_scale, c.C, c.lut, c.tau_b, c.K4, hist_b);
                            }
                        }
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Tiled kernel: TMA-staged rows, persistent over trials.  Warp roles inside a block:
//   warps 0 .. ncw-1   consumers: thread r owns row (pass*rows + r) of the current trial
//   warp  ncw          producer: one thread streams the block's tiles through the ring of stages
//   warp  ncw+1        epilogue: turns a finished trial's histograms into out_done / out_step / out_sync
// The histograms (and the per-warp maxima) are double-buffered: consumers fill buffer j&1 for their j-th
// trial and go straight on to the next trial while the epilogue warp sums, scans, writes and clears the
// buffer.  Named barriers hand the buffers over: kBarReady+b (consumers arrive, epilogue waits) and
// kBarFree+b (epilogue arrives, consumers wait before reusing the buffer two trials later).
// NQ = 16-byte quads of a row per chunk held in registers (box width = 4*NQ floats at most).
// A consumer thread adds its row's samples in order; per group of eight, if every lane of the warp is
// still below the first threshold the samples are bin 0 (one register add); if every lane is at or
// above the last threshold they are in the bin nobody reads; otherwise each running sum is binned
// through the lookup table.
// ------------------------------------------------------------------------------------------
constexpr int kBarReady = 2;  // +0, +1
constexpr int kBarFree = 4;   // +0, +1

// Barrier numbers are compile-time immediates (a run-time number would make the compiler reserve all 16
// hardware barriers for every block); b selects between the two buffers' barriers.
template <int ID>
__device__ __forceinline__ void bar_sync_imm(int threads)
{
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "r"(threads) : "memory");
}
template <int ID>
__device__ __forceinline__ void bar_arrive_imm(int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"n"(ID), "r"(threads) : "memory");
}
template <int BASE>
__device__ __forceinline__ void buffer_barrier_sync(int b, int threads)
{
    if (b == 0) bar_sync_imm<BASE>(threads);
    else bar_sync_imm<BASE + 1>(threads);
}
template <int BASE>
__device__ __forceinline__ void buffer_barrier_arrive(int b, int threads)
{
    if (b == 0) bar_arrive_imm<BASE>(threads);
    else bar_arrive_imm<BASE + 1>(threads);
}

// The epilogue warp's loop (all 32 lanes).  Bins are taken 32 at a time: lane l sums bin k0+l over the
// copies (and clears it), a warp scan gives the prefix, a carry links the blocks of 32.
template <int RULE>
__device__ __forceinline__ void epilogue_warp(const SweepParams &p, const SmemTail &s, int lane, int ncw)
{
    const int K = p.K, H = p.hist_copies, HS = p.hist_stride;
    const int bar_threads = ncw * 32 + 32;
    int j = 0;
    for (long long t = blockIdx.x; t < p.T; t += gridDim.x, ++j) {
        const int b = j & 1;
        buffer_barrier_sync<kBarReady>(b, bar_threads);  // every consumer has finished trial t
        int *hist = s.hist + b * H * HS;
        float *fmax = s.fmax + b * H * HS;  // rule 1 only
        const float Tmax = warp_max(lane < ncw ? s.smax[32 * b + lane] : 0.0f);
        const float t_comm = p.t_comm_vec ? p.t_comm_vec[t] : p.t_comm;
        float *step_row = p.out_step + t * K;
        int32_t *done_row = p.out_done + t * K;
        int carry = 0;
        float fm_carry = 0.0f;
        // Four consecutive bins per lane, 128 bins per step, with 16-byte accesses throughout (when the shapes and
        // pointers allow): a quarter of the scans and well under half the instructions of the scalar loop below.
        for (int k0 = 0; p.epi_vec && k0 < K; k0 += 128) {
            const int k = k0 + 4 * lane;
            const bool in = k < K;  // K is a multiple of 4: a lane's four bins are all inside or all outside
            int4 h = make_int4(0, 0, 0, 0);
            float4 fm = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (in) {
#pragma unroll 2
                for (int c = 0; c < H; ++c) {
                    int4 *hp = reinterpret_cast<int4 *>(hist + c * HS + k);
                    const int4 v = *hp;
                    *hp = make_int4(0, 0, 0, 0);
                    h.x += v.x; h.y += v.y; h.z += v.z; h.w += v.w;
                    if (RULE == 1) {
                        float4 *fp = reinterpret_cast<float4 *>(fmax + c * HS + k);
                        const float4 f = *fp;
                        *fp = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                        fm.x = fmaxf(fm.x, f.x); fm.y = fmaxf(fm.y, f.y); fm.z = fmaxf(fm.z, f.z); fm.w = fmaxf(fm.w, f.w);
                    }
                }
            }
            h.y += h.x; h.z += h.y; h.w += h.z;  // inclusive inside the lane
            const int incl = warp_inclusive_scan(h.w, lane);
            const int base = carry + incl - h.w;  // everything before this lane's bins
            carry += __shfl_sync(0xffffffffu, incl, 31);
            float4 st;
            if (RULE == 0) {
                const float4 tq = in ? *reinterpret_cast<const float4 *>(s.tau_s + k) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                st.x = fminf(tq.x, Tmax); st.y = fminf(tq.y, Tmax); st.z = fminf(tq.z, Tmax); st.w = fminf(tq.w, Tmax);
            } else {
                // max_n W_n(k) = max_{j <= k} fmax[j]
                fm.y = fmaxf(fm.y, fm.x); fm.z = fmaxf(fm.z, fm.y); fm.w = fmaxf(fm.w, fm.z);
                const float fincl = warp_inclusive_max_scan(fm.w, lane);
                float before = __shfl_up_sync(0xffffffffu, fincl, 1);
                before = fmaxf(fm_carry, lane > 0 ? before : 0.0f);
                fm_carry = fmaxf(fm_carry, __shfl_sync(0xffffffffu, fincl, 31));
                st.x = fmaxf(before, fm.x); st.y = fmaxf(before, fm.y); st.z = fmaxf(before, fm.z); st.w = fmaxf(before, fm.w);
            }
            if (in) {
                *reinterpret_cast<int4 *>(done_row + k) = make_int4(base + h.x, base + h.y, base + h.z, base + h.w);
                *reinterpret_cast<float4 *>(step_row + k) =
                    make_float4(__fadd_rn(st.x, t_comm), __fadd_rn(st.y, t_comm), __fadd_rn(st.z, t_comm), __fadd_rn(st.w, t_comm));
            }
        }
        // Otherwise: 32 bins at a time, lane l sums bin k0+l over the copies (and clears it), a warp scan gives the
        // prefix, a carry links the blocks of 32.
        for (int k0 = p.epi_vec ? K : 0; k0 < K; k0 += 32) {
            const int k = k0 + lane;
            int h = 0;
            float fm = 0.0f;
            if (k < K) {
                for (int c = 0; c < H; ++c) {
                    h += hist[c * HS + k];
                    hist[c * HS + k] = 0;
                    if (RULE == 1) {
                        fm = fmaxf(fm, fmax[c * HS + k]);
                        fmax[c * HS + k] = 0.0f;
                    }
                }
            }
            const int incl = warp_inclusive_scan(h, lane);
            float step;
            if (RULE == 0) {
                step = __fadd_rn(fminf(k < K ? s.tau_s[k] : 0.0f, Tmax), t_comm);
            } else {
                const float fm_incl = warp_inclusive_max_scan(fm, lane);
                step = __fadd_rn(fmaxf(fm_carry, fm_incl), t_comm);
                fm_carry = fmaxf(fm_carry, __shfl_sync(0xffffffffu, fm_incl, 31));
            }
            if (k < K) {
                done_row[k] = carry + incl;
                step_row[k] = step;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        for (int c = lane; c < H; c += 32) {  // the two bins past the last threshold
            hist[c * HS + K] = 0;
            hist[c * HS + K + 1] = 0;
        }
        if (RULE == 1) {
            for (int c = lane; c < H; c += 32) {
                fmax[c * HS + K] = 0.0f;
                fmax[c * HS + K + 1] = 0.0f;
            }
        }
        if (lane == 0 && p.out_sync != nullptr) p.out_sync[t] = __fadd_rn(Tmax, t_comm);
        buffer_barrier_arrive<kBarFree>(b, bar_threads);  // buffer b is clear again
    }
}

// The consumer threads' loop over the block's trials (tiled kernel).
template <int NQ, int RULE, bool BATCH, bool DIRECT>
__device__ __forceinline__ void tiled_trials(const SweepParams &p, const SmemTail &s, const BinCtx &ctx, unsigned char *stage0,
                                             uint64_t *full, uint64_t *empty, int tid, int lane, int warp, int ncw,
                                             int *myhist0, unsigned fmax_delta, unsigned off_zero)
{
    const int S = p.stages;
    const int bar_threads = ncw * 32 + 32;
    const int hist_buf_ints = p.hist_copies * p.hist_stride;
    // byte offset of this thread's quad q inside a stage: row_off + ((16 q) ^ swz)
    // (threads past the last row of the box read the last row instead: always inside the stage)
    const uint32_t row_off = (uint32_t)min(tid, p.rows - 1) * (uint32_t)p.pitch;
    const uint32_t swz = ((row_off >> 7) & (uint32_t)p.swz_mask) << 4;
    int st = 0;
    uint32_t ph = 0;
    int j = 0;
    for (long long t = blockIdx.x; t < p.T; t += gridDim.x, ++j) {
        const int b = j & 1;
        if (j >= 2) buffer_barrier_sync<kBarFree>(b, bar_threads);  // the epilogue warp has cleared buffer b
        int *myhist = myhist0 + b * hist_buf_ints;
        unsigned char *hist_b = reinterpret_cast<unsigned char *>(myhist);
        float rowmax = 0.0f, fin0 = 0.0f;
        int cnt0 = 0;
        for (int pass = 0; pass < p.passes; ++pass) {
            const bool valid = (tid < p.rows) && (pass * p.rows + tid < p.N);
            float P = 0.0f;
            unsigned prev = off_zero;  // rule 1: bin (byte offset) of the running time before the next micro-batch
            for (int c = 0; c < p.chunks; ++c) {
                mbar_wait(&full[st], ph, kErrLoadNeverArrived);
                const unsigned char *stage = stage0 + (size_t)st * p.stage_bytes + row_off;
                uint64_t *empty_bar = &empty[st];
                if (++st == S) {
                    st = 0;
                    ph ^= 1u;
                }
                const int nq = (c == p.chunks - 1) ? p.nq_last : NQ;
                float4 v[NQ];
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (q < nq) v[q] = *reinterpret_cast<const float4 *>(stage + ((uint32_t)(q * 16) ^ swz));
                    else v[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                }
                consume_chunk<NQ, RULE, BATCH, DIRECT>(v, 4 * nq, valid, lane, ctx, hist_b, fmax_delta, P, prev, cnt0, fin0, empty_bar);
            }
            if (valid) rowmax = fmaxf(rowmax, P);
        }
        if (cnt0 > 0) {
            atomicAdd(myhist, cnt0);
            if (RULE == 1) raise_max(reinterpret_cast<float *>(hist_b + fmax_delta), fin0);
        }
        rowmax = warp_max(rowmax);
        if (lane == 0) s.smax[32 * b + warp] = rowmax;
        buffer_barrier_arrive<kBarReady>(b, bar_threads);  // hand buffer b to the epilogue warp
    }
}

template <int NQ, int RULE, bool BATCH>
__global__ void __launch_bounds__(kMaxRowsPerPass + 64, NQ <= 4 ? 3 : 2)
dc_sweep_tiled(const __grid_constant__ CUtensorMap lat_map, const SweepParams p)
{
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment by pointer arithmetic on the shared array itself (a round trip through an integer
    // would hide the address space from the compiler and turn every shared access into a generic one)
    unsigned char *smem = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    unsigned char *stage0 = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)p.stages * p.stage_bytes);
    uint64_t *empty = full + kMaxStages;
    const SmemTail s = carve_tail(reinterpret_cast<unsigned char *>(empty + kMaxStages), p);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ncw = (blockDim.x >> 5) - 2;  // consumer warps; then the producer warp, then the epilogue warp
    const int S = p.stages;

    // The producer thread sets up the barriers and fills the whole ring before the block builds its tables: the
    // first tiles are on their way from HBM while the thresholds are read and the lookup table is built.
    // (tile = one chunk of one pass of one trial; the block's tiles in order: trial, pass, chunk)
    long long prod_t = blockIdx.x;
    int prod_pass = 0, prod_c = 0, prod_issued = 0;
    auto issue_tile = [&](int st) {
        mbar_arrive_expect_tx(&full[st], (uint32_t)(p.rows * p.pitch));
        tma_load_3d(stage0 + (size_t)st * p.stage_bytes, &lat_map, prod_c * p.bw, prod_pass * p.rows, (int)prod_t, &full[st]);
        if (++prod_c == p.chunks) {
            prod_c = 0;
            if (++prod_pass == p.passes) {
                prod_pass = 0;
                prod_t += gridDim.x;
            }
        }
    };
    if (warp == ncw && lane == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], ncw);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        while (prod_issued < S && prod_t < p.T) issue_tile(prod_issued++);
    }
    load_thresholds(p, s, tid, blockDim.x);
    __syncthreads();  // also: the initialised barriers are visible to every thread
    build_lut(p, s, tid, blockDim.x);

    if (warp == ncw) {
        // ---------------- producer: the rest of the tiles, each into the stage its predecessor has been read out of
        if (lane == 0) {
            int st = 0;
            uint32_t ph = 1;  // parity of the current use of stage st (every stage has been used once)
            while (prod_t < p.T) {
                mbar_wait(&empty[st], ph ^ 1u, kErrStageNeverFreed);
                issue_tile(st);
                if (++st == S) {
                    st = 0;
                    ph ^= 1u;
                }
            }
        }
        return;
    }
    if (warp == ncw + 1) {
        epilogue_warp<RULE>(p, s, lane, ncw);
        return;
    }

    // ---------------- consumers
    int *myhist0 = s.hist + ((warp % p.warp_groups) * p.lane_copies + (lane & (p.lane_copies - 1))) * p.hist_stride;
    // rule 1: byte distance from a histogram entry to the finish-time maximum of the same buffer, copy and bin
    const unsigned fmax_delta = (unsigned)(reinterpret_cast<unsigned char *>(s.fmax) - reinterpret_cast<unsigned char *>(s.hist));
    const BinCtx ctx = make_bin_ctx(p, s);
    const bool one = ctx.one;
    const unsigned off_zero = RULE == 1 ? bin_of_zero(ctx) : 0u;  // rule 1 only
    if (s.meta[3] != 0 && one && p.direct_bins != 0)
        tiled_trials<NQ, RULE, BATCH, true>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, myhist0, fmax_delta, off_zero);
    else
        tiled_trials<NQ, RULE, BATCH, false>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, myhist0, fmax_delta, off_zero);
}

// ------------------------------------------------------------------------------------------
// Flat kernel: rows whose length is not a multiple of 4 (so a tensor map cannot describe them), up to
// kFlatMaxM samples, and any row length up to that when the base pointer is only 4-byte aligned.  Consecutive rows of a trial are one contiguous span of the
// tensor.  A tile is `rows` consecutive rows (a multiple of 32, at most 32 KB); the producer brings the 16-byte
// aligned span that covers it into a stage with ONE plain bulk copy (cp.async.bulk, no tensor map) and thread r
// of the tile's warps reads its row from float offset delta + r*M with 4-byte shared loads, 32 samples at a time.
// Whole rows have to be resident, so long rows mean few rows per tile: the consumer warps are therefore split
// into G groups of rows/32 warps, tile i goes to group i mod G, and the groups work on different tiles at the
// same time.  The ring has a multiple of G stages, so a stage is only ever used by one group and each group sees
// its own stages in order, like a ring of its own (for short rows G = 1: the tiled kernel's schedule).  Everything
// after the loads is the tiled kernel's code (consume_chunk, epilogue warp, double-buffered histograms).  The
// few floats before the first and after the last 16-byte boundary inside the tensor cannot be bulk-copied in
// bounds; the producer moves them with ordinary loads.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// NQ = 16-byte quads of a row per chunk held in registers: 8 (32 samples), fewer for rows of at most 16 samples.
template <int RULE, bool BATCH, int NQ>
__global__ void __launch_bounds__(kMaxRowsPerPass + 64, 2) dc_sweep_flat(const SweepParams p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    unsigned char *stage0 = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)p.stages * p.stage_bytes);
    uint64_t *empty = full + kMaxStages;
    const SmemTail s = carve_tail(reinterpret_cast<unsigned char *>(empty + kMaxStages), p);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ncw = (blockDim.x >> 5) - 2;
    const int S = p.stages;
    const int R = p.rows, Pt = p.passes, G = p.flat_groups, wpg = p.tile_warps;  // tiles per trial, groups, warps per group
    const unsigned long long NM = (unsigned long long)p.N * (unsigned long long)p.M;
    const unsigned long long total = (unsigned long long)p.T * NM;
    // The base pointer is 4-byte aligned; float i of the tensor sits on a 16-byte boundary iff (i + a) % 4 == 0,
    // where a = floats from the last such boundary to the base.  Bulk copies start and end on such floats INSIDE
    // the tensor; the up to 3 floats before the first and after the last boundary go by ordinary loads.
    const unsigned long long a = (unsigned long long)((reinterpret_cast<uintptr_t>(p.lat) & 15u) >> 2);
    const unsigned long long first4 = (4ull - a) & 3ull;                    // first aligned float of the tensor
    const unsigned long long last4 = total - ((total + a) & 3ull);          // one past the last aligned group

    // the producer thread sets up the barriers and fills the ring before the block builds its tables
    long long prod_t = blockIdx.x;
    int prod_q = 0, prod_issued = 0;  // next tile: trial, tile inside the trial
    auto issue_tile = [&](int st) {
        const int row0 = prod_q * R;
        const int nrows = min(R, p.N - row0);
        const unsigned long long b0 = (unsigned long long)prod_t * NM + (unsigned long long)row0 * p.M;
        const unsigned long long e0 = b0 + (unsigned long long)nrows * p.M;
        // stage float s holds tensor float b0 - delta + s, delta = (b0 + a) % 4: the span's first float keeps
        // its position inside its 16-byte group
        const unsigned long long delta = (b0 + a) & 3ull;
        const unsigned long long c0 = (b0 >= delta) ? b0 - delta : first4;   // aligned start, not before the tensor
        unsigned long long c1 = e0 + ((4ull - ((e0 + a) & 3ull)) & 3ull);     // aligned end, not past the tensor
        if (c1 > last4) c1 = last4;
        if (c1 < c0) c1 = c0;
        float *dst = reinterpret_cast<float *>(stage0 + (size_t)st * p.stage_bytes);
        // floats of the span outside [c0, c1): at most 3 at the very start and 3 at the very end of the tensor
        for (unsigned long long i = b0; i < e0 && i < c0; ++i) dst[i + delta - b0] = p.lat[i];
        for (unsigned long long i = (c1 > b0 ? c1 : b0); i < e0; ++i) dst[i + delta - b0] = p.lat[i];
        const uint32_t bytes = (uint32_t)((c1 - c0) * 4ull);
        mbar_arrive_expect_tx(&full[st], bytes);
        if (bytes != 0u) bulk_load_1d(dst + (c0 + delta - b0), p.lat + c0, bytes, &full[st]);
        if (++prod_q == Pt) {
            prod_q = 0;
            prod_t += gridDim.x;
        }
    };
    if (warp == ncw && lane == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], wpg);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        while (prod_issued < S && prod_t < p.T) issue_tile(prod_issued++);
    }
    load_thresholds(p, s, tid, blockDim.x);
    __syncthreads();  // also: the initialised barriers are visible to every thread
    build_lut(p, s, tid, blockDim.x);

    if (warp == ncw) {
        // ---------------- producer: the rest of the tiles, in order, each into the stage tile i - S has left
        if (lane == 0) {
            int st = 0;
            uint32_t ph = 1;
            while (prod_t < p.T) {
                mbar_wait(&empty[st], ph ^ 1u, kErrStageNeverFreed);
                issue_tile(st);
                if (++st == S) {
                    st = 0;
                    ph ^= 1u;
                }
            }
        }
        return;
    }
    if (warp == ncw + 1) {
        epilogue_warp<RULE>(p, s, lane, ncw);
        return;
    }

    // ---------------- consumers
    const int bar_threads = ncw * 32 + 32;
    const int M = p.M;
    const int hist_buf_ints = p.hist_copies * p.hist_stride;
    int *myhist0 = s.hist + ((warp % p.warp_groups) * p.lane_copies + (lane & (p.lane_copies - 1))) * p.hist_stride;
    const unsigned fmax_delta = (unsigned)(reinterpret_cast<unsigned char *>(s.fmax) - reinterpret_cast<unsigned char *>(s.hist));
    const BinCtx ctx = make_bin_ctx(p, s);
    const unsigned off_zero = RULE == 1 ? bin_of_zero(ctx) : 0u;
    const int grp = warp / wpg;
    const int r = (warp - grp * wpg) * 32 + lane;  // this thread's row inside its group's tiles (< R)
    // The block's tiles are numbered i = 0, 1, ... in the producer's order (trial, then tile inside the trial);
    // tile i uses stage i mod S in ring phase i / S and belongs to group i mod G.  `rel` is this group's next
    // tile counted from the current trial's first tile.
    int rel = grp;
    int st = grp % S;
    uint32_t ph = (uint32_t)((grp / S) & 1);
    int j = 0;
    for (long long t = blockIdx.x; t < p.T; t += gridDim.x, ++j) {
        const int b = j & 1;
        if (j >= 2) buffer_barrier_sync<kBarFree>(b, bar_threads);
        int *myhist = myhist0 + b * hist_buf_ints;
        unsigned char *hist_b = reinterpret_cast<unsigned char *>(myhist);
        float rowmax = 0.0f, fin0 = 0.0f;
        int cnt0 = 0;
        for (; rel < Pt; rel += G) {
            const int row0 = rel * R;
            const bool valid = row0 + r < p.N;
            const unsigned long long b0 = (unsigned long long)t * NM + (unsigned long long)row0 * M;
            const int delta = (int)((b0 + a) & 3ull);
            float P = 0.0f;
            unsigned prev = off_zero;
            mbar_wait(&full[st], ph, kErrLoadNeverArrived);
            // (threads past the tile's last row read row r all the same: inside the stage, never counted)
            const float *row = reinterpret_cast<const float *>(stage0 + (size_t)st * p.stage_bytes) + delta + r * M;
            uint64_t *empty_bar = &empty[st];
            st += G;
            while (st >= S) {
                st -= S;
                ph ^= 1u;
            }
            constexpr int CW = 4 * NQ;  // samples per chunk
            for (int m0 = 0; m0 < M; m0 += CW) {
                const int ns = min(CW, M - m0);
                float4 v[NQ];
#pragma unroll
                for (int e = 0; e < CW; ++e) sample_ref(v, e) = (e < ns) ? row[m0 + e] : 0.0f;
                consume_chunk<NQ, RULE, BATCH, false>(v, ns, valid, lane, ctx, hist_b, fmax_delta, P, prev, cnt0, fin0,
                                                      (m0 + CW >= M) ? empty_bar : nullptr);
            }
            if (valid) rowmax = fmaxf(rowmax, P);
        }
        rel -= Pt;
        if (cnt0 > 0) {
            atomicAdd(myhist, cnt0);
            if (RULE == 1) raise_max(reinterpret_cast<float *>(hist_b + fmax_delta), fin0);
        }
        rowmax = warp_max(rowmax);
        if (lane == 0) s.smax[32 * b + warp] = rowmax;
        buffer_barrier_arrive<kBarReady>(b, bar_threads);
    }
}

// ------------------------------------------------------------------------------------------
// Plain-load kernel for what neither staged kernel takes (rows longer than kFlatMaxM whose length is not a
// multiple of 4 or whose base is only 4-byte aligned).  No TMA: for each chunk of 32 columns a warp loads the
// 32-float pieces of its 32 rows with ordinary coalesced loads (lane = column), parks them in a 32 x 33 tile of
// its own in shared memory and each lane then takes its row's 32 samples from there (lane = row).  The walk is
// the staged kernels' (consume_chunk); the epilogue is done by the whole block per trial.
// ------------------------------------------------------------------------------------------
constexpr int kPlainTileFloats = 32 * 33;

template <int RULE>
__global__ void __launch_bounds__(kMaxRowsPerPass) dc_sweep_plain(const SweepParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;
    float *tile = reinterpret_cast<float *>(smem_raw) + warp * kPlainTileFloats;
    const SmemTail s = carve_tail(smem_raw + (size_t)(nthr >> 5) * kPlainTileFloats * sizeof(float), p);
    load_thresholds(p, s, tid, nthr);
    __syncthreads();
    build_lut(p, s, tid, nthr);

    const int M = p.M;
    const BinCtx ctx = make_bin_ctx(p, s);
    const unsigned off_zero = RULE == 1 ? bin_of_zero(ctx) : 0u;
    int *myhist = s.hist + (warp & (p.hist_copies - 1)) * p.hist_stride;
    unsigned char *hist_b = reinterpret_cast<unsigned char *>(myhist);
    const unsigned fmax_delta = (unsigned)(reinterpret_cast<unsigned char *>(s.fmax) - reinterpret_cast<unsigned char *>(s.hist));

    for (long long t = blockIdx.x; t < p.T; t += gridDim.x) {
        float rowmax = 0.0f, fin0 = 0.0f;
        int cnt0 = 0;
        for (int pass = 0; pass < p.passes; ++pass) {
            const int n0 = pass * p.rows + warp * 32;   // this warp's first row in the trial
            const bool valid = n0 + lane < p.N;
            const int nrows = min(32, p.N - n0);         // rows of this warp that exist (may be <= 0)
            const float *src = p.lat + ((size_t)t * p.N + (size_t)max(n0, 0)) * M;
            float P = 0.0f;
            unsigned prev = off_zero;
            for (int m0 = 0; m0 < M; m0 += 32) {
                const int ns = min(32, M - m0);
                // lane = column: row rr's piece is one coalesced read of up to 128 bytes
#pragma unroll 8
                for (int rr = 0; rr < 32; ++rr) {
                    float x = 0.0f;
                    if (rr < nrows && lane < ns) x = __ldg(src + (size_t)rr * M + m0 + lane);
                    tile[rr * 33 + lane] = x;
                }
                __syncwarp();
                float4 v[8];  // lane = row
#pragma unroll
                for (int e = 0; e < 32; ++e) sample_ref(v, e) = tile[lane * 33 + e];
                __syncwarp();
                consume_chunk<8, RULE, false, false>(v, ns, valid, lane, ctx, hist_b, fmax_delta, P, prev, cnt0, fin0, nullptr);
            }
            if (valid) rowmax = fmaxf(rowmax, P);
        }
        if (cnt0 > 0) {
            atomicAdd(myhist, cnt0);
            if (RULE == 1) raise_max(reinterpret_cast<float *>(hist_b + fmax_delta), fin0);
        }
        trial_epilogue(p, t, rowmax, tid, nthr, kConsumerBarrier, s.tau_s, s.hist, s.smax, s.wtot, s.fmax, s.wmx);
    }
}

// ------------------------------------------------------------------------------------------
// Trial statistics (fp64), two deterministic phases.
// Phase 1: block (column tile of 32 thresholds, chunk of trials): 8 warps take the chunk's trials
// round-robin, lanes are thresholds; per-warp sums are combined in warp order.
// Workspace layout: double part[chunks][4][K] (sum step, sum done as int64 bits, sum done/step,
// sum S) followed by double sync_part[chunks].
// ------------------------------------------------------------------------------------------
constexpr int kRedWarps = 8;

__global__ void __launch_bounds__(kRedWarps * 32, 4)
dc_reduce_partial(const float *__restrict__ step, const int32_t *__restrict__ done, const float *__restrict__ sync,
                  long long T, int K, double NM, int chunks, long long rows_per_chunk, double *ws)
{
    __shared__ double sh[kRedWarps][4][32];
    __shared__ double shs[kRedWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    const int chunk = blockIdx.y;
    const long long t0 = chunk * rows_per_chunk;
    const long long t1 = min(T, t0 + rows_per_chunk);
    double s_step = 0.0, s_ratio = 0.0, s_S = 0.0;
    long long s_done = 0;
    const double nan = __longlong_as_double(0x7ff8000000000000LL);
    const double inv_NM = 1.0 / NM;
    if (k < K) {
        // four rows in flight per thread (the loads do not depend on each other); summed in row order
        for (long long t = t0 + warp; t < t1; t += 4 * kRedWarps) {
            float st_f[4], sy_f[4];
            int dn_i[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long tt = t + (long long)u * kRedWarps;
                const bool ok = tt < t1;
                st_f[u] = ok ? step[tt * K + k] : 1.0f;
                dn_i[u] = ok ? done[tt * K + k] : 0;
                sy_f[u] = (ok && sync) ? sync[tt] : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (t + (long long)u * kRedWarps < t1) {
                    const double st = (double)st_f[u];
                    const double dn = (double)dn_i[u];
                    const double sy = sync ? (double)sy_f[u] : nan;
                    s_step += st;
                    s_done += dn_i[u];
                    const double r = 1.0 / st;  // one division per element; the quotients below are products with it
                    s_ratio += dn * r;
                    s_S += (sy * r) * (dn * inv_NM);
                }
            }
        }
    }
    sh[warp][0][lane] = s_step;
    sh[warp][1][lane] = __longlong_as_double(s_done);
    sh[warp][2][lane] = s_ratio;
    sh[warp][3][lane] = s_S;
    // sum of sync over this chunk (only the first column tile does it)
    double ssum = 0.0;
    if (blockIdx.x == 0 && sync) {
        for (long long t = t0 + threadIdx.x; t < t1; t += kRedWarps * 32) ssum += (double)sync[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
        if (lane == 0) shs[warp] = ssum;
    }
    __syncthreads();
    if (warp == 0 && k < K) {
        double a = 0.0, c = 0.0, d = 0.0;
        long long b = 0;
        for (int w = 0; w < kRedWarps; ++w) {
            a += sh[w][0][lane];
            b += __double_as_longlong(sh[w][1][lane]);
            c += sh[w][2][lane];
            d += sh[w][3][lane];
        }
        double *part = ws + (size_t)chunk * 4 * K;
        part[0 * K + k] = a;
        part[1 * K + k] = __longlong_as_double(b);
        part[2 * K + k] = c;
        part[3 * K + k] = d;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double v = nan;
        if (sync) {
            v = 0.0;
            for (int w = 0; w < kRedWarps; ++w) v += shs[w];
        }
        ws[(size_t)chunks * 4 * K + chunk] = v;
    }
}

// Phase 2: block = 32 thresholds; warp w adds the partial sums of chunks w, w+8, ... and the eight warp sums
// are combined in warp order (a fixed order: reproducible).
__global__ void __launch_bounds__(kRedWarps * 32)
dc_reduce_final(const double *__restrict__ ws, long long T, int K, double NM, int chunks, double *stats, double *baseline)
{
    __shared__ double sh[kRedWarps][4][32];
    __shared__ double shs[kRedWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    double a = 0.0, c = 0.0, d = 0.0;
    long long b = 0;
    if (k < K) {
        for (int ch = warp; ch < chunks; ch += kRedWarps) {
            const double *part = ws + (size_t)ch * 4 * K;
            a += part[0 * K + k];
            b += __double_as_longlong(part[1 * K + k]);
            c += part[2 * K + k];
            d += part[3 * K + k];
        }
    }
    sh[warp][0][lane] = a;
    sh[warp][1][lane] = __longlong_as_double(b);
    sh[warp][2][lane] = c;
    sh[warp][3][lane] = d;
    if (blockIdx.x == 0 && lane == 0) {
        double ssum = 0.0;
        for (int ch = warp; ch < chunks; ch += kRedWarps) ssum += ws[(size_t)chunks * 4 * K + ch];
        shs[warp] = ssum;
    }
    __syncthreads();
    if (warp == 0 && k < K) {
        a = 0.0; c = 0.0; d = 0.0; b = 0;
        for (int w = 0; w < kRedWarps; ++w) {
            a += sh[w][0][lane];
            b += __double_as_longlong(sh[w][1][lane]);
            c += sh[w][2][lane];
            d += sh[w][3][lane];
        }
        const double Td = (double)T;
        stats[DC_STAT_MEAN_STEP * K + k] = a / Td;
        stats[DC_STAT_DONE_FRAC * K + k] = (double)b / (Td * NM);
        stats[DC_STAT_THR * K + k] = (double)b / a;
        stats[DC_STAT_THR_MEAN * K + k] = c / Td;
        stats[DC_STAT_S_EFF * K + k] = d / Td;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double ssum = 0.0;
        for (int w = 0; w < kRedWarps; ++w) ssum += shs[w];
        baseline[0] = ssum / (double)T;
        baseline[1] = ((double)T * NM) / ssum;
    }
}

// tau* = first index of the maximum, NaN never wins (one warp).
__global__ void __launch_bounds__(32)
dc_argmax_kernel(const double *__restrict__ obj, const float *__restrict__ taus, int K, int32_t *out_k, float *out_tau,
                 double *out_value)
{
    const int lane = threadIdx.x;
    int best = -1;
    double bv = 0.0;
    for (int k = lane; k < K; k += 32) {
        const double v = obj[k];
        if (v != v) continue;
        if (best < 0 || v > bv) {
            best = k;
            bv = v;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int ob = __shfl_xor_sync(0xffffffffu, best, o);
        const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const bool take = (ob >= 0) && (best < 0 || ov > bv || (ov == bv && ob < best));
        if (take) {
            best = ob;
            bv = ov;
        }
    }
    if (lane == 0) {
        const double nan = __longlong_as_double(0x7ff8000000000000LL);
        *out_k = best;
        *out_tau = best >= 0 ? taus[best] : __int_as_float(0x7fc00000);
        *out_value = best >= 0 ? bv : nan;
    }
}

// Closed-form companion (App. C.2), one thread per threshold, fp64:
//   Eq. 5/10  E[M~(tau)]/M = (1/M) sum_m Phi((tau - m mu) / sqrt(m sigma^2))
//   Eq. 4/12  E[T] = sqrt(M sigma^2) ((1-g) Phi^-1(1 - 1/N) + g Phi^-1(1 - 1/(e N))) + M mu   (T without T^c)
//   Eq. 11    E[S_eff(tau)] = (E[M~]/M) (E[T] + T^c) / (min(tau, E[T]) + T^c)
// out[0][k], out[1][k], out[2][k] = E[M~]/M, min(tau_k, E[T]) + T^c, E[S_eff]; scalars[0] = E[T].
__global__ void __launch_bounds__(128)
dc_closed_form_kernel(double mu, double sigma, long long M, long long N, double t_comm, double mean_T,
                      const float *__restrict__ taus, int K, double *out, double *scalars)
{
    const double g = 0.57721566490153286061;
    double ET = mean_T;
    if (!(mean_T >= 0.0)) {
        const double z = (1.0 - g) * normcdfinv(1.0 - 1.0 / (double)N) + g * normcdfinv(1.0 - 1.0 / (exp(1.0) * (double)N));
        ET = sqrt((double)M * sigma * sigma) * z + (double)M * mu;
    }
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k == 0) scalars[0] = ET;
    if (k >= K) return;
    const double tau = (double)taus[k];
    double em = 0.0;
    for (long long m = 1; m <= M; ++m) em += normcdf((tau - (double)m * mu) / sqrt((double)m * sigma * sigma));
    const double step = fmin(tau, ET) + t_comm;
    out[0 * (size_t)K + k] = em / (double)M;
    out[1 * (size_t)K + k] = step;
    out[2 * (size_t)K + k] = (em / (double)M) * (ET + t_comm) / step;
}

// Few trials, many workers: dc_simulate_split sweeps every trial as G groups of N/G workers (the tensor is the
// same bytes read as [T*G][N/G][M]) and this kernel puts the groups back together: completed counts add up,
// step times and the synchronous time are maxima (rounding is monotone, so max_g fl(x_g + t_comm) equals
// fl(max_g x_g + t_comm), and min(tau, .) commutes with the maximum).
__global__ void __launch_bounds__(256)
dc_combine_groups(const float *__restrict__ g_step, const int32_t *__restrict__ g_done, const float *__restrict__ g_sync,
                  long long T, int G, int K, float *out_step, int32_t *out_done, float *out_sync)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;  // index into [T][K]
    if (i < T * K) {
        const long long t = i / K;
        const int k = (int)(i - t * K);
        int d = 0;
        float st = g_step[(t * G) * K + k];
        for (int g = 0; g < G; ++g) {
            d += g_done[(t * G + g) * K + k];
            st = fmaxf(st, g_step[(t * G + g) * K + k]);
        }
        out_done[i] = d;
        out_step[i] = st;
    }
    if (out_sync != nullptr && i < T) {
        float sy = g_sync[i * G];
        for (int g = 1; g < G; ++g) sy = fmaxf(sy, g_sync[i * G + g]);
        out_sync[i] = sy;
    }
}

// Data precondition check: counts latencies that are negative, NaN or infinite, and thresholds
// that are NaN or smaller than their predecessor.
__global__ void __launch_bounds__(256)
dc_check_kernel(const float *__restrict__ lat, unsigned long long total, const float *__restrict__ taus, int K,
                unsigned long long *counters)
{
    unsigned long long bad = 0;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const float x = lat[i];
        if (!(x >= 0.0f) || !(x <= 3.402823466e38f)) ++bad;
    }
    if (bad) atomicAdd(&counters[0], bad);
    if (blockIdx.x == 0) {
        unsigned long long badt = 0;
        for (int k = threadIdx.x; k < K; k += blockDim.x) {
            const float x = taus[k];
            if (x != x) ++badt;
            else if (k > 0 && !(taus[k - 1] <= x)) ++badt;
        }
        if (badt) atomicAdd(&counters[1], badt);
    }
}

// Measurement aid: reads a float array once with 16-byte loads (eight in flight per thread) and does nothing
// else.  Its duration on the bytes of a latency tensor is what the memory system allows a read-only pass of
// that size; the sweep kernel's duration is reported next to it.
__global__ void __launch_bounds__(256) dc_read_probe_kernel(const float4 *__restrict__ x, unsigned long long n4, float *sink)
{
    float acc = 0.0f;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 7ull * stride < n4; i += 8ull * stride) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldg(x + i + (unsigned long long)u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc += (v[u].x + v[u].y) + (v[u].z + v[u].w);
    }
    for (; i < n4; i += stride) {
        const float4 v = __ldg(x + i);
        acc += (v.x + v.y) + (v.z + v.w);
    }
    if (acc == -1.0f) *sink = acc;  // never true for latencies >= 0; keeps the loads alive
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
    return fn;
}

struct DeviceInfo {
    int sms = 0;
    int max_smem_optin = 0;
    int smem_per_sm = 0;
};
bool device_info(DeviceInfo *out)
{
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (cache[dev].sms == 0) {
        int sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
        int per_sm = 0;
        if (cudaDeviceGetAttribute(&per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess) return false;
        cache[dev].smem_per_sm = per_sm;
        cache[dev].max_smem_optin = smem;
        cache[dev].sms = sms;
    }
    *out = cache[dev];
    return true;
}

int floor_pow2(int v)
{
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

int g_tune_stages = 0;       // 0 = automatic
int g_tune_lane_copies = 0;  // 0 = automatic
int g_tune_warp_groups = 0;  // 0 = automatic
int g_tune_box_floats = 0;   // 0 = automatic
int g_tune_batch = 0;        // 0 = automatic, 1 = off, 2 = on
int g_tune_direct = 0;       // 0 = automatic (on), 1 = off, 2 = on
int g_tune_flat_tile_warps = 0, g_tune_flat_groups = 0, g_tune_flat_depth = 0;  // flat kernel; all three or none
int g_last_simulate_launches = 0;
int g_last_reduce_launches = 0;
int g_last_argmax_launches = 0;

int validate_simulate(const float *lat, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K,
                      const float *out_step, const int32_t *out_done, int32_t rule)
{
    if (!lat || !taus || !out_step || !out_done) return DC_ERR_NULL;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return DC_ERR_SHAPE;
    if (K > DC_MAX_K) return DC_ERR_RANGE;
    if (N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX || T > (int64_t)INT32_MAX) return DC_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(lat) & 3) || (reinterpret_cast<uintptr_t>(taus) & 3) ||
        (reinterpret_cast<uintptr_t>(out_step) & 3) || (reinterpret_cast<uintptr_t>(out_done) & 3))
        return DC_ERR_ALIGN;
    if (rule != DC_RULE_FINISH_BEFORE_TAU && rule != DC_RULE_START_BEFORE_TAU) return DC_ERR_UNSUPPORTED;
    return DC_OK;
}

bool tiled_ok(const float *lat, int64_t M) { return (M % 4 == 0) && ((reinterpret_cast<uintptr_t>(lat) & 15) == 0); }
bool flat_ok(const float *lat, int64_t M)
{
    return !tiled_ok(lat, M) && M <= kFlatMaxM;  // any 4-byte aligned base (validate_simulate checks that)
}

template <int RULE, bool BATCH, int NQ>
int launch_flat_q(const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di, cudaStream_t stream)
{
    auto kernel = dc_sweep_flat<RULE, BATCH, NQ>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, block, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
    const long long grid = (T < (long long)occ * di.sms) ? T : (long long)occ * di.sms;
    kernel<<<(unsigned)grid, block, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

template <int RULE, bool BATCH>
int launch_flat(const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di, cudaStream_t stream)
{
    // rows of at most 16 samples are one short chunk
    if (p.M <= 4) return launch_flat_q<RULE, BATCH, 1>(p, block, smem, T, di, stream);
    if (p.M <= 8) return launch_flat_q<RULE, BATCH, 2>(p, block, smem, T, di, stream);
    if (p.M <= 16) return launch_flat_q<RULE, BATCH, 4>(p, block, smem, T, di, stream);
    return launch_flat_q<RULE, BATCH, 8>(p, block, smem, T, di, stream);
}

template <int NQ, int RULE, bool BATCH>
int launch_tiled_b(const CUtensorMap &map, const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di,
                   cudaStream_t stream)
{
    auto kernel = dc_sweep_tiled<NQ, RULE, BATCH>;
    // Per instantiation and device: the largest dynamic shared memory opted into so far, and the occupancy of
    // the last (block, smem) asked for -- repeated calls with one shape then cost no runtime queries.
    static std::mutex lock;
    static size_t smem_opted[64] = {};
    static struct { int block; size_t smem; int occ; } last[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DC_ERR_CUDA;
    int occ = 0;
    {
        std::lock_guard<std::mutex> guard(lock);
        if (smem > smem_opted[dev]) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
            smem_opted[dev] = smem;
        }
        if (last[dev].occ > 0 && last[dev].block == block && last[dev].smem == smem) {
            occ = last[dev].occ;
        } else {
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, block, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
            last[dev].block = block;
            last[dev].smem = smem;
            last[dev].occ = occ;
        }
    }
    const long long grid = (T < (long long)occ * di.sms) ? T : (long long)occ * di.sms;
    kernel<<<(unsigned)grid, block, smem, stream>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

template <int NQ, int RULE>
int launch_tiled(const CUtensorMap &map, const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di,
                 cudaStream_t stream)
{
    // rule 1 has one binning path only
    if constexpr (RULE == 0) {
        if (p.batch_lookups) return launch_tiled_b<NQ, RULE, true>(map, p, block, smem, T, di, stream);
    }
    return launch_tiled_b<NQ, RULE, false>(map, p, block, smem, T, di, stream);
}

// Shared-memory layout of a block of the staged kernels (tiled and flat): ring depth, histogram copies, table
// size.  Needs p.stage_bytes, p.chunks and the row-thread count; fills the rest and the dynamic shared bytes.
int choose_block_layout(SweepParams &p, int row_threads, int K, int rule, const DeviceInfo &di, size_t *smem_out,
                        int stage_cap = 3)
{
    p.lut_cells = min(kLutCellsMax, 4 * K);
    // Rows that fit one tile gain from looking up a whole group's bins before touching the histogram (the
    // chains overlap); longer rows measured faster with lookups and updates interleaved.
    p.batch_lookups = g_tune_batch > 0 ? g_tune_batch - 1 : ((p.chunks == 1 || p.short_launch) ? 1 : 0);
    // Arithmetic binning of evenly spaced thresholds measured faster wherever a group's bins are computed before
    // its updates (rows of one tile, and the start-before-tau rule), slower for long rows under the paper's rule.
    p.direct_bins = g_tune_direct > 0 ? g_tune_direct - 1
                                      : ((rule == DC_RULE_START_BEFORE_TAU || p.chunks == 1 || p.short_launch) ? 1 : 0);
    // Shared memory per block: aim at two resident blocks per SM.  Histogram copies: lane l of warp w
    // adds into copy (w % warp_groups) * lane_copies + (l % lane_copies); copies used by one warp start
    // 32 / lane_copies banks apart so that equal bins of different lanes do not collide.
    p.nbuf = 2;
    const int ncw = row_threads / 32;
    const size_t budget2 = (size_t)di.smem_per_sm / 2 - 1024 - 256;  // two blocks per SM
    size_t smem = 0;
    bool fits = false;
    // Candidates: ring depth first (bytes in flight matter most), then histogram copies, from the
    // preferred configuration down to the smallest one.  The first that leaves room for two blocks per
    // SM wins; the smallest one is taken even if only one block fits.
    // (a ring deeper than three tiles measured slower on every workload, whatever the tile size)
    // (a negative stage_cap fixes the ring depth at -stage_cap: the flat kernel's groups x stages per group)
    const int s_max = stage_cap < 0 ? -stage_cap
                                    : (g_tune_stages > 0 ? g_tune_stages : min(stage_cap, max(2, kStageBudgetBytes / p.stage_bytes)));
    const int s_min = stage_cap < 0 ? -stage_cap : (g_tune_stages > 0 ? g_tune_stages : 2);
    const int lc_first = g_tune_lane_copies > 0 ? g_tune_lane_copies : 4;
    const int lc_last = g_tune_lane_copies > 0 ? g_tune_lane_copies : 1;
    const int wg_first = g_tune_warp_groups > 0 ? min(g_tune_warp_groups, ncw) : min(2, ncw);
    const int wg_last = g_tune_warp_groups > 0 ? wg_first : 1;
    const bool forced = g_tune_stages > 0 && g_tune_lane_copies > 0 && g_tune_warp_groups > 0;
    // (when a fixed ring alone is too large for two blocks, the same search runs against one block's limit)
    const size_t ring_min = (size_t)s_min * p.stage_bytes;
    const size_t budget = (stage_cap < 0 && ring_min + 4096 > budget2) ? (size_t)di.max_smem_optin : budget2;
    for (int st = s_max; st >= s_min && !fits; --st) {
        for (int lc = lc_first; lc >= lc_last && !fits; lc >>= 1) {
            for (int wg = wg_first; wg >= wg_last && !fits; wg >>= 1) {
                p.stages = st;
                p.lane_copies = lc;
                p.warp_groups = wg;
                p.hist_copies = wg * lc;
                if (rule == DC_RULE_START_BEFORE_TAU) p.aux_copies = p.hist_copies;
                const int want = lc > 1 ? 32 / lc : 1;
                p.hist_stride = (K + 2 + 3) & ~3;  // a multiple of 4: copies start 16-byte aligned
                while (lc > 1 && p.hist_stride % 32 != want % 32) ++p.hist_stride;
                smem = 1024 + 2 * kMaxStages * sizeof(uint64_t) + (size_t)st * p.stage_bytes +
                       tail_bytes(K, p.nbuf * p.hist_copies, p.hist_stride, p.lut_cells, p.nbuf * p.aux_copies);
                p.epi_vec = (K % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.out_step) & 15) == 0) &&
                            ((reinterpret_cast<uintptr_t>(p.out_done) & 15) == 0);
                const bool smallest = (st == s_min && lc == lc_last && wg == wg_last);
                if (smem <= budget || smallest || forced) fits = true;
            }
        }
    }
    if (!fits) return DC_ERR_RANGE;
    *smem_out = smem;
    return DC_OK;
}

int simulate_impl(const float *lat, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, float t_comm,
                  const float *t_comm_vec, float *out_step, int32_t *out_done, float *out_sync, int32_t rule, void *stream_v)
{
    if (t_comm_vec && (reinterpret_cast<uintptr_t>(t_comm_vec) & 3)) return DC_ERR_ALIGN;
    const int rc = validate_simulate(lat, T, N, M, taus, K, out_step, out_done, rule);
    if (rc != DC_OK) return rc;
    if (out_sync && (reinterpret_cast<uintptr_t>(out_sync) & 3)) return DC_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    DeviceInfo di;
    if (!device_info(&di)) return DC_ERR_CUDA;

    SweepParams p;
    memset(&p, 0, sizeof(p));
    p.lat = lat;
    p.taus = taus;
    p.out_step = out_step;
    p.out_done = out_done;
    p.out_sync = out_sync;
    p.T = T;
    p.N = (int)N;
    p.M = (int)M;
    p.K = K;
    p.t_comm = t_comm;
    p.t_comm_vec = t_comm_vec;
    p.passes = (int)((N + kMaxRowsPerPass - 1) / kMaxRowsPerPass);
    p.rows = (int)((N + p.passes - 1) / p.passes);
    const int row_threads = ((p.rows + 31) / 32) * 32;
    p.hist_stride = K + 1;
    p.hist_copies = floor_pow2(min(row_threads / 32, max(1, kHistBudgetBytes / (int)(sizeof(int) * p.hist_stride))));
    p.lane_copies = 1;
    p.warp_groups = 1;
    p.lut_cells = 0;
    p.one = 1;
    p.nbuf = 1;
    p.batch_lookups = 0;
    p.rule = rule;
    p.aux_copies = rule == DC_RULE_START_BEFORE_TAU ? p.hist_copies : 0;

    if (tiled_ok(lat, M)) {
        EncodeTiledFn encode = get_encode_fn();
        if (!encode) return DC_ERR_CUDA;
        p.bw = (int)(M < 32 ? M : 32);
        // Launches of well under a second's worth of bandwidth (below 1 GiB of latencies) are shaped by their start
        // and their tail: 16-float tiles need fewer registers and less shared memory, so three blocks fit an SM,
        // more loads are in flight from the first microsecond and the last wave is finer.  Measured 5-25 % faster
        // on 0.4 GB inputs of 32- to 128-sample rows, 3-5 % slower on inputs of 2 GB and more.
        p.short_launch = (g_tune_box_floats == 0 && M >= 32 && M % 16 == 0 &&
                          (uint64_t)T * (uint64_t)N * (uint64_t)M * 4ull < (1ull << 30)) ? 1 : 0;
        if ((g_tune_box_floats == 16 && M % 16 == 0) || p.short_launch) p.bw = 16;
        p.chunks = (int)((M + p.bw - 1) / p.bw);
        const int last_cols = (int)(M - (int64_t)(p.chunks - 1) * p.bw);
        p.nq_last = last_cols / 4;
        p.pitch = p.bw * 4;
        CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_NONE;
        p.swz_mask = 0;
        if (p.pitch == 128) { swz = CU_TENSOR_MAP_SWIZZLE_128B; p.swz_mask = 7; }
        else if (p.pitch == 64) { swz = CU_TENSOR_MAP_SWIZZLE_64B; p.swz_mask = 3; }
        else if (p.pitch == 32) { swz = CU_TENSOR_MAP_SWIZZLE_32B; p.swz_mask = 1; }
        p.stage_bytes = ((p.rows * p.pitch + 1023) / 1024) * 1024;
        size_t smem = 0;
        {
            const int lrc0 = choose_block_layout(p, row_threads, K, rule, di, &smem);
            if (lrc0 != DC_OK) return lrc0;
        }

        CUtensorMap map;
        const cuuint64_t gdim[3] = {(cuuint64_t)M, (cuuint64_t)N, (cuuint64_t)T};
        const cuuint64_t gstride[2] = {(cuuint64_t)M * 4, (cuuint64_t)N * (cuuint64_t)M * 4};
        const cuuint32_t box[3] = {(cuuint32_t)p.bw, (cuuint32_t)p.rows, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(lat), gdim, gstride, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DC_ERR_CUDA;

        if (smem > (size_t)di.max_smem_optin) return DC_ERR_RANGE;
        const int block = row_threads + 64;
        const int nq = p.bw / 4;
        int lrc;
        if (rule == DC_RULE_FINISH_BEFORE_TAU) {
            if (nq <= 1) lrc = launch_tiled<1, 0>(map, p, block, smem, T, di, stream);
            else if (nq <= 2) lrc = launch_tiled<2, 0>(map, p, block, smem, T, di, stream);
            else if (nq <= 4) lrc = launch_tiled<4, 0>(map, p, block, smem, T, di, stream);
            else lrc = launch_tiled<8, 0>(map, p, block, smem, T, di, stream);
        } else {
            if (nq <= 1) lrc = launch_tiled<1, 1>(map, p, block, smem, T, di, stream);
            else if (nq <= 2) lrc = launch_tiled<2, 1>(map, p, block, smem, T, di, stream);
            else if (nq <= 4) lrc = launch_tiled<4, 1>(map, p, block, smem, T, di, stream);
            else lrc = launch_tiled<8, 1>(map, p, block, smem, T, di, stream);
        }
        if (lrc == DC_OK) g_last_simulate_launches = 1;
        return lrc;
    }

    if (flat_ok(lat, M)) {
        // Warps per tile wt: the largest power of two whose tile (32 wt whole rows) stays within 32 KB, no more than
        // the trial has rows for.  Eight: one group, three stages (the tiled kernel's schedule).  Fewer: about six
        // consumer warps in G groups with one stage each (the groups overlap each other; measured best on rows of
        // 65, 126 and 255 samples against fewer groups with two stages each and against eight warps).
        int best_wt = 8;
        while (best_wt > 1 && (size_t)best_wt * 32 * (size_t)M * 4 + 32 > 32768) best_wt >>= 1;
        const bool short_rows = best_wt == 8;
        if ((int64_t)best_wt * 32 > N) best_wt = (int)((N + 31) / 32);
        const int tiles = (int)((N + (int64_t)best_wt * 32 - 1) / ((int64_t)best_wt * 32));
        int best_g = short_rows ? 1 : min(best_wt >= 4 ? 2 : 6 / best_wt, tiles);
        int best_d = best_g == 1 ? 3 : 1;
        if (g_tune_flat_tile_warps > 0 && g_tune_flat_groups > 0 && g_tune_flat_depth > 0) {
            best_wt = g_tune_flat_tile_warps;
            if ((int64_t)best_wt * 32 > N) best_wt = (int)((N + 31) / 32);
            best_g = g_tune_flat_groups;
            best_d = g_tune_flat_depth;
            if (best_g * best_wt > 8 || best_g * best_d > kMaxStages) return DC_ERR_RANGE;
        }
        if (best_wt <= 0) return DC_ERR_RANGE;
        const int wt = best_wt;
        p.rows = wt * 32;
        p.tile_warps = wt;
        p.passes = (int)((N + p.rows - 1) / p.rows);
        p.bw = (int)M;
        p.chunks = (int)((M + 31) / 32);
        p.pitch = (int)M * 4;
        p.stage_bytes = (int)((((size_t)p.rows * M * 4 + 32) + 1023) / 1024 * 1024);
        // If the ring and the tables of a large grid do not fit a block's shared memory together, take fewer groups
        // (a single group: three stages, then two).
        const bool forced_split = g_tune_flat_tile_warps > 0 && g_tune_flat_groups > 0 && g_tune_flat_depth > 0;
        int groups = min(best_g, p.passes), depth = best_d;
        if (!forced_split && groups == 1) depth = 3;
        size_t smem = 0;
        int flat_threads = 0;
        for (;;) {
            p.flat_groups = groups;
            flat_threads = groups * wt * 32;
            const int lrc0 = choose_block_layout(p, flat_threads, K, rule, di, &smem, -(groups * depth));
            if (lrc0 == DC_OK && smem <= (size_t)di.max_smem_optin) break;
            if (forced_split) return DC_ERR_RANGE;
            if (groups > 1) {
                --groups;
                depth = groups == 1 ? 3 : 1;
            } else if (depth > 2) {
                depth = 2;
            } else {
                return DC_ERR_RANGE;
            }
        }
        const int block = flat_threads + 64;
        int lrc;
        if (rule == DC_RULE_FINISH_BEFORE_TAU)
            lrc = p.batch_lookups ? launch_flat<0, true>(p, block, smem, T, di, stream) : launch_flat<0, false>(p, block, smem, T, di, stream);
        else
            lrc = launch_flat<1, false>(p, block, smem, T, di, stream);
        if (lrc == DC_OK) g_last_simulate_launches = 1;
        return lrc;
    }

    // plain-load kernel
    p.rows = row_threads;  // one row per thread per pass
    p.passes = (int)((N + p.rows - 1) / p.rows);
    p.hist_stride = (K + 2 + 3) & ~3;
    p.hist_copies = floor_pow2(min(row_threads / 32, max(1, kHistBudgetBytes / (int)(sizeof(int) * p.hist_stride))));
    p.aux_copies = rule == DC_RULE_START_BEFORE_TAU ? p.hist_copies : 0;
    p.lut_cells = min(kLutCellsMax, 4 * K);
    const size_t smem = (size_t)(row_threads / 32) * kPlainTileFloats * sizeof(float) +
                        tail_bytes(K, p.hist_copies, p.hist_stride, p.lut_cells, p.aux_copies);
    if (smem > (size_t)di.max_smem_optin) return DC_ERR_RANGE;
    auto kernel = rule == DC_RULE_FINISH_BEFORE_TAU ? dc_sweep_plain<0> : dc_sweep_plain<1>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, p.rows, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
    const long long grid = (T < (long long)occ * di.sms) ? T : (long long)occ * di.sms;
    kernel<<<(unsigned)grid, p.rows, smem, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    g_last_simulate_launches = 1;
    return DC_OK;
}

struct ReducePlan {
    int chunks;
    long long rows_per_chunk;
};
ReducePlan reduce_plan(int64_t T)
{
    ReducePlan r;
    long long chunks = (T + 31) / 32;
    if (chunks > kReduceChunksMax) chunks = kReduceChunksMax;
    if (chunks < 1) chunks = 1;
    r.rows_per_chunk = (T + chunks - 1) / chunks;
    r.chunks = (int)((T + r.rows_per_chunk - 1) / r.rows_per_chunk);
    return r;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

// Partial sums of dc_reduce_trials_static.  Part of the library image: each GPU that loads the library
// holds these DC_STATIC_SCRATCH_BYTES until the process exits.  In host code this name is only a handle
// for cudaGetSymbolAddress; kernels are given the address that call returns.
static __device__ __align__(256) double g_static_reduce_scratch[kReduceChunksMax * (4 * DC_STATIC_MAX_K + 1)];
static_assert(sizeof(double) * kReduceChunksMax * (4 * DC_STATIC_MAX_K + 1) == DC_STATIC_SCRATCH_BYTES,
              "header and array disagree about the scratch size");

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------
extern "C" {

int dc_simulate(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, float t_comm,
                float *out_step, int32_t *out_done, void *stream)
{
    return simulate_impl(latencies, T, N, M, taus, K, t_comm, nullptr, out_step, out_done, nullptr, DC_RULE_FINISH_BEFORE_TAU, stream);
}

int dc_simulate_ex(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, float t_comm,
                   float *out_step, int32_t *out_done, float *out_sync, int32_t rule, void *stream)
{
    return simulate_impl(latencies, T, N, M, taus, K, t_comm, nullptr, out_step, out_done, out_sync, rule, stream);
}

int dc_simulate_tc(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K,
                   const float *t_comm_trials, float *out_step, int32_t *out_done, float *out_sync, int32_t rule, void *stream)
{
    if (!t_comm_trials) return DC_ERR_NULL;
    return simulate_impl(latencies, T, N, M, taus, K, 0.0f, t_comm_trials, out_step, out_done, out_sync, rule, stream);
}

// Groups per trial for dc_simulate_split: the smallest divisor G of N that gives T*G >= two blocks per SM while
// leaving at least 64 workers per group (else the largest divisor that leaves 64); 1 when nothing is gained.
static int64_t split_groups(int64_t T, int64_t N, int sms)
{
    const int64_t want = 2 * (int64_t)sms;
    if (T >= want || N < 128) return 1;
    int64_t best = 1;
    for (int64_t g = 2; g <= N / 64; ++g) {
        if (N % g != 0) continue;
        best = g;
        if (T * g >= want) break;
    }
    return best;
}

size_t dc_simulate_split_workspace_bytes(int64_t T, int64_t N, int64_t M, int32_t K)
{
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return 0;
    DeviceInfo di;
    if (!device_info(&di)) return 0;
    const int64_t G = split_groups(T, N, di.sms);
    if (G <= 1) return 0;
    return align_up((size_t)T * G * K * 4, 256) * 2 + align_up((size_t)T * G * 4, 256);
}

int dc_simulate_split(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, float t_comm,
                      float *out_step, int32_t *out_done, float *out_sync, int32_t rule, void *workspace,
                      size_t workspace_bytes, void *stream_v)
{
    const int rc = validate_simulate(latencies, T, N, M, taus, K, out_step, out_done, rule);
    if (rc != DC_OK) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return DC_ERR_CUDA;
    const int64_t G = split_groups(T, N, di.sms);
    if (G <= 1) return simulate_impl(latencies, T, N, M, taus, K, t_comm, nullptr, out_step, out_done, out_sync, rule, stream_v);
    if (T * G > (int64_t)INT32_MAX) return DC_ERR_RANGE;
    const size_t need = align_up((size_t)T * G * K * 4, 256) * 2 + align_up((size_t)T * G * 4, 256);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return DC_ERR_WORKSPACE;
    unsigned char *w = static_cast<unsigned char *>(workspace);
    float *g_step = reinterpret_cast<float *>(w);
    w += align_up((size_t)T * G * K * 4, 256);
    int32_t *g_done = reinterpret_cast<int32_t *>(w);
    w += align_up((size_t)T * G * K * 4, 256);
    float *g_sync = reinterpret_cast<float *>(w);
    const int src = simulate_impl(latencies, T * G, N / G, M, taus, K, t_comm, nullptr, g_step, g_done, g_sync, rule, stream_v);
    if (src != DC_OK) return src;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const long long items = (long long)T * K > T ? (long long)T * K : T;
    dc_combine_groups<<<(unsigned)((items + 255) / 256), 256, 0, stream>>>(g_step, g_done, g_sync, T, (int)G, K, out_step, out_done, out_sync);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    g_last_simulate_launches = 2;
    return DC_OK;
}

int dc_simulate_plan(const float *latencies, int64_t T, int64_t N, int64_t M, int32_t K)
{
    if (!latencies) return -DC_ERR_NULL;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return -DC_ERR_SHAPE;
    if (K > DC_MAX_K || N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX || T > (int64_t)INT32_MAX)
        return -DC_ERR_RANGE;
    if (reinterpret_cast<uintptr_t>(latencies) & 3) return -DC_ERR_ALIGN;
    return tiled_ok(latencies, M) ? 0 : (flat_ok(latencies, M) ? 2 : 1);
}

size_t dc_reduce_workspace_bytes(int64_t T, int32_t K)
{
    if (T <= 0 || K <= 0) return 0;
    const ReducePlan r = reduce_plan(T);
    return sizeof(double) * ((size_t)r.chunks * 4 * (size_t)K + (size_t)r.chunks);
}

int dc_reduce_trials(const float *out_step, const int32_t *out_done, const float *out_sync, int64_t T, int32_t K, int64_t N,
                     int64_t M, double *stats, double *baseline, void *workspace, size_t workspace_bytes, void *stream_v)
{
    if (!out_step || !out_done || !stats || !baseline) return DC_ERR_NULL;
    if (T <= 0 || K <= 0 || N <= 0 || M <= 0) return DC_ERR_SHAPE;
    if (K > DC_MAX_K || N * M > (int64_t)INT32_MAX) return DC_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(stats) & 7) || (reinterpret_cast<uintptr_t>(baseline) & 7)) return DC_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 7) || workspace_bytes < dc_reduce_workspace_bytes(T, K))
        return DC_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const ReducePlan r = reduce_plan(T);
    const double NM = (double)N * (double)M;
    double *ws = static_cast<double *>(workspace);
    dim3 grid1((unsigned)((K + 31) / 32), (unsigned)r.chunks);
    dc_reduce_partial<<<grid1, kRedWarps * 32, 0, stream>>>(out_step, out_done, out_sync, T, K, NM, r.chunks, r.rows_per_chunk, ws);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    dc_reduce_final<<<(unsigned)((K + 31) / 32), kRedWarps * 32, 0, stream>>>(ws, T, K, NM, r.chunks, stats, baseline);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    g_last_reduce_launches = 2;
    return DC_OK;
}

int dc_reduce_trials_static(const float *out_step, const int32_t *out_done, const float *out_sync, int64_t T, int32_t K,
                            int64_t N, int64_t M, double *stats, double *baseline, void *stream_v)
{
    if (!out_step || !out_done || !stats || !baseline) return DC_ERR_NULL;
    if (T <= 0 || K <= 0 || N <= 0 || M <= 0) return DC_ERR_SHAPE;
    if (K > DC_STATIC_MAX_K || N * M > (int64_t)INT32_MAX) return DC_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(stats) & 7) || (reinterpret_cast<uintptr_t>(baseline) & 7)) return DC_ERR_ALIGN;
    // Device address of the built-in scratch, looked up once per device with that device current.
    static std::mutex lock;
    static double *scratch_of_device[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DC_ERR_CUDA;
    double *ws = nullptr;
    {
        std::lock_guard<std::mutex> guard(lock);
        if (scratch_of_device[dev] == nullptr) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_reduce_scratch) != cudaSuccess || ptr == nullptr) return DC_ERR_CUDA;
            scratch_of_device[dev] = static_cast<double *>(ptr);
        }
        ws = scratch_of_device[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const ReducePlan r = reduce_plan(T);  // at most kReduceChunksMax chunks, whatever T is
    const double NM = (double)N * (double)M;
    dim3 grid1((unsigned)((K + 31) / 32), (unsigned)r.chunks);
    dc_reduce_partial<<<grid1, kRedWarps * 32, 0, stream>>>(out_step, out_done, out_sync, T, K, NM, r.chunks, r.rows_per_chunk, ws);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    dc_reduce_final<<<(unsigned)((K + 31) / 32), kRedWarps * 32, 0, stream>>>(ws, T, K, NM, r.chunks, stats, baseline);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    return DC_OK;
}

int dc_argmax_tau(const double *stats, const float *taus, int32_t K, int32_t objective, int32_t *out_k, float *out_tau,
                  double *out_value, void *stream_v)
{
    if (!stats || !taus || !out_k || !out_tau || !out_value) return DC_ERR_NULL;
    if (K <= 0) return DC_ERR_SHAPE;
    if (K > DC_MAX_K) return DC_ERR_RANGE;
    if (objective != DC_STAT_S_EFF && objective != DC_STAT_THR && objective != DC_STAT_THR_MEAN) return DC_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(stats) & 7) || (reinterpret_cast<uintptr_t>(out_value) & 7)) return DC_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    dc_argmax_kernel<<<1, 32, 0, stream>>>(stats + (size_t)objective * K, taus, K, out_k, out_tau, out_value);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    g_last_argmax_launches = 1;
    return DC_OK;
}

int dc_sweep_device(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, float t_comm,
                    int32_t rule, int32_t objective, float *out_step, int32_t *out_done, float *out_sync, double *stats,
                    double *baseline, int32_t *out_k, float *out_tau, double *out_value, void *workspace,
                    size_t workspace_bytes, void *stream)
{
    // everything the three steps would refuse is refused before the first of them is enqueued
    if (!out_sync || !stats || !baseline || !out_k || !out_tau || !out_value) return DC_ERR_NULL;
    int rc = validate_simulate(latencies, T, N, M, taus, K, out_step, out_done, rule);
    if (rc != DC_OK) return rc;
    if (objective != DC_STAT_S_EFF && objective != DC_STAT_THR && objective != DC_STAT_THR_MEAN) return DC_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(stats) & 7) || (reinterpret_cast<uintptr_t>(baseline) & 7) ||
        (reinterpret_cast<uintptr_t>(out_value) & 7) || (reinterpret_cast<uintptr_t>(out_sync) & 3))
        return DC_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 7) || workspace_bytes < dc_reduce_workspace_bytes(T, K))
        return DC_ERR_WORKSPACE;
    rc = simulate_impl(latencies, T, N, M, taus, K, t_comm, nullptr, out_step, out_done, out_sync, rule, stream);
    if (rc != DC_OK) return rc;
    rc = dc_reduce_trials(out_step, out_done, out_sync, T, K, N, M, stats, baseline, workspace, workspace_bytes, stream);
    if (rc != DC_OK) return rc;
    return dc_argmax_tau(stats, taus, K, objective, out_k, out_tau, out_value, stream);
}

int dc_closed_form(double mu, double sigma, int64_t M, int64_t N, double t_comm, double mean_T, const float *taus,
                   int32_t K, double *out, double *scalars, void *stream_v)
{
    if (!taus || !out || !scalars) return DC_ERR_NULL;
    if (M <= 0 || N < 2 || K <= 0) return DC_ERR_SHAPE;
    if (K > DC_MAX_K || !(sigma > 0.0) || !(sigma < 1e300) || !(mu == mu) || !(t_comm == t_comm)) return DC_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(out) & 7) || (reinterpret_cast<uintptr_t>(scalars) & 7) ||
        (reinterpret_cast<uintptr_t>(taus) & 3))
        return DC_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    dc_closed_form_kernel<<<(unsigned)((K + 127) / 128), 128, 0, stream>>>(mu, sigma, M, N, t_comm, mean_T, taus, K, out, scalars);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

int dc_check_inputs(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K, int64_t *counters,
                    int64_t *report_host, void *stream_v)
{
    if (!latencies || !taus || !counters) return DC_ERR_NULL;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return DC_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(counters) & 7) return DC_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    DeviceInfo di;
    if (!device_info(&di)) return DC_ERR_CUDA;
    if (cudaMemsetAsync(counters, 0, 16, stream) != cudaSuccess) return DC_ERR_CUDA;
    const unsigned long long total = (unsigned long long)T * (unsigned long long)N * (unsigned long long)M;
    unsigned long long want = (total + 255) / 256;
    const unsigned grid = (unsigned)(want < (unsigned long long)di.sms * 8 ? (want ? want : 1) : (unsigned long long)di.sms * 8);
    dc_check_kernel<<<grid, 256, 0, stream>>>(latencies, total, taus, K, reinterpret_cast<unsigned long long *>(counters));
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
    int64_t host[2] = {0, 0};
    if (cudaMemcpyAsync(host, counters, 16, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return DC_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return DC_ERR_CUDA;
    if (report_host) {
        report_host[0] = host[0];
        report_host[1] = host[1];
    }
    if (host[0] != 0) return DC_ERR_LATENCIES;
    if (host[1] != 0) return DC_ERR_TAUS;
    return DC_OK;
}

int dc_read_probe(const float *data, int64_t count, float *sink, void *stream_v)
{
    if (!data || !sink) return DC_ERR_NULL;
    if (count <= 0) return DC_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(data) & 15) || (reinterpret_cast<uintptr_t>(sink) & 3)) return DC_ERR_ALIGN;
    DeviceInfo di;
    if (!device_info(&di)) return DC_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    dc_read_probe_kernel<<<(unsigned)(8 * di.sms), 256, 0, stream>>>(reinterpret_cast<const float4 *>(data),
                                                                     (unsigned long long)count / 4ull, sink);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

int dc_device_status(uint32_t *flags_host)
{
    unsigned int flags = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&flags, g_wait_expired, sizeof(flags)) != cudaSuccess) return DC_ERR_CUDA;
    if (flags != 0 && cudaMemcpyToSymbol(g_wait_expired, &zero, sizeof(zero)) != cudaSuccess) return DC_ERR_CUDA;
    if (flags_host) *flags_host = flags;
    return flags == 0 ? DC_OK : DC_ERR_DEVICE;
}

size_t dc_sweep_host_workspace_bytes(int64_t T, int64_t N, int64_t M, int32_t K, int64_t chunk_trials)
{
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0 || chunk_trials <= 0) return 0;
    if (chunk_trials > T) chunk_trials = T;
    const size_t chunk = align_up((size_t)chunk_trials * (size_t)N * (size_t)M * 4, 1024);
    size_t total = 2 * chunk;
    total += align_up((size_t)K * 4, 256);                       // taus
    total += align_up((size_t)T * (size_t)K * 4, 256) * 2;       // step, done
    total += align_up((size_t)T * 4, 256);                       // sync
    total += align_up((size_t)DC_NSTATS * (size_t)K * 8, 256);   // stats
    total += 256;                                                // baseline[2], value, k, tau
    total += align_up(dc_reduce_workspace_bytes(T, K), 256);
    return total;
}

int dc_sweep_host(const float *latencies_host, int64_t T, int64_t N, int64_t M, const float *taus_host, int32_t K,
                  float t_comm, int32_t rule, int32_t objective, int64_t chunk_trials, double *stats_host,
                  double *baseline_host, int32_t *k_star_host, float *tau_star_host, void *workspace, size_t workspace_bytes,
                  void *stream_v)
{
    if (!latencies_host || !taus_host || !stats_host || !baseline_host || !k_star_host || !tau_star_host) return DC_ERR_NULL;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0 || chunk_trials <= 0) return DC_ERR_SHAPE;
    if (K > DC_MAX_K || N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX || T > (int64_t)INT32_MAX)
        return DC_ERR_RANGE;
    if (rule != DC_RULE_FINISH_BEFORE_TAU && rule != DC_RULE_START_BEFORE_TAU) return DC_ERR_UNSUPPORTED;
    if (objective != DC_STAT_S_EFF && objective != DC_STAT_THR && objective != DC_STAT_THR_MEAN) return DC_ERR_UNSUPPORTED;
    if (chunk_trials > T) chunk_trials = T;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 1023) ||
        workspace_bytes < dc_sweep_host_workspace_bytes(T, N, M, K, chunk_trials))
        return DC_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    // carve the workspace
    unsigned char *w = static_cast<unsigned char *>(workspace);
    const size_t chunk_bytes = align_up((size_t)chunk_trials * (size_t)N * (size_t)M * 4, 1024);
    float *buf[2] = {reinterpret_cast<float *>(w), reinterpret_cast<float *>(w + chunk_bytes)};
    w += 2 * chunk_bytes;
    float *d_taus = reinterpret_cast<float *>(w);
    w += align_up((size_t)K * 4, 256);
    float *d_step = reinterpret_cast<float *>(w);
    w += align_up((size_t)T * (size_t)K * 4, 256);
    int32_t *d_done = reinterpret_cast<int32_t *>(w);
    w += align_up((size_t)T * (size_t)K * 4, 256);
    float *d_sync = reinterpret_cast<float *>(w);
    w += align_up((size_t)T * 4, 256);
    double *d_stats = reinterpret_cast<double *>(w);
    w += align_up((size_t)DC_NSTATS * (size_t)K * 8, 256);
    double *d_base = reinterpret_cast<double *>(w);        // [2]
    double *d_value = d_base + 2;
    int32_t *d_k = reinterpret_cast<int32_t *>(d_base + 3);
    float *d_tau = reinterpret_cast<float *>(d_base + 4);
    w += 256;
    void *d_red = w;
    const size_t red_bytes = dc_reduce_workspace_bytes(T, K);

    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ready[2] = {nullptr, nullptr}, freed[2] = {nullptr, nullptr};
    int rc = DC_OK;
    bool cuda_fail = false;
#define DC_TRY(call)                                  \
    do {                                              \
        if (!cuda_fail && (call) != cudaSuccess) {    \
            cuda_fail = true;                         \
        }                                             \
    } while (0)
    DC_TRY(cudaStreamCreateWithFlags(&copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
        DC_TRY(cudaEventCreateWithFlags(&ready[i], cudaEventDisableTiming));
        DC_TRY(cudaEventCreateWithFlags(&freed[i], cudaEventDisableTiming));
    }
    DC_TRY(cudaMemcpyAsync(d_taus, taus_host, (size_t)K * 4, cudaMemcpyHostToDevice, stream));
    int launches = 0;
    const int64_t nchunks = (T + chunk_trials - 1) / chunk_trials;
    for (int64_t c = 0; c < nchunks && !cuda_fail && rc == DC_OK; ++c) {
        const int b = (int)(c & 1);
        const int64_t t0 = c * chunk_trials;
        const int64_t tn = (t0 + chunk_trials <= T) ? chunk_trials : (T - t0);
        if (c >= 2) DC_TRY(cudaStreamWaitEvent(copy_stream, freed[b], 0));
        DC_TRY(cudaMemcpyAsync(buf[b], latencies_host + (size_t)t0 * N * M, (size_t)tn * N * M * 4, cudaMemcpyHostToDevice,
                               copy_stream));
        DC_TRY(cudaEventRecord(ready[b], copy_stream));
        DC_TRY(cudaStreamWaitEvent(stream, ready[b], 0));
        if (!cuda_fail) {
            rc = simulate_impl(buf[b], tn, N, M, d_taus, K, t_comm, nullptr, d_step + (size_t)t0 * K, d_done + (size_t)t0 * K,
                               d_sync + t0, rule, stream);
            launches += 1;
        }
        DC_TRY(cudaEventRecord(freed[b], stream));
    }
    if (!cuda_fail && rc == DC_OK)
        rc = dc_reduce_trials(d_step, d_done, d_sync, T, K, N, M, d_stats, d_base, d_red, red_bytes, stream);
    if (!cuda_fail && rc == DC_OK) rc = dc_argmax_tau(d_stats, d_taus, K, objective, d_k, d_tau, d_value, stream);
    if (!cuda_fail && rc == DC_OK) {
        DC_TRY(cudaMemcpyAsync(stats_host, d_stats, (size_t)DC_NSTATS * K * 8, cudaMemcpyDeviceToHost, stream));
        DC_TRY(cudaMemcpyAsync(baseline_host, d_base, 16, cudaMemcpyDeviceToHost, stream));
        DC_TRY(cudaMemcpyAsync(k_star_host, d_k, 4, cudaMemcpyDeviceToHost, stream));
        DC_TRY(cudaMemcpyAsync(tau_star_host, d_tau, 4, cudaMemcpyDeviceToHost, stream));
    }
    // always drain both streams before the events and the copy stream go away
    if (copy_stream) cudaStreamSynchronize(copy_stream);
    if (cudaStreamSynchronize(stream) != cudaSuccess) cuda_fail = true;
#undef DC_TRY
    for (int i = 0; i < 2; ++i) {
        if (ready[i]) cudaEventDestroy(ready[i]);
        if (freed[i]) cudaEventDestroy(freed[i]);
    }
    if (copy_stream) cudaStreamDestroy(copy_stream);
    if (cuda_fail) return DC_ERR_CUDA;
    if (rc == DC_OK) g_last_simulate_launches = launches;
    return rc;
}

int dc_tune(int32_t key, int32_t value)
{
    if (key == DC_TUNE_STAGES && (value == 0 || (value >= 2 && value <= kMaxStages))) {
        g_tune_stages = value;
        return DC_OK;
    }
    if (key == DC_TUNE_LANE_COPIES && (value == 0 || value == 1 || value == 2 || value == 4 || value == 8)) {
        g_tune_lane_copies = value;
        return DC_OK;
    }
    if (key == DC_TUNE_WARP_GROUPS && value >= 0 && value <= 8) {
        g_tune_warp_groups = value;
        return DC_OK;
    }
    if (key == DC_TUNE_BATCH_LOOKUPS && value >= 0 && value <= 2) {
        g_tune_batch = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_TILE_WARPS && value >= 0 && value <= 8) {
        g_tune_flat_tile_warps = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_GROUPS && value >= 0 && value <= 8) {
        g_tune_flat_groups = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_DEPTH && value >= 0 && value <= 4) {
        g_tune_flat_depth = value;
        return DC_OK;
    }
    if (key == DC_TUNE_DIRECT_BINS && value >= 0 && value <= 2) {
        g_tune_direct = value;
        return DC_OK;
    }
    if (key == DC_TUNE_BOX_FLOATS && (value == 0 || value == 16 || value == 32)) {
        g_tune_box_floats = value;
        return DC_OK;
    }
    return DC_ERR_UNSUPPORTED;
}

int dc_simulate_launches(void) { return g_last_simulate_launches; }
int dc_reduce_trials_launches(void) { return g_last_reduce_launches; }
int dc_argmax_tau_launches(void) { return g_last_argmax_launches; }

const char *dc_kernel_version(void) { return "sweep-tiled-13"; }

const char *dc_status_string(int status)
{
    switch (status) {
    case DC_OK: return "ok";
    case DC_ERR_NULL: return "a required pointer is NULL";
    case DC_ERR_SHAPE: return "T, N, M and K must be positive";
    case DC_ERR_ALIGN: return "a pointer is not aligned as documented";
    case DC_ERR_RANGE: return "a size is beyond what the library supports";
    case DC_ERR_TAUS: return "thresholds are not non-decreasing or contain NaN";
    case DC_ERR_CUDA: return "a CUDA call failed";
    case DC_ERR_UNSUPPORTED: return "unknown rule or objective";
    case DC_ERR_LATENCIES: return "latencies contain a negative, NaN or infinite value";
    case DC_ERR_WORKSPACE: return "workspace is NULL, misaligned or too small";
    case DC_ERR_DEVICE: return "a bounded wait inside a kernel expired";
    default: return "unknown status";
    }
}

}  // extern "C"
