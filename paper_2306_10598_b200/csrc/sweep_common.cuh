// Shared by the three sweep kernels: parameters, PTX wrappers, the shared-memory carve-up, threshold tables,
// binning, and what a consumer thread does with one chunk of its row.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// constants
// ------------------------------------------------------------------------------------------
constexpr int kMaxRowsPerPass = 256;          // rows (threads) of one trial handled per pass; also the TMA box limit
constexpr int kMaxStages = 8;
constexpr int kStageBudgetBytes = 96 * 1024;  // shared memory spent on the ring of stages per block
constexpr int kHistBudgetBytes = 32 * 1024;   // shared memory spent on per-warp histograms per block
constexpr uint32_t kWaitHintNs = 10000;       // longest one try of an mbarrier wait may keep the thread parked
constexpr uint32_t kWaitLimit = 1u << 20;     // tries of one mbarrier wait before giving up (a fraction of a second to a few seconds)
constexpr int kReduceChunksMax = 64;          // partial sums per threshold in dc_reduce_trials
constexpr int kConsumerBarrier = 1;           // named barrier used by the consumer warps
constexpr int kFlatMaxM = 255;                // longest row the flat kernel can take (32 rows of it fill a 32 KB stage)
constexpr int kFlatAutoMaxM = 127;            // longest row it is given by default (32 rows within 16 KB)
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
    int grid_mode;     // host only: DC_TUNE_EVEN_GRID
    int epi_vec;       // staged kernels: the epilogue warp may take four bins per lane with 16-byte accesses
                       // (K a multiple of 4, out_step / out_done 16-byte aligned, hist_stride a multiple of 4)
    int box_y;         // tiled kernel: height of one pass in the tensor map's second coordinate (rows, or 128-byte lines
                       // when rows shorter than a line are fetched as whole lines)
    int g;             // staged kernels: trials per tile (several whole trials share a tile; else 1)
    int tile_y, tile_z;  // tiled kernel: what one tile adds to the tensor map's second and third coordinate (0, 1 for a
                       // tile of one trial; 0, g for g whole trials in one pass; g N, 0 for g trials whose rows are
                       // taken as one run of g N consecutive rows of the [T N][M] view, cut into equal passes)
    int epi_sub;       // tiled kernel, g > 1: lanes of the epilogue warp per trial (K/4, a power of two), or 0 for one
                       // trial at a time
    int lean;          // tiled kernel: 1 = every chunk of a row is full, so the short form of the consumer loop applies
    int spare;         // 1 = one more histogram copy (and finish-time copy) after the real ones, which nothing reads:
                       // lanes without a row of their own add there
};
// copies of one trial's histogram in shared memory, over all buffers and trials of a tile, plus the spare one
__host__ __device__ inline int hist_slots(const SweepParams &p) { return p.nbuf * p.g * p.hist_copies + p.spare; }
__host__ __device__ inline int fmax_slots(const SweepParams &p) { return p.aux_copies ? p.nbuf * p.g * p.aux_copies + p.spare : 0; }

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
// One try: the hardware may park the thread for up to kWaitHintNs before it answers "not yet", so a waiting warp
// costs the scheduler next to nothing instead of spinning through issue slots that other warps could use.
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity), "r"(kWaitHintNs)
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

// Shared-memory accesses by 32-bit shared-window address, for the consumer loop.  Through ordinary pointers every
// address there is a 64-bit sum (two integer instructions per access, and the bins need two accesses per sample); a
// 32-bit base plus a byte offset is one.  The increments are the constant 1 on purpose: for that the assembler emits
// the form of the shared-memory atomic that adds up lanes with equal addresses in one step, whereas a variable
// increment serialises them (measured: eight times the bank conflicts).
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));  // thresholds and tables: written once before the block's first barrier
    return v;
}
__device__ __forceinline__ unsigned lds_u16(uint32_t addr)
{
    unsigned short v;
    asm("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds_stage_f32x4(uint32_t addr)
{
    float4 v;  // volatile: stays between the wait for the stage and its release
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void red_shared_inc(uint32_t addr)
{
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr));
}
__device__ __forceinline__ void red_shared_max(uint32_t addr, int v)
{
    asm volatile("red.shared.max.s32 [%0], %1;" ::"r"(addr), "r"(v));
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
                         // [3] the thresholds are evenly spaced enough for direct binning, [4..5] its scale, shift,
                         // [6] the last finite threshold (as bits)
    unsigned short *lut; // lut_cells + 1 entries (tiled kernel only)
    float *wmx;          // rule 1, plain kernel: warp totals of the prefix-maximum scan
    float *fmax;         // rule 1: [nbuf][g][hist_copies][hist_stride], laid out like hist: largest finish time among
                         // the micro-batches whose start time lies in the bin
    int *segmax;         // staged kernels: [nbuf][g] largest row total of each trial of a tile (bit pattern of a
                         // non-negative float, raised with atomicMax)
};
__device__ __forceinline__ SmemTail carve_tail(unsigned char *base, const SweepParams &p)
{
    SmemTail s;
    s.tau_s = reinterpret_cast<float *>(base);
    s.hist = reinterpret_cast<int *>(s.tau_s + ((p.K + 4) & ~3));  // K + 1 thresholds, padded to 16 bytes
    s.smax = reinterpret_cast<float *>(s.hist + hist_slots(p) * p.hist_stride);
    s.wtot = reinterpret_cast<int *>(s.smax + 32);
    s.meta = s.wtot + 32;
    s.lut = reinterpret_cast<unsigned short *>(s.meta + 8);
    s.wmx = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(s.lut) +
                                      (((size_t)(p.lut_cells + 1) * sizeof(unsigned short) + 15) & ~(size_t)15));
    s.fmax = s.wmx + 32;
    s.segmax = reinterpret_cast<int *>(s.fmax + fmax_slots(p) * p.hist_stride);
    return s;
}
// hist_copies and fmax_copies count all buffers and trials of a tile and the spare copy (hist_slots, fmax_slots);
// seg_slots = nbuf * g
__host__ __device__ inline size_t tail_bytes(int K, int hist_copies, int hist_stride, int lut_cells, int fmax_copies,
                                             int seg_slots = 0)
{
    return sizeof(float) * (size_t)((K + 4) & ~3) + sizeof(int) * (size_t)hist_copies * hist_stride + 72 * sizeof(int) +
           (((size_t)(lut_cells + 1) * sizeof(unsigned short) + 15) & ~(size_t)15) + 32 * sizeof(float) +
           sizeof(float) * (size_t)fmax_copies * hist_stride + sizeof(int) * (size_t)((seg_slots + 3) & ~3);
}

__device__ __forceinline__ void load_thresholds(const SweepParams &p, const SmemTail &s, int tid, int nthr)
{
    for (int k = tid; k < p.K; k += nthr) s.tau_s[k] = p.taus[k];
    if (tid == 0) s.tau_s[p.K] = __int_as_float(0x7f800000);  // +inf sentinel
    for (int i = tid; i < hist_slots(p) * p.hist_stride; i += nthr) s.hist[i] = 0;
    for (int i = tid; i < fmax_slots(p) * p.hist_stride; i += nthr) s.fmax[i] = 0.0f;
    for (int i = tid; i < p.nbuf * p.g; i += nthr) s.segmax[i] = 0;
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
        s.meta[6] = __float_as_int(klo <= khi ? s.tau_s[khi] : ninf);  // the last finite threshold (-inf if none)
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
    uint32_t lut_a, tau_a;    // the same two as shared-window addresses
    unsigned K4;
    bool one;                 // the table guarantees at most one threshold to step over
    float dscale, dshift;     // direct binning (only used when the grid qualifies)
    unsigned K;
    float tau_first, tau_last;
    float tau_top;            // the last FINITE threshold: running sums below it have a cell inside the tables
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
    c.lut_a = smem_addr(s.lut);
    c.tau_a = smem_addr(s.tau_s);
    c.K4 = 4u * (unsigned)p.K;
    c.one = s.meta[0] != 0;
    c.dscale = __int_as_float(s.meta[4]);
    c.dshift = __int_as_float(s.meta[5]);
    c.K = (unsigned)p.K;
    c.tau_first = s.tau_s[0];
    c.tau_last = s.tau_s[p.K - 1];
    c.tau_top = __int_as_float(s.meta[6]);
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
    constexpr int GS = (4 * NQ) % 8 == 0 ? 8 : 4;  // samples per group (a chunk is a whole number of groups)
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
// The short form of consume_chunk, for rows all of whose chunks are full (4*NQ samples each).  Nothing in it asks whether a lane
// has a row of its own: such a lane shadows the last row of the tile (same shared-memory data, so the votes need no
// validity term) and is handed the spare histogram copy, which nothing reads, and counters that are dropped.
// ------------------------------------------------------------------------------------------
// The groups of a chunk that hold samples to bin.  CLAMP = false when every lane's running sums of the chunk are
// below the last finite threshold: cell() is monotone, so the cell index then cannot pass that threshold's and needs
// no upper bound (negative and NaN inputs convert to 0 either way).
// `bin` gives the shared-window address of a sample's bin in this thread's histogram copy: the cell arithmetic or
// the table proposes the bin, the threshold itself decides (tau_s[K] = +inf).
// ONE = the proposal is at most one threshold short (no cell of the table holds two finite thresholds; always so for
// the cell arithmetic); otherwise the thresholds are stepped over one by one.
template <int NS, int GS, int RULE, bool BATCH, bool DIRECT, bool CLAMP, bool ONE>
__device__ __forceinline__ void bin_groups(const float (&s)[NS], const BinCtx &c, uint32_t hist_a, unsigned fmax_delta,
                                           unsigned &prev, int &cnt0, float &fin0)
{
    auto bin = [&](float x) -> uint32_t {
        uint32_t off;
        if (DIRECT) {
            unsigned cell = __float2uint_rz(__fmaf_rn(x, c.dscale, c.dshift));
            if (CLAMP) cell = min(cell, c.K);
            off = 4u * cell;
        } else {
            unsigned cell = __float2uint_rz(__fmul_rn(__fsub_rn(x, c.lut_lo), c.lut_scale));
            if (CLAMP) cell = min(cell, c.C);
            off = lds_u16(c.lut_a + 2u * cell);
        }
        if (!ONE) {
            while (off < c.K4 && x >= lds_f32(c.tau_a + off)) off += 4u;  // (tau_s[K] = +inf ends it too)
            return hist_a + off;
        }
        const uint32_t ha = hist_a + off;
        return (x >= lds_f32(c.tau_a + off)) ? ha + 4u : ha;
    };
#pragma unroll
    for (int g = 0; g < NS; g += GS) {
        if (g + GS < NS && __all_sync(0xffffffffu, s[g + GS - 1] < c.tau_first)) {  // (the last group is never low here)
            cnt0 += GS;
            if (RULE == 1) fin0 = fmaxf(fin0, s[g + GS - 1]);
            continue;
        }
        if (RULE == 0) {
            if (BATCH) {
                uint32_t ha[GS];
#pragma unroll
                for (int e = 0; e < GS; ++e) ha[e] = bin(s[g + e]);
#pragma unroll
                for (int e = 0; e < GS; ++e) red_shared_inc(ha[e]);
            } else {
#pragma unroll
                for (int e = 0; e < GS; ++e) red_shared_inc(bin(s[g + e]));
            }
        } else {
            // `prev` is the ADDRESS of the bin of the running time before the next micro-batch (hist_a = bin 0)
            uint32_t ha[GS];
#pragma unroll
            for (int e = 0; e < GS; ++e) ha[e] = bin(s[g + e]);
#pragma unroll
            for (int e = 0; e < GS; ++e) {
                // bin 0 stays in registers (count and largest finish time), every other bin is updated in place; a
                // predicated form without the branch measured 15-20 % slower (its increments are serialised)
                if (prev != hist_a) {
                    red_shared_inc(prev);
                    red_shared_max(prev + fmax_delta, __float_as_int(s[g + e]));
                } else {
                    ++cnt0;
                    fin0 = fmaxf(fin0, s[g + e]);
                }
                prev = ha[e];
            }
        }
    }
}

template <int NQ, int RULE, bool BATCH, bool DIRECT, bool ONE>
__device__ __forceinline__ void consume_full(const float4 (&v)[NQ], int lane, const BinCtx &c, uint32_t hist_a,
                                             unsigned fmax_delta, float &P, unsigned &prev, int &cnt0, float &fin0,
                                             uint64_t *release_bar)
{
    constexpr int NS = 4 * NQ;
    constexpr int GS = (NS % 8 == 0) ? 8 : 4;  // samples per group
    const float before = P;  // running sum before the chunk
    float s[NS];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        P = __fadd_rn(P, v[q].x); s[4 * q + 0] = P;
        P = __fadd_rn(P, v[q].y); s[4 * q + 1] = P;
        P = __fadd_rn(P, v[q].z); s[4 * q + 2] = P;
        P = __fadd_rn(P, v[q].w); s[4 * q + 3] = P;
    }
    // The vote needs every lane's last running sum, i.e. every shared-memory read of the stage by this warp has
    // returned; the count operand of the arrive depends on the vote (arrive_one is 1), so the release cannot move
    // ahead of the reads.
    const bool chunk_low = __all_sync(0xffffffffu, P < c.tau_first);
    if (lane == 0) mbar_arrive_count(release_bar, chunk_low ? 1u : c.arrive_one);
    if (chunk_low) {
        cnt0 += NS;
        if (RULE == 1) fin0 = fmaxf(fin0, P);
        return;
    }
    // Every lane at or above the last threshold before the chunk: under the paper's rule all its samples fall into
    // the bin nobody reads, under the start-before-tau rule none of its micro-batches is started.
    if (__all_sync(0xffffffffu, RULE == 0 ? before >= c.tau_last : prev >= hist_a + c.K4)) return;
    if (__all_sync(0xffffffffu, P < c.tau_top))
        bin_groups<NS, GS, RULE, BATCH, DIRECT, false, ONE>(s, c, hist_a, fmax_delta, prev, cnt0, fin0);
    else
        bin_groups<NS, GS, RULE, BATCH, DIRECT, true, ONE>(s, c, hist_a, fmax_delta, prev, cnt0, fin0);
}

}  // namespace
