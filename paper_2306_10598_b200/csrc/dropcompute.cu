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
#include "dropcompute_dev.h"

#include "sweep_common.cuh"
#include "sweep_tiled.cuh"
#include "sweep_flat.cuh"
#include "sweep_plain.cuh"
#include "sweep_scaled.cuh"
#include "stats_kernels.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static std::mutex lock;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> guard(lock);
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
    static std::mutex lock;
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> guard(lock);
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

// Blocks for `units` equal pieces of work (trials, or tiles of several trials) that the blocks take round-robin: as
// many as fit the GPU at once (`resident`).  mode 2 (DC_TUNE_EVEN_GRID) takes the FEWEST blocks that still finish in
// the same number of rounds instead, so that no block sits out the last round; that pays only where the kernel is
// bound by memory bandwidth alone, and measured 0-8 % slower on the workloads here, whose blocks are bound by their
// own pace: the blocks left over in the last round run faster when they have the GPU to themselves.
long long even_grid(long long units, long long resident, int mode = 0)
{
    if (units <= resident) return units;
    if (mode != 2) return resident;
    const long long rounds = (units + resident - 1) / resident;
    return (units + rounds - 1) / rounds;
}

constexpr int kPackedMinRounds = 3;  // packed tiles of several trials only when every resident block gets about this many

int floor_pow2(int v)
{
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

// Expert settings (dc_tune).  They are process-wide, but every call works from ONE consistent copy taken under
// the lock when it starts, so a dc_tune from another host thread can never tear a launch configuration.
struct Tune {
    int stages = 0;        // 0 = automatic
    int lane_copies = 0;   // 0 = automatic
    int warp_groups = 0;   // 0 = automatic
    int box_floats = 0;    // 0 = automatic
    int batch = 0;         // 0 = automatic, 1 = off, 2 = on
    int direct = 0;        // 0 = automatic (on), 1 = off, 2 = on
    int flat_max_m = 0;    // 0 = automatic (kFlatAutoMaxM), else the longest row the flat kernel is given (<= kFlatMaxM)
    int flat_tile_warps = 0, flat_groups = 0, flat_depth = 0;  // flat kernel; all three or none
    int lean = 0;          // 0 = automatic (on), 1 = off, 2 = on: the short consumer loop for rows of full chunks
    int whole_lines = 0;   // 0 = automatic (on), 1 = off: rows shorter than 128 bytes fetched as whole 128-byte lines
    int l2_promotion = 0;  // 0 = automatic (256 bytes), 1 = none, 2 = 64, 3 = 128, 4 = 256 bytes
    int even_grid = 0;     // 0 = automatic (1), 1 = as many blocks as fit the GPU, 2 = the fewest blocks with as many rounds
    int tile_trials = 0;   // 0 = automatic, else the most trials of few workers that share a tile
};
std::mutex g_tune_lock;
Tune g_tune;
Tune tune_snapshot()
{
    std::lock_guard<std::mutex> guard(g_tune_lock);
    return g_tune;
}

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
bool flat_ok(const float *lat, int64_t M, const Tune &tune)
{
    // any 4-byte aligned base; rows beyond kFlatAutoMaxM measured faster in the plain-load kernel
    return !tiled_ok(lat, M) && M <= (tune.flat_max_m > 0 ? tune.flat_max_m : kFlatAutoMaxM);
}

template <int RULE, bool BATCH, int NQ>
int launch_flat_q(const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di, cudaStream_t stream)
{
    auto kernel = dc_sweep_flat<RULE, BATCH, NQ>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, block, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
    const long long grid = even_grid(T, (long long)occ * di.sms);
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

template <int NQ, int RULE, bool BATCH, bool WIDE, bool LEAN>
int launch_tiled_k(const CUtensorMap &map, const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di,
                   cudaStream_t stream)
{
    auto kernel = dc_sweep_tiled<NQ, RULE, BATCH, WIDE, LEAN>;
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
    const long long grid = even_grid(T, (long long)occ * di.sms, p.grid_mode);
    kernel<<<(unsigned)grid, block, smem, stream>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

// Rows of full chunks get the kernel with the short consumer loop, the others the kernel with the general one; tiles of
// two whole trials (WIDE) only exist for rows of one full chunk.
template <int NQ, int RULE, bool BATCH, bool WIDE = false>
int launch_tiled_b(const CUtensorMap &map, const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di,
                   cudaStream_t stream)
{
    if (p.lean) return launch_tiled_k<NQ, RULE, BATCH, WIDE, true>(map, p, block, smem, T, di, stream);
    if constexpr (WIDE) return DC_ERR_RANGE;
    else return launch_tiled_k<NQ, RULE, BATCH, false, false>(map, p, block, smem, T, di, stream);
}

template <int NQ, int RULE>
int launch_tiled(const CUtensorMap &map, const SweepParams &p, int block, size_t smem, long long T, const DeviceInfo &di,
                 cudaStream_t stream)
{
    // rule 1 has one binning path only; tiles of two whole trials are compiled for chunks of 12 and 16 floats
    if constexpr (NQ == 3 || NQ == 4) {
        if (block > kMaxRowsPerPass + 64) {
            if constexpr (RULE == 0) {
                if (p.batch_lookups) return launch_tiled_b<NQ, RULE, true, true>(map, p, block, smem, T, di, stream);
            }
            return launch_tiled_b<NQ, RULE, false, true>(map, p, block, smem, T, di, stream);
        }
    }
    if (block > kMaxRowsPerPass + 64) return DC_ERR_RANGE;
    if constexpr (RULE == 0) {
        if (p.batch_lookups) return launch_tiled_b<NQ, RULE, true>(map, p, block, smem, T, di, stream);
    }
    return launch_tiled_b<NQ, RULE, false>(map, p, block, smem, T, di, stream);
}

// Shared-memory layout of a block of the staged kernels (tiled and flat): ring depth, histogram copies, table
// size.  Needs p.stage_bytes, p.chunks and the row-thread count; fills the rest and the dynamic shared bytes.
int choose_block_layout(SweepParams &p, int row_threads, int K, int rule, const DeviceInfo &di, const Tune &tune,
                        size_t *smem_out, int stage_cap = 3)
{
    p.lut_cells = min(kLutCellsMax, 4 * K);
    // Rows that fit one tile gain from looking up a whole group's bins before touching the histogram (the
    // chains overlap); longer rows measured faster with lookups and updates interleaved.
    p.batch_lookups = tune.batch > 0 ? tune.batch - 1 : ((p.chunks == 1 || p.short_launch) ? 1 : 0);
    // Arithmetic binning of evenly spaced thresholds measured faster wherever a group's bins are computed before
    // its updates (rows of one tile, and the start-before-tau rule), slower for long rows under the paper's rule.
    p.direct_bins = tune.direct > 0 ? tune.direct - 1
                                      : ((rule == DC_RULE_START_BEFORE_TAU || p.chunks == 1 || p.short_launch) ? 1 : 0);
    // Shared memory per block: aim at two resident blocks per SM.  Histogram copies: lane l of warp w
    // adds into copy (w % warp_groups) * lane_copies + (l % lane_copies); copies used by one warp start
    // 32 / lane_copies banks apart so that equal bins of different lanes do not collide.
    // Tiles of several small trials whose outputs take the epilogue warp four steps or more are finished by the
    // consumer warps themselves, all of them at once (one buffer); otherwise the epilogue warp works on one buffer
    // while the consumers fill the other.  Measured with 64 thresholds: trials of 8 workers 3-4 times faster that
    // way, of 32 workers 1.3-1.5 times, of 64 and 100 workers 15-35 % slower.
    {
        const bool sub = p.g > 1 && K % 4 == 0 && K <= 128 && ((K / 4) & (K / 4 - 1)) == 0;
        const int per_step = sub ? 32 / (K / 4) : 1;
        p.nbuf = (p.g > 1 && (p.g + per_step - 1) / per_step >= 4) ? 1 : 2;
    }
    p.spare = 1;
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
                                    : (tune.stages > 0 ? tune.stages : min(stage_cap, max(2, kStageBudgetBytes / p.stage_bytes)));
    const int s_min = stage_cap < 0 ? -stage_cap : (tune.stages > 0 ? tune.stages : 2);
    // Several small trials per tile: the fewer workers a trial has, the more trials a warp's lanes are spread over
    // and the fewer histogram copies per trial are worth their shared memory.
    const int lc_auto = p.g > 1 ? (p.N >= 32 ? 4 : (p.N >= 16 ? 2 : 1)) : 4;
    const int lc_first = tune.lane_copies > 0 ? tune.lane_copies : lc_auto;
    const int lc_last = tune.lane_copies > 0 ? tune.lane_copies : 1;
    const int wg_first = tune.warp_groups > 0 ? min(tune.warp_groups, ncw) : (p.g > 1 ? 1 : min(2, ncw));
    const int wg_last = tune.warp_groups > 0 ? wg_first : 1;
    const bool forced = tune.stages > 0 && tune.lane_copies > 0 && tune.warp_groups > 0;
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
                       tail_bytes(K, hist_slots(p), p.hist_stride, p.lut_cells, fmax_slots(p), p.nbuf * p.g);
                p.epi_vec = (K % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.out_step) & 15) == 0) &&
                            ((reinterpret_cast<uintptr_t>(p.out_done) & 15) == 0);
                // Several small trials per tile: when K/4 is a power of two up to 32 the epilogue warp takes 32/(K/4)
                // trials at once.
                p.epi_sub = 0;
                if (p.g > 1 && p.epi_vec && K <= 128 && ((K / 4) & (K / 4 - 1)) == 0) p.epi_sub = K / 4;
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
    const Tune tune = tune_snapshot();

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
    p.g = 1;
    p.batch_lookups = 0;
    p.rule = rule;
    p.aux_copies = rule == DC_RULE_START_BEFORE_TAU ? p.hist_copies : 0;
    p.grid_mode = tune.even_grid;

    if (tiled_ok(lat, M)) {
        EncodeTiledFn encode = get_encode_fn();
        if (!encode) return DC_ERR_CUDA;
        // Chunk length (floats of a row per box).  Rows all of whose chunks are full take the short consumer loop,
        // so a row length that 32 does not divide is cut into equal chunks of 12, 16 or 24 floats when that works.
        p.bw = (int)(M < 32 ? M : 32);
        if (M > 32 && M % 32 != 0) {
            for (int cand : {24, 16, 12}) {
                if (M % cand == 0) {
                    p.bw = cand;
                    break;
                }
            }
        }
        // Launches of well under a second's worth of bandwidth (below 1 GiB of latencies) are shaped by their start
        // and their tail: 16-float tiles need fewer registers and less shared memory, so three blocks fit an SM,
        // more loads are in flight from the first microsecond and the last wave is finer.  Measured 5-25 % faster
        // on 0.4 GB inputs of 32- to 128-sample rows, 3-5 % slower on inputs of 2 GB and more.
        p.short_launch = (tune.box_floats == 0 && M >= 32 && M % 16 == 0 &&
                          (uint64_t)T * (uint64_t)N * (uint64_t)M * 4ull < (1ull << 30)) ? 1 : 0;
        if ((tune.box_floats == 16 && M % 16 == 0) || p.short_launch) p.bw = 16;
        if (tune.box_floats == 32) p.bw = (int)(M < 32 ? M : 32);
        p.chunks = (int)((M + p.bw - 1) / p.bw);
        const int last_cols = (int)(M - (int64_t)(p.chunks - 1) * p.bw);
        p.nq_last = last_cols / 4;
        p.pitch = p.bw * 4;
        const int nq = p.bw / 4;
        // the kernel is compiled for 1, 2, 3, 4, 6 and 8 quads per chunk; other chunk lengths run in the next size up
        // (each further size costs a quarter more build time and measured 3 % on the rows it would serve)
        const int nq_inst = nq <= 4 ? nq : (nq <= 6 ? 6 : 8);
        p.lean = (tune.lean != 1 && last_cols == p.bw && nq == nq_inst) ? 1 : 0;
        // Several whole trials of few workers share a tile: g trials of N rows each, g N <= 256, as many as it takes
        // to give every resident block about one tile, within what the histograms of g trials may take.
        if (N <= kMaxRowsPerPass / 2) {
            int64_t gmax = kMaxRowsPerPass / N;
            const int64_t hist_cap = (int64_t)kHistBudgetBytes / (2 * 4 * (int64_t)(K + 8));
            if (gmax > hist_cap) gmax = hist_cap;
            if (tune.tile_trials > 0 && gmax > tune.tile_trials) gmax = tune.tile_trials;
            int64_t g = (T + 2 * (int64_t)di.sms - 1) / (2 * (int64_t)di.sms);
            if (g > gmax) g = gmax;
            if (g < 1) g = 1;
            if (g > 1) {
                p.g = (int)g;
                p.passes = 1;
                p.rows = (int)(g * N);
            }
        }
        // Trials that do not fill whole warps leave lanes idle in the last warp of every pass (200 workers: 24 of 224;
        // two trials of 100 workers likewise).  Packed tiles: G trials are one run of G N consecutive rows of the
        // [T N][M] view, cut into P >= 2 equal passes of at most 256 rows (200 workers: 5 trials = 1000 rows = 4 passes
        // of 250 rows on 256 lanes, 2.3 % idle instead of 10.7 %); a trial then starts in the middle of a pass.  Taken
        // when it leaves clearly fewer lanes idle and there are enough tiles for a few rounds.  Measured on 100 and 200
        // workers, 8192 and more trials: start-before-tau rule 12-20 % faster (its heavier per-trial epilogue also
        // takes two trials per step instead of one); the paper's rule 4-17 % faster on rows of 12 samples, 10 % on rows
        // of 100 (general loop), level to 4 % slower on rows of 32 and 64, which therefore stay as they were.
        bool packed = false;
        if (N < kMaxRowsPerPass && tune.tile_trials != 1 && (uint64_t)T * (uint64_t)N < (1ull << 31) - 4096) {
            const int64_t hist_cap = (int64_t)kHistBudgetBytes / (2 * 4 * 4 * (int64_t)(K + 8));  // two buffers, four copies
            int64_t gmax = min((int64_t)8, hist_cap);
            // (the epilogue warp must keep up: with K/4 lanes per trial it takes several trials per step; otherwise at
            // most three trials per tile, as choose_block_layout hands longer tiles to the consumer warps)
            if (!(K % 4 == 0 && K <= 128 && ((K / 4) & (K / 4 - 1)) == 0)) gmax = min(gmax, (int64_t)3);
            if (tune.tile_trials > 1 && gmax > tune.tile_trials) gmax = tune.tile_trials;
            const double idle1 = 1.0 - (double)p.rows / (double)(((p.rows + 31) / 32) * 32);  // as chosen so far
            double best_idle = idle1;
            int best_g = 1, best_p = 1, best_rows = 0;
            for (int64_t G = p.g + 1; G <= gmax; ++G) {
                const int64_t P = (G * N + kMaxRowsPerPass - 1) / kMaxRowsPerPass;
                if (P < 2) continue;
                const int64_t rows = (G * N + P - 1) / P;
                const double idle = 1.0 - (double)(G * N) / (double)(((rows + 31) / 32) * 32 * P);
                if (idle < best_idle - 0.005) {
                    best_idle = idle;
                    best_g = (int)G;
                    best_p = (int)P;
                    best_rows = (int)rows;
                }
            }
            // (under the paper's rule, rows of 32 samples and more in the short loop measured level to 4 % slower packed)
            const bool pays = rule == DC_RULE_START_BEFORE_TAU || M <= 16 || !p.lean;
            const bool enough = tune.tile_trials > 1 || (pays && T / best_g >= (int64_t)kPackedMinRounds * 3 * di.sms);
            if (best_g > 1 && idle1 - best_idle >= 0.04 && enough) {
                packed = true;
                p.g = best_g;
                p.passes = best_p;
                p.rows = best_rows;
            }
        }
        if (!packed && p.g == 1 && N > kMaxRowsPerPass / 2 && N < kMaxRowsPerPass && (nq_inst == 3 || nq_inst == 4) && p.chunks == 1 && p.lean && tune.tile_trials != 1 &&
                   T >= 8 * (int64_t)di.sms && K <= 512) {
            // Two whole trials per tile when that leaves clearly fewer idle lanes than one (200 workers: 24 of 224
            // lanes idle alone, 16 of 416 as a pair).  Rows of one chunk only: measured 3-6 % faster there (200
            // workers, 12 and 16 samples), level or slower on rows of two chunks.
            const double idle1 = 1.0 - (double)N / (double)(((N + 31) / 32) * 32);
            const double idle2 = 1.0 - (double)(2 * N) / (double)(((2 * N + 31) / 32) * 32);
            if (idle1 - idle2 >= 0.04) {
                p.g = 2;
                p.passes = 1;
                p.rows = (int)(2 * N);
            }
        }
        const int row_threads_t = ((p.rows + 31) / 32) * 32;
        CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_NONE;
        p.swz_mask = 0;
        if (p.pitch == 128) { swz = CU_TENSOR_MAP_SWIZZLE_128B; p.swz_mask = 7; }
        else if (p.pitch == 64) { swz = CU_TENSOR_MAP_SWIZZLE_64B; p.swz_mask = 3; }
        else if (p.pitch == 32) { swz = CU_TENSOR_MAP_SWIZZLE_32B; p.swz_mask = 1; }
        p.box_y = p.rows;
        // Rows shorter than a 128-byte line: consecutive rows are contiguous in memory, so when every pass of every
        // trial starts and ends on a line the tensor is described to the copy unit as lines of 32 floats and a tile
        // is so many whole lines (a quarter to an eighth of the requests of row-sized pieces).  The tile in shared
        // memory is the same dense copy of its rows; of "no swizzle" and the 128-byte swizzle the one with fewer
        // bank conflicts for "lane r reads 16 bytes of row r" is taken.
        const bool whole_lines = !packed && tune.whole_lines != 1 && M < 32 && (N * M) % 32 == 0 && ((int64_t)p.rows * M) % 32 == 0 &&
                                 (p.g > 1 || N % p.rows == 0);
        if (whole_lines) {
            int worst[2] = {0, 0};
            for (int mode = 0; mode < 2; ++mode) {
                for (int q = 0; q < nq; ++q) {
                    for (int r0 = 0; r0 < 32 && r0 < p.rows; r0 += 8) {
                        int hits[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                        for (int r = r0; r < r0 + 8 && r < p.rows; ++r) {
                            unsigned chunk = (unsigned)(r * (int)M / 4 + q);
                            if (mode == 1) chunk ^= (chunk >> 3) & 7u;
                            const int hcount = ++hits[chunk & 7u];
                            if (hcount > worst[mode]) worst[mode] = hcount;
                        }
                    }
                }
            }
            const bool use_swizzle = worst[1] < worst[0];
            swz = use_swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
            p.swz_mask = use_swizzle ? 7 : 0;
            p.box_y = (int)((int64_t)p.rows * M / 32);
        }
        p.stage_bytes = ((p.rows * p.pitch + 1023) / 1024) * 1024;
        size_t smem = 0;
        {
            const int lrc0 = choose_block_layout(p, row_threads_t, K, rule, di, tune, &smem);
            if (lrc0 != DC_OK) return lrc0;
        }

        CUtensorMap map;
        cuuint64_t gdim[3] = {(cuuint64_t)M, (cuuint64_t)N, (cuuint64_t)T};
        cuuint64_t gstride[2] = {(cuuint64_t)M * 4, (cuuint64_t)N * (cuuint64_t)M * 4};
        cuuint32_t box[3] = {(cuuint32_t)p.bw, (cuuint32_t)(p.g > 1 ? N : p.rows), (cuuint32_t)p.g};
        if (whole_lines) {  // [T][N*M/32 lines][32 floats]
            gdim[0] = 32;
            gdim[1] = (cuuint64_t)(N * M / 32);
            gstride[0] = 128;
            box[0] = 32;
            box[1] = (cuuint32_t)((p.g > 1 ? N : (int64_t)p.rows) * M / 32);
        }
        p.tile_y = 0;
        p.tile_z = p.g;
        if (packed) {  // [1][T N rows][M floats]: a tile's rows are consecutive whatever trial they belong to
            gdim[1] = (cuuint64_t)T * (cuuint64_t)N;
            gdim[2] = 1;
            gstride[1] = (cuuint64_t)T * (cuuint64_t)N * (cuuint64_t)M * 4;
            box[1] = (cuuint32_t)p.rows;
            box[2] = 1;
            p.tile_y = (int)(p.g * N);
            p.tile_z = 0;
        }
        const cuuint32_t estr[3] = {1, 1, 1};
        if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(lat), gdim, gstride, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   tune.l2_promotion == 1 ? CU_TENSOR_MAP_L2_PROMOTION_NONE
                   : tune.l2_promotion == 2 ? CU_TENSOR_MAP_L2_PROMOTION_L2_64B
                   : tune.l2_promotion == 3 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DC_ERR_CUDA;

        if (smem > (size_t)di.max_smem_optin) return DC_ERR_RANGE;
        const int block = row_threads_t + 64;
        const long long tiles = (T + p.g - 1) / p.g;
        int lrc;
        if (rule == DC_RULE_FINISH_BEFORE_TAU) {
            switch (nq_inst) {
            case 1: lrc = launch_tiled<1, 0>(map, p, block, smem, tiles, di, stream); break;
            case 2: lrc = launch_tiled<2, 0>(map, p, block, smem, tiles, di, stream); break;
            case 3: lrc = launch_tiled<3, 0>(map, p, block, smem, tiles, di, stream); break;
            case 4: lrc = launch_tiled<4, 0>(map, p, block, smem, tiles, di, stream); break;
            case 6: lrc = launch_tiled<6, 0>(map, p, block, smem, tiles, di, stream); break;
            default: lrc = launch_tiled<8, 0>(map, p, block, smem, tiles, di, stream); break;
            }
        } else {
            switch (nq_inst) {
            case 1: lrc = launch_tiled<1, 1>(map, p, block, smem, tiles, di, stream); break;
            case 2: lrc = launch_tiled<2, 1>(map, p, block, smem, tiles, di, stream); break;
            case 3: lrc = launch_tiled<3, 1>(map, p, block, smem, tiles, di, stream); break;
            case 4: lrc = launch_tiled<4, 1>(map, p, block, smem, tiles, di, stream); break;
            case 6: lrc = launch_tiled<6, 1>(map, p, block, smem, tiles, di, stream); break;
            default: lrc = launch_tiled<8, 1>(map, p, block, smem, tiles, di, stream); break;
            }
        }
        return lrc;
    }

    if (flat_ok(lat, M, tune)) {
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
        if (tune.flat_tile_warps > 0 && tune.flat_groups > 0 && tune.flat_depth > 0) {
            best_wt = tune.flat_tile_warps;
            if ((int64_t)best_wt * 32 > N) best_wt = (int)((N + 31) / 32);
            best_g = tune.flat_groups;
            best_d = tune.flat_depth;
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
        const bool forced_split = tune.flat_tile_warps > 0 && tune.flat_groups > 0 && tune.flat_depth > 0;
        int groups = min(best_g, p.passes), depth = best_d;
        if (!forced_split && groups == 1) depth = 3;
        size_t smem = 0;
        int flat_threads = 0;
        for (;;) {
            p.flat_groups = groups;
            flat_threads = groups * wt * 32;
            const int lrc0 = choose_block_layout(p, flat_threads, K, rule, di, tune, &smem, -(groups * depth));
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
                        tail_bytes(K, hist_slots(p), p.hist_stride, p.lut_cells, fmax_slots(p), p.nbuf * p.g);
    if (smem > (size_t)di.max_smem_optin) return DC_ERR_RANGE;
    auto kernel = rule == DC_RULE_FINISH_BEFORE_TAU ? dc_sweep_plain<0> : dc_sweep_plain<1>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, p.rows, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
    const long long grid = even_grid(T, (long long)occ * di.sms);
    kernel<<<(unsigned)grid, p.rows, smem, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return DC_ERR_CUDA;
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

int dc_simulate_scaled(const float *latencies, int64_t T, int64_t N, int64_t M, const float *taus, int32_t K,
                       const float *worker_scale, float t_comm, float *out_step, int32_t *out_done, float *out_sync, int32_t rule,
                       void *stream_v)
{
    if (!worker_scale) return DC_ERR_NULL;
    const int rc = validate_simulate(latencies, T, N, M, taus, K, out_step, out_done, rule);
    if (rc != DC_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(worker_scale) & 3) || (out_sync && (reinterpret_cast<uintptr_t>(out_sync) & 3))) return DC_ERR_ALIGN;
    DeviceInfo di;
    if (!device_info(&di)) return DC_ERR_CUDA;
    const size_t smem = scaled_smem_bytes(K);
    if (smem > (size_t)di.max_smem_optin) return DC_ERR_RANGE;
    auto kernel = rule == DC_RULE_FINISH_BEFORE_TAU ? dc_sweep_scaled<0> : dc_sweep_scaled<1>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DC_ERR_CUDA;
    // a block is one thread per worker, in whole warps, up to kScaledThreads (more workers: several rows per thread)
    const int block = (int)min((int64_t)kScaledThreads, ((N + 31) / 32) * 32);
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, block, smem) != cudaSuccess || occ < 1) return DC_ERR_CUDA;
    const long long grid = even_grid(T, (long long)occ * di.sms);
    kernel<<<(unsigned)grid, block, smem, static_cast<cudaStream_t>(stream_v)>>>(latencies, taus, worker_scale, T, (int)N, (int)M, K,
                                                                                      t_comm, out_step, out_done, out_sync);
    return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
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
    return DC_OK;
}

int dc_simulate_plan(const float *latencies, int64_t T, int64_t N, int64_t M, int32_t K)
{
    if (!latencies) return -DC_ERR_NULL;
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return -DC_ERR_SHAPE;
    if (K > DC_MAX_K || N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX || T > (int64_t)INT32_MAX)
        return -DC_ERR_RANGE;
    if (reinterpret_cast<uintptr_t>(latencies) & 3) return -DC_ERR_ALIGN;
    return tiled_ok(latencies, M) ? 0 : (flat_ok(latencies, M, tune_snapshot()) ? 2 : 1);
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
    if (K > DC_MAX_K || N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX) return DC_ERR_RANGE;
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
    return DC_OK;
}

int dc_reduce_trials_static(const float *out_step, const int32_t *out_done, const float *out_sync, int64_t T, int32_t K,
                            int64_t N, int64_t M, double *stats, double *baseline, void *stream_v)
{
    if (!out_step || !out_done || !stats || !baseline) return DC_ERR_NULL;
    if (T <= 0 || K <= 0 || N <= 0 || M <= 0) return DC_ERR_SHAPE;
    if (K > DC_STATIC_MAX_K || N > INT32_MAX || M > INT32_MAX || N * M > (int64_t)INT32_MAX) return DC_ERR_RANGE;
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
    dc_check_kernel<<<grid, 256, 0, stream>>>(latencies, total, (unsigned long long)T * (unsigned long long)N, (int)M, taus, K,
                                              reinterpret_cast<unsigned long long *>(counters));
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
    // The private copy stream starts after everything the caller has enqueued on `stream` so far (which may
    // still be using the workspace).
    cudaEvent_t entered = nullptr;
    DC_TRY(cudaEventCreateWithFlags(&entered, cudaEventDisableTiming));
    DC_TRY(cudaEventRecord(entered, stream));
    DC_TRY(cudaStreamWaitEvent(copy_stream, entered, 0));
    DC_TRY(cudaMemcpyAsync(d_taus, taus_host, (size_t)K * 4, cudaMemcpyHostToDevice, stream));
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
    if (entered) cudaEventDestroy(entered);
    if (copy_stream) cudaStreamDestroy(copy_stream);
    if (cuda_fail) return DC_ERR_CUDA;
    return rc;
}

int dc_tune(int32_t key, int32_t value)
{
    std::lock_guard<std::mutex> guard(g_tune_lock);
    Tune &tune = g_tune;
    if (key == DC_TUNE_STAGES && (value == 0 || (value >= 2 && value <= kMaxStages))) {
        tune.stages = value;
        return DC_OK;
    }
    if (key == DC_TUNE_LANE_COPIES && (value == 0 || value == 1 || value == 2 || value == 4 || value == 8)) {
        tune.lane_copies = value;
        return DC_OK;
    }
    if (key == DC_TUNE_WARP_GROUPS && value >= 0 && value <= 8) {
        tune.warp_groups = value;
        return DC_OK;
    }
    if (key == DC_TUNE_BATCH_LOOKUPS && value >= 0 && value <= 2) {
        tune.batch = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_MAX_M && value >= 0 && value <= kFlatMaxM) {
        tune.flat_max_m = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_TILE_WARPS && value >= 0 && value <= 8) {
        tune.flat_tile_warps = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_GROUPS && value >= 0 && value <= 8) {
        tune.flat_groups = value;
        return DC_OK;
    }
    if (key == DC_TUNE_FLAT_DEPTH && value >= 0 && value <= 4) {
        tune.flat_depth = value;
        return DC_OK;
    }
    if (key == DC_TUNE_DIRECT_BINS && value >= 0 && value <= 2) {
        tune.direct = value;
        return DC_OK;
    }
    if (key == DC_TUNE_BOX_FLOATS && (value == 0 || value == 16 || value == 32)) {
        tune.box_floats = value;
        return DC_OK;
    }
    if (key == DC_TUNE_LEAN_LOOP && value >= 0 && value <= 2) {
        tune.lean = value;
        return DC_OK;
    }
    if (key == DC_TUNE_L2_PROMOTION && value >= 0 && value <= 4) {
        tune.l2_promotion = value;
        return DC_OK;
    }
    if (key == DC_TUNE_EVEN_GRID && value >= 0 && value <= 2) {
        tune.even_grid = value;
        return DC_OK;
    }
    if (key == DC_TUNE_WHOLE_LINES && value >= 0 && value <= 2) {
        tune.whole_lines = value;
        return DC_OK;
    }
    if (key == DC_TUNE_TILE_TRIALS && value >= 0 && value <= kMaxRowsPerPass) {
        tune.tile_trials = value;
        return DC_OK;
    }
    return DC_ERR_UNSUPPORTED;
}

int dc_launch_count(int32_t entry_point, int64_t T, int64_t N, int64_t M, int32_t K, int64_t chunk_trials)
{
    if (T <= 0 || N <= 0 || M <= 0 || K <= 0) return -DC_ERR_SHAPE;
    switch (entry_point) {
    case DC_ENTRY_SIMULATE: return 1;  // (dc_simulate_scaled too)
    case DC_ENTRY_SIMULATE_SPLIT: {
        DeviceInfo di;
        if (!device_info(&di)) return -DC_ERR_CUDA;
        return split_groups(T, N, di.sms) > 1 ? 2 : 1;
    }
    case DC_ENTRY_REDUCE_TRIALS: return 2;
    case DC_ENTRY_ARGMAX_TAU: return 1;
    case DC_ENTRY_SWEEP_DEVICE: return 4;
    case DC_ENTRY_SWEEP_HOST: {
        if (chunk_trials <= 0) return -DC_ERR_SHAPE;
        if (chunk_trials > T) chunk_trials = T;
        const int64_t nchunks = (T + chunk_trials - 1) / chunk_trials;
        return nchunks + 3 > (int64_t)INT32_MAX ? -DC_ERR_RANGE : (int)(nchunks + 3);
    }
    default: return -DC_ERR_UNSUPPORTED;
    }
}

#ifndef DC_SOURCE_HASH
#define DC_SOURCE_HASH "unhashed"
#endif
const char *dc_kernel_version(void) { return "sweep-" DC_SOURCE_HASH; }

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
