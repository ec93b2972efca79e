/*
 * dropcompute_dev.h -- measurement and tuning aids of the DropCompute threshold-sweep library.
 *
 * Nothing in this header is part of the method (the paper has no counterpart to any of it) and a user of
 * Algorithm 2 never needs it: benchmarks, profiles and tests use these entry points to pick launch
 * configurations by hand, to time a plain read of the same bytes, to count launches and to tell library
 * builds apart.  The product interface is dropcompute.h.
 */
#ifndef DROPCOMPUTE_DEV_H_
#define DROPCOMPUTE_DEV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Which kernel dc_simulate_ex would use for a shape: 0 = tiled kernel (M a multiple of 4 and a 16-byte aligned
 * pointer), 2 = flat kernel (any other case with M <= 127, or up to DC_TUNE_FLAT_MAX_M: other row lengths, or a
 * pointer that is only 4-byte aligned), 1 = plain-load kernel (such cases with longer rows), negative = -dc_status. */
int dc_simulate_plan(const float *latencies, int64_t T, int64_t N, int64_t M, int32_t K);

/*
 * dc_tune -- expert knob for performance experiments; process-wide: it affects dc_simulate* calls of any host
 * thread that START after it returns (a call already running keeps the settings it started with).
 * Results never depend on it.  value 0 restores the automatic choice.
 *   DC_TUNE_STAGES       depth of the shared-memory ring the tiled kernel streams rows through (2..8)
 *   DC_TUNE_LANE_COPIES  histogram copies a warp spreads its lanes over in the tiled kernel (1, 2, 4 or 8)
 *   DC_TUNE_WARP_GROUPS  groups of warps with histogram copies of their own (1..8)
 *   DC_TUNE_BATCH_LOOKUPS 1 = bin each running sum and update the histogram at once, 2 = look up the bins of a
 *                        whole group of eight first (lower latency, better for trials that fit one tile)
 *   DC_TUNE_BOX_FLOATS   floats of a row fetched per tile (16 or 32; 16 needs M to be a multiple of 16)
 *   DC_TUNE_DIRECT_BINS  1 = always bin through the lookup table, 2 = bin evenly spaced thresholds arithmetically
 *                        (one multiply-add and one comparison per sample, no table read) in the tiled kernel
 *   DC_TUNE_FLAT_MAX_M   longest row (1..255) the flat kernel is given instead of the plain-load kernel (default 127)
 *   DC_TUNE_FLAT_TILE_WARPS, DC_TUNE_FLAT_GROUPS, DC_TUNE_FLAT_DEPTH  flat kernel (row length not a multiple
 *                        of 4): warps per tile (tile = 32 x that many rows), groups of warps working on different
 *                        tiles at once, ring stages per group; used only when all three are set, and a setting
 *                        whose tiles or ring do not fit makes dc_simulate* return DC_ERR_RANGE
 *   DC_TUNE_LEAN_LOOP    1 = always the general consumer loop, 2 (and 0) = the short loop wherever every chunk of a
 *                        row is full (tiled kernel)
 *   DC_TUNE_TILE_TRIALS  the most trials of few workers (N <= 128) that may share one tile of the tiled kernel
 *                        (1 = one trial per tile)
 *   DC_TUNE_WHOLE_LINES  1 = rows shorter than 128 bytes are always fetched row by row, 2 (and 0) = as whole
 *                        128-byte lines wherever the passes of every trial start and end on a line (tiled kernel)
 *   DC_TUNE_EVEN_GRID    1 (and 0) = as many blocks as the GPU holds at once, 2 = the fewest blocks that need no more
 *                        rounds over the trials than that (tiled kernel)
 *   DC_TUNE_L2_PROMOTION granularity at which the copy unit's reads are promoted in L2: 1 = none, 2 = 64, 3 = 128,
 *                        4 (and 0) = 256 bytes (tiled kernel)
 * Returns DC_ERR_UNSUPPORTED for an unknown key or value.
 */
#define DC_TUNE_STAGES 1
#define DC_TUNE_LANE_COPIES 2
#define DC_TUNE_WARP_GROUPS 3
#define DC_TUNE_BOX_FLOATS 4
#define DC_TUNE_BATCH_LOOKUPS 5
#define DC_TUNE_DIRECT_BINS 6
#define DC_TUNE_FLAT_TILE_WARPS 7
#define DC_TUNE_FLAT_GROUPS 8
#define DC_TUNE_FLAT_DEPTH 9
#define DC_TUNE_FLAT_MAX_M 11
#define DC_TUNE_LEAN_LOOP 12
#define DC_TUNE_TILE_TRIALS 13
#define DC_TUNE_WHOLE_LINES 14
#define DC_TUNE_EVEN_GRID 15
#define DC_TUNE_L2_PROMOTION 16
int dc_tune(int32_t key, int32_t value);

/*
 * dc_launch_count -- how many kernels one successful call of an entry point enqueues for a shape (a pure
 * function of its arguments and the current device's SM count; nothing is launched, nothing remembered).
 *   entry_point   DC_ENTRY_*      chunk_trials   only for DC_ENTRY_SWEEP_HOST (trials per host-to-device copy)
 * Returns the count, or -dc_status.
 */
#define DC_ENTRY_SIMULATE 0       /* dc_simulate, dc_simulate_ex, dc_simulate_tc */
#define DC_ENTRY_SIMULATE_SPLIT 1
#define DC_ENTRY_REDUCE_TRIALS 2  /* dc_reduce_trials, dc_reduce_trials_static */
#define DC_ENTRY_ARGMAX_TAU 3
#define DC_ENTRY_SWEEP_DEVICE 4
#define DC_ENTRY_SWEEP_HOST 5
int dc_launch_count(int32_t entry_point, int64_t T, int64_t N, int64_t M, int32_t K, int64_t chunk_trials);

/*
 * dc_read_probe -- enqueues a kernel that reads
 * data[0 .. count - count % 4) once with 16-byte loads and does nothing else.  Timed on a latency tensor it gives
 * the duration of a plain read-only pass over those bytes, which benchmarks report beside the sweep's.
 *   data   DEVICE, 16-byte aligned, count floats (all >= 0, as latencies are)
 *   sink   DEVICE, one float; never written for such data
 */
int dc_read_probe(const float *data, int64_t count, float *sink, void *stream);

/* "sweep-" followed by a hash of the CUDA sources the library was built from: changes whenever a kernel
 * changes, so a profile filed under one tag is never mistaken for a measurement of another build. */
const char *dc_kernel_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DROPCOMPUTE_DEV_H_ */
