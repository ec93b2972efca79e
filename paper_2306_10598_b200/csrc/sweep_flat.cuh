// The flat sweep kernel: whole rows by plain bulk copies.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Flat kernel: rows whose length is not a multiple of 4 (so a tensor map cannot describe them), up to
// kFlatAutoMaxM samples (kFlatMaxM on request), and any row length up to that when the base pointer is only 4-byte
// aligned.  Consecutive rows of a trial are one contiguous span of the
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
        {   // largest row total of the trial (non-negative floats order like their bit patterns)
            const unsigned wm = __reduce_max_sync(0xffffffffu, (unsigned)__float_as_int(rowmax));
            if (lane == 0) atomicMax(&s.segmax[b], (int)wm);
        }
        buffer_barrier_arrive<kBarReady>(b, bar_threads);
    }
}

}  // namespace
