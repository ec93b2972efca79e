// The plain-load sweep kernel: warp-staged 32 x 32 pieces by ordinary loads.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Plain-load kernel for what neither staged kernel takes (rows longer than kFlatAutoMaxM whose length is not a
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
            // lane = column: row rr's piece of a chunk is one coalesced read of up to 128 bytes.  The next chunk's
            // pieces are requested before the current chunk is walked, so the loads overlap the walk.
            float nx[32];
            auto fetch = [&](int m0) {
                const int ns = min(32, M - m0);
#pragma unroll
                for (int rr = 0; rr < 32; ++rr) {
                    nx[rr] = 0.0f;
                    if (rr < nrows && lane < ns) nx[rr] = __ldg(src + (size_t)rr * M + m0 + lane);
                }
            };
            fetch(0);
            for (int m0 = 0; m0 < M; m0 += 32) {
                const int ns = min(32, M - m0);
#pragma unroll
                for (int rr = 0; rr < 32; ++rr) tile[rr * 33 + lane] = nx[rr];
                __syncwarp();
                float4 v[8];  // lane = row
#pragma unroll
                for (int e = 0; e < 32; ++e) sample_ref(v, e) = tile[lane * 33 + e];
                __syncwarp();
                if (m0 + 32 < M) fetch(m0 + 32);
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

}  // namespace
