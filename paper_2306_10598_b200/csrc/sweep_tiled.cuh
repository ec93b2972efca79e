// The tiled sweep kernel (TMA tensor map) and the epilogue warp it shares with the flat kernel.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Tiled kernel: TMA-staged rows, persistent over tiles.  A tile is one trial taken in passes of up to 256 rows, or g
// whole trials: of few workers each in one pass (g N <= 256 rows; two trials of up to 256 rows in the WIDE
// instantiations), or as one run of g N consecutive rows cut into equal passes, where a trial may start in the middle
// of a pass (the row -> trial map is then worked out per pass).
// Warp roles inside a block:
//   warps 0 .. ncw-1   consumers: thread r owns row r of the current tile
//   warp  ncw          producer: one thread streams the block's tiles through the ring of stages
//   warp  ncw+1        epilogue: turns a finished tile's histograms into out_done / out_step / out_sync
// The histograms (and the maxima) are double-buffered: consumers fill buffer j&1 for their j-th tile and go
// straight on to the next one while the epilogue warp sums, scans, writes and clears the buffer.  Named barriers
// hand the buffers over: kBarReady+b (consumers arrive, epilogue waits) and kBarFree+b (epilogue arrives,
// consumers wait before reusing the buffer two tiles later).  Tiles of many small trials are finished by the
// consumer warps themselves instead (one buffer, the epilogue warp returns at once).
// NQ = 16-byte quads of a row per chunk held in registers (box width = 4*NQ floats at most).
// A consumer thread adds its row's samples in order; per group of samples, if every lane of the warp is still
// below the first threshold the samples are bin 0 (one register add); if every lane is at or above the last
// threshold they are in the bin nobody reads; otherwise each running sum is binned through the lookup table (or
// by arithmetic on evenly spaced thresholds) and settled by exact comparisons with the thresholds.
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

// One finished trial (all 32 lanes of a warp): its histograms (p.hist_copies copies at `hist`, finish-time maxima at
// `fmax` under rule 1) become out_done / out_step / out_sync of trial t, and are cleared.  Bins are taken 128 (or 32)
// at a time: a lane sums its bins over the copies (and clears them), a warp scan gives the prefix, a carry links the
// steps.  `segmax` holds the bit pattern of the trial's largest row total.
template <int RULE>
__device__ __forceinline__ void epilogue_trial(const SweepParams &p, const SmemTail &s, int *hist, float *fmax, int *segmax,
                                               long long t, int lane)
{
    const int K = p.K, H = p.hist_copies, HS = p.hist_stride;
    const float Tmax = __int_as_float(*segmax);
    const float t_comm = p.t_comm_vec ? p.t_comm_vec[t] : p.t_comm;
    float *step_row = p.out_step + t * K;
    int32_t *done_row = p.out_done + t * K;
    int carry = 0;
    float fm_carry = 0.0f;
    // Four consecutive bins per lane, 128 bins per step, with 16-byte accesses throughout (when the shapes
    // and pointers allow): a quarter of the scans and well under half the instructions of the scalar loop.
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
    if (lane == 0) {
        *segmax = 0;
        if (p.out_sync != nullptr) p.out_sync[t] = __fadd_rn(Tmax, t_comm);
    }
}

// Several small trials in one step of a warp: L = p.epi_sub = K/4 lanes (a power of two) take one trial, four bins
// each, and the scans run inside groups of L lanes, so 32/L trials of a tile (seg0, seg0 + 1, ...) go through the warp
// at once.  `slot0` = index of the tile's first trial among the histogram slots.
template <int RULE>
__device__ __forceinline__ void epilogue_small_trials(const SweepParams &p, const SmemTail &s, int slot0, long long t0, int seg0,
                                                      int lane)
{
    const int K = p.K, H = p.hist_copies, HS = p.hist_stride, G = p.g;
    const int L = p.epi_sub;
    const int sub = lane & (L - 1), k = 4 * sub;
    const int seg = seg0 + lane / L;
    const long long t = t0 + seg;
    const bool in = seg < G && t < p.T;
    int4 h = make_int4(0, 0, 0, 0);
    float4 fm = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    float Tmax = 0.0f;
    if (in) {
        for (int c = 0; c < H; ++c) {
            int4 *hp = reinterpret_cast<int4 *>(s.hist + ((slot0 + seg) * H + c) * HS + k);
            const int4 v = *hp;
            *hp = make_int4(0, 0, 0, 0);
            h.x += v.x; h.y += v.y; h.z += v.z; h.w += v.w;
            if (RULE == 1) {
                float4 *fp = reinterpret_cast<float4 *>(s.fmax + ((slot0 + seg) * H + c) * HS + k);
                const float4 f = *fp;
                *fp = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                fm.x = fmaxf(fm.x, f.x); fm.y = fmaxf(fm.y, f.y); fm.z = fmaxf(fm.z, f.z); fm.w = fmaxf(fm.w, f.w);
            }
        }
        Tmax = __int_as_float(s.segmax[slot0 + seg]);
    }
    h.y += h.x; h.z += h.y; h.w += h.z;  // inclusive inside the lane
    int incl = h.w;
    for (int o = 1; o < L; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, o, L);
        if (sub >= o) incl += u;
    }
    const int base = incl - h.w;  // everything before this lane's bins, within its trial
    float4 st;
    if (RULE == 0) {
        const float4 tq = *reinterpret_cast<const float4 *>(s.tau_s + k);
        st.x = fminf(tq.x, Tmax); st.y = fminf(tq.y, Tmax); st.z = fminf(tq.z, Tmax); st.w = fminf(tq.w, Tmax);
    } else {
        fm.y = fmaxf(fm.y, fm.x); fm.z = fmaxf(fm.z, fm.y); fm.w = fmaxf(fm.w, fm.z);
        float fincl = fm.w;
        for (int o = 1; o < L; o <<= 1) {
            const float u = __shfl_up_sync(0xffffffffu, fincl, o, L);
            if (sub >= o) fincl = fmaxf(fincl, u);
        }
        float before = __shfl_up_sync(0xffffffffu, fincl, 1, L);
        before = sub > 0 ? before : 0.0f;
        st.x = fmaxf(before, fm.x); st.y = fmaxf(before, fm.y); st.z = fmaxf(before, fm.z); st.w = fmaxf(before, fm.w);
    }
    if (in) {
        const float t_comm = p.t_comm_vec ? p.t_comm_vec[t] : p.t_comm;
        *reinterpret_cast<int4 *>(p.out_done + t * K + k) = make_int4(base + h.x, base + h.y, base + h.z, base + h.w);
        *reinterpret_cast<float4 *>(p.out_step + t * K + k) =
            make_float4(__fadd_rn(st.x, t_comm), __fadd_rn(st.y, t_comm), __fadd_rn(st.z, t_comm), __fadd_rn(st.w, t_comm));
        if (sub == 0) {  // the two bins past the last threshold, the trial's maximum, the synchronous time
            for (int c = 0; c < H; ++c) {
                s.hist[((slot0 + seg) * H + c) * HS + K] = 0;
                s.hist[((slot0 + seg) * H + c) * HS + K + 1] = 0;
                if (RULE == 1) {
                    s.fmax[((slot0 + seg) * H + c) * HS + K] = 0.0f;
                    s.fmax[((slot0 + seg) * H + c) * HS + K + 1] = 0.0f;
                }
            }
            s.segmax[slot0 + seg] = 0;
            if (p.out_sync != nullptr) p.out_sync[t] = __fadd_rn(Tmax, t_comm);
        }
    }
}

// The trials of one finished tile, shared out over `nw` warps (this is warp `w` of them): whole trials, or groups of
// small trials per step.  slot0 = index of the tile's first trial among the histogram slots.
template <int RULE>
__device__ __forceinline__ void epilogue_tile(const SweepParams &p, const SmemTail &s, int slot0, long long tile, int w, int nw,
                                              int lane)
{
    const int G = p.g, seg_ints = p.hist_copies * p.hist_stride;
    const long long t0 = tile * G;
    if (p.epi_sub > 0) {
        const int per_step = 32 / p.epi_sub;
        for (int seg0 = w * per_step; seg0 < G; seg0 += nw * per_step) epilogue_small_trials<RULE>(p, s, slot0, t0, seg0, lane);
    } else {
        for (int seg = w; seg < G && t0 + seg < p.T; seg += nw)  // (nothing was added for trials past the last one)
            epilogue_trial<RULE>(p, s, s.hist + (slot0 + seg) * seg_ints, s.fmax + (slot0 + seg) * seg_ints,
                                 s.segmax + slot0 + seg, t0 + seg, lane);
    }
}

// The epilogue warp's loop (all 32 lanes) over the block's tiles when a tile is one trial: the consumers fill
// histogram buffer j&1 for their j-th trial and go straight on while this warp turns the other buffer into outputs.
// (Tiles of several small trials are finished by the consumer warps themselves, see tiled_trials.)
template <int RULE>
__device__ __forceinline__ void epilogue_warp(const SweepParams &p, const SmemTail &s, int lane, int ncw)
{
    if (p.nbuf == 1) return;
    const int bar_threads = ncw * 32 + 32;
    const long long tiles = (p.T + p.g - 1) / p.g;
    int j = 0;
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++j) {
        const int b = j & 1;
        buffer_barrier_sync<kBarReady>(b, bar_threads);  // every consumer has finished this tile
        epilogue_tile<RULE>(p, s, b * p.g, tile, 0, 1, lane);
        buffer_barrier_arrive<kBarFree>(b, bar_threads);  // buffer b is clear again
    }
}

// The consumer threads' loop over the block's tiles (tiled kernel).  A tile is p.g whole trials (thread r owns row
// pass * p.rows + r of the tile's g*N rows in pass `pass`, which belongs to trial (that row) / N of the tile), or one
// trial whose workers are taken in p.passes passes of p.rows rows.  LEAN = every chunk of a row is full (consume_full).
template <int NQ, int RULE, bool BATCH, bool DIRECT, bool LEAN, bool ONE, bool MULTI>
__device__ __forceinline__ void tiled_trials_g(const SweepParams &p, const SmemTail &s, const BinCtx &ctx, unsigned char *stage0,
                                             uint64_t *full, uint64_t *empty, int tid, int lane, int warp, int ncw,
                                             unsigned fmax_delta, unsigned off_zero)
{
    const int S = p.stages, G = MULTI ? p.g : 1;  // (MULTI = several trials per tile: compiled apart, the one-trial loop carries none of it)
    const int bar_threads = ncw * 32 + 32;
    const int seg_ints = p.hist_copies * p.hist_stride;  // one trial's histograms
    // Threads past the last row of the tile shadow rows of the tile (different ones, so that what they add to the
    // spare histogram copy spreads over its bins like real rows do).
    const int row = tid < p.rows ? tid : tid % p.rows;
    const int copy = (warp % p.warp_groups) * p.lane_copies + (lane & (p.lane_copies - 1));
    int *copy0 = s.hist + copy * p.hist_stride;  // this thread's copy in the histograms of buffer 0, trial 0
    // Byte offset of this thread's quad q inside a stage.  The tile is a dense copy of its rows; the hardware
    // swizzle XORs bits 4..6 of an offset with (bits 7..9 & swz_mask), which moves 16-byte quads inside 128-byte lines
    // (rows may be shorter than a line, or not a divisor of it, when they are fetched as whole lines).
    const uint32_t row_off = (uint32_t)row * (uint32_t)p.pitch;
    uint32_t qoff[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const uint32_t o = row_off + (uint32_t)(q * 16);
        qoff[q] = o ^ (((o >> 7) & (uint32_t)p.swz_mask) << 4);
    }
    // the spare histogram copy (after all real ones, never read): where lanes without a row of their own add
    const uint32_t spare_a = smem_addr(s.hist + (hist_slots(p) - 1) * p.hist_stride);
    const uint32_t stage0_a = smem_addr(stage0);
    const long long tiles = (p.T + G - 1) / G;
    int st = 0;
    uint32_t ph = 0;
    int j = 0;
    const bool own_epilogue = p.nbuf == 1;  // tiles of several small trials: the consumer warps finish them themselves
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++j) {
        const int b = own_epilogue ? 0 : (j & 1);
        if (!own_epilogue && j >= 2) buffer_barrier_sync<kBarFree>(b, bar_threads);  // the epilogue warp has cleared buffer b
        float rowmax = 0.0f, fin0 = 0.0f;
        int cnt0 = 0;
        int *myhist = copy0 + b * G * seg_ints;
        for (int pass = 0; pass < p.passes; ++pass) {
            // This thread's row in this pass, the trial of the tile it belongs to, and whether both exist.  With
            // several trials per tile the tile's rows are one run of G N rows taken p.rows at a time, so a thread's
            // rows in different passes belong to different trials and everything it counts is handed over per pass.
            int seg = 0;
            bool valid;
            if (G > 1) {
                seg = (pass * p.rows + tid) / p.N;
                valid = tid < p.rows && seg < G && tile * G + seg < p.T;
                if (!valid) seg = 0;
                myhist = copy0 + (b * G + seg) * seg_ints;
            } else {
                valid = tid < p.rows && pass * p.rows + tid < p.N;
            }
            unsigned char *hist_b = reinterpret_cast<unsigned char *>(myhist);
            float P = 0.0f, pass_fin0 = 0.0f;
            int pass_cnt0 = 0;
            const uint32_t hist_a = valid ? smem_addr(hist_b) : spare_a;  // (short loop) where this lane adds in this pass
            // rule 1: bin of the running time before the next micro-batch, as a byte offset (general loop) or as the
            // address of that bin in this lane's histogram copy (short loop)
            unsigned prev = LEAN ? hist_a + off_zero : off_zero;
            for (int c = 0; c < p.chunks; ++c) {
                mbar_wait(&full[st], ph, kErrLoadNeverArrived);
                const unsigned char *stage = stage0 + (size_t)st * p.stage_bytes;
                const uint32_t stage_a = stage0_a + (uint32_t)st * (uint32_t)p.stage_bytes;
                uint64_t *empty_bar = &empty[st];
                if (++st == S) {
                    st = 0;
                    ph ^= 1u;
                }
                float4 v[NQ];
                if (LEAN) {
#pragma unroll
                    for (int q = 0; q < NQ; ++q) v[q] = lds_stage_f32x4(stage_a + qoff[q]);
                    consume_full<NQ, RULE, BATCH, DIRECT, ONE>(v, lane, ctx, hist_a, fmax_delta, P, prev, pass_cnt0, pass_fin0, empty_bar);
                } else {
                    const int nq = (c == p.chunks - 1) ? p.nq_last : NQ;
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        if (q < nq) v[q] = *reinterpret_cast<const float4 *>(stage + qoff[q]);
                        else v[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    }
                    consume_chunk<NQ, RULE, BATCH, DIRECT>(v, 4 * nq, valid, lane, ctx, hist_b, fmax_delta, P, prev, pass_cnt0, pass_fin0, empty_bar);
                }
            }
            // (a lane without a row in this pass drops what it counted: the row's owner has it)
            if (G > 1 && p.N >= 32) {
                // The 32 consecutive rows of a warp belong to at most two trials: the lanes of each add up what they
                // kept in registers (bin-0 counts; largest bin-0 finish time; largest total) and one lane hands it over
                // (any copy of the trial's histograms will do, they are summed in the end).  Running sums are
                // non-negative, so their bit patterns order like integers and 0 is "nothing".
                const int s0 = __shfl_sync(0xffffffffu, seg, 0);
                const bool in0 = valid && seg == s0, in1 = valid && seg != s0;
                const unsigned others = __ballot_sync(0xffffffffu, in1);
                auto hand_over = [&](bool in, int trial_seg, int lane_out) {
                    const int cnt = __reduce_add_sync(0xffffffffu, in ? pass_cnt0 : 0);
                    const int tot = __reduce_max_sync(0xffffffffu, in ? __float_as_int(P) : 0);
                    const int fin = RULE == 1 ? __reduce_max_sync(0xffffffffu, in ? __float_as_int(pass_fin0) : 0) : 0;
                    if (lane == lane_out) {
                        int *h = copy0 + (b * G + trial_seg) * seg_ints;
                        if (cnt > 0) {
                            atomicAdd(h, cnt);
                            if (RULE == 1) raise_max(reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(h) + fmax_delta), __int_as_float(fin));
                        }
                        if (tot > 0) atomicMax(&s.segmax[b * G + trial_seg], tot);
                    }
                };
                hand_over(in0, s0, 0);
                if (others != 0u) {
                    const int src = __ffs(others) - 1;
                    hand_over(in1, __shfl_sync(0xffffffffu, seg, src), src);
                }
            } else if (valid) {
                if (G > 1) {
                    if (pass_cnt0 > 0) {
                        atomicAdd(myhist, pass_cnt0);
                        if (RULE == 1) raise_max(reinterpret_cast<float *>(hist_b + fmax_delta), pass_fin0);
                    }
                    // largest row total of the trial: running sums are non-negative, so their bit patterns order like integers
                    atomicMax(&s.segmax[b * G + seg], __float_as_int(P));
                } else {
                    rowmax = fmaxf(rowmax, P);
                    cnt0 += pass_cnt0;
                    fin0 = fmaxf(fin0, pass_fin0);
                }
            }
        }
        if (G == 1) {
            if (cnt0 > 0) {
                atomicAdd(myhist, cnt0);
                if (RULE == 1) raise_max(reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(myhist) + fmax_delta), fin0);
            }
            const unsigned wm = __reduce_max_sync(0xffffffffu, (unsigned)__float_as_int(rowmax));
            if (lane == 0) atomicMax(&s.segmax[b], (int)wm);
        }
        if (own_epilogue) {
            // every consumer has added its rows; each warp then turns a share of the tile's trials into outputs and
            // clears their histograms; nobody starts the next tile before all of that is done
            bar_sync_imm<kConsumerBarrier>(ncw * 32);
            epilogue_tile<RULE>(p, s, 0, tile, warp, ncw, lane);
            bar_sync_imm<kConsumerBarrier>(ncw * 32);
        } else {
            buffer_barrier_arrive<kBarReady>(b, bar_threads);  // hand buffer b to the epilogue warp
        }
    }
}

template <int NQ, int RULE, bool BATCH, bool DIRECT, bool LEAN, bool ONE = true>
__device__ __forceinline__ void tiled_trials(const SweepParams &p, const SmemTail &s, const BinCtx &ctx, unsigned char *stage0,
                                             uint64_t *full, uint64_t *empty, int tid, int lane, int warp, int ncw,
                                             unsigned fmax_delta, unsigned off_zero)
{
    if (p.g > 1) tiled_trials_g<NQ, RULE, BATCH, DIRECT, LEAN, ONE, true>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
    else tiled_trials_g<NQ, RULE, BATCH, DIRECT, LEAN, ONE, false>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
}

// WIDE = tiles of two trials of 129-256 workers each (up to 512 rows, 16 consumer warps): fewer idle lanes in the last
// warp of a trial and half the hand-overs per trial.
// LEAN = every chunk of every row is full: the kernel holds the short consumer loop only (three forms: cell
// arithmetic, table, table with several thresholds per cell); otherwise the general loop only (two forms).  Keeping
// the two apart keeps each kernel's code small: with both loops in one kernel the general one measured 5-17 % slower.
template <int NQ, int RULE, bool BATCH, bool WIDE, bool LEAN>
__global__ void __launch_bounds__(WIDE ? 2 * kMaxRowsPerPass + 64 : kMaxRowsPerPass + 64, WIDE ? 2 : (NQ <= 4 ? 3 : 2))
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
    // first boxes are on their way from HBM while the thresholds are read and the lookup table is built.
    // (box = one chunk of one pass of one tile; the block's boxes in order: tile, pass, chunk.  With several trials
    // per tile the box is {chunk, all N workers, g trials}; trials past the last one are zero-filled.)
    const long long tiles = (p.T + p.g - 1) / p.g;
    long long prod_t = blockIdx.x;
    int prod_pass = 0, prod_c = 0, prod_issued = 0;
    auto issue_tile = [&](int st) {
        mbar_arrive_expect_tx(&full[st], (uint32_t)(p.rows * p.pitch));
        tma_load_3d(stage0 + (size_t)st * p.stage_bytes, &lat_map, prod_c * p.bw, prod_pass * p.box_y + (int)(prod_t * p.tile_y),
                    (int)(prod_t * p.tile_z), &full[st]);
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
        while (prod_issued < S && prod_t < tiles) issue_tile(prod_issued++);
    }
    load_thresholds(p, s, tid, blockDim.x);
    __syncthreads();  // also: the initialised barriers are visible to every thread
    build_lut(p, s, tid, blockDim.x);

    if (warp == ncw) {
        // ---------------- producer: the rest of the tiles, each into the stage its predecessor has been read out of
        if (lane == 0) {
            int st = 0;
            uint32_t ph = 1;  // parity of the current use of stage st (every stage has been used once)
            while (prod_t < tiles) {
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
    // rule 1: byte distance from a histogram entry to the finish-time maximum of the same buffer, trial, copy and bin
    const unsigned fmax_delta = (unsigned)(reinterpret_cast<unsigned char *>(s.fmax) - reinterpret_cast<unsigned char *>(s.hist));
    const BinCtx ctx = make_bin_ctx(p, s);
    const bool one = ctx.one;
    const unsigned off_zero = RULE == 1 ? bin_of_zero(ctx) : 0u;  // rule 1 only
    const bool direct = s.meta[3] != 0 && one && p.direct_bins != 0;
    if constexpr (LEAN) {
        if (direct) tiled_trials<NQ, RULE, BATCH, true, true, true>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
        else if (one) tiled_trials<NQ, RULE, BATCH, false, true, true>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
        else tiled_trials<NQ, RULE, BATCH, false, true, false>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
    } else {
        if (direct) tiled_trials<NQ, RULE, BATCH, true, false>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
        else tiled_trials<NQ, RULE, BATCH, false, false>(p, s, ctx, stage0, full, empty, tid, lane, warp, ncw, fmax_delta, off_zero);
    }
}

}  // namespace
