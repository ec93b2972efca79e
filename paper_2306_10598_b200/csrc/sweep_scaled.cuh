// The sweep for heterogeneous workers: worker n works against its own thresholds s_n * tau_k.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// App. C.2 remarks that workers need not be identical (each may have its own mu_n, sigma_n).  Here worker n is given
// the threshold theta_{n,k} = fl32(s_n * tau_k) (one fp32 product, s_n > 0) instead of the common tau_k:
//   rule 0  micro-batch m counts iff P_{n,m} < theta_{n,k}; the worker's time is min{theta_{n,k}, T_n} (Sec. 4.3 per
//           worker) and the step is the maximum of those over workers plus T^c;
//   rule 1  micro-batch m is run iff P_{n,m-1} < theta_{n,k}; the worker's time is the finish time of the last one run.
// theta_{n,k} is non-decreasing in k (rounding is monotone), so a running sum P of row n falls into the bin
// j = #{k : theta_{n,k} <= P}.  The table over the COMMON thresholds proposes a bin for P / s_n; exact comparisons
// of P with fl32(s_n * tau_k) on both sides of the proposal settle it, so the bins are those of the definition
// whatever the proposal was.  Sixteen samples of a row are held in registers at a time: their running sums are
// formed first (left to right), quads that every lane of the warp still has below its first threshold are counted
// in a register, the others are binned sample by sample.
//
// One block per trial at a time, thread r takes rows r, r + blockDim, ...; everything per trial lives in shared memory:
//   hist[j]   completed (rule 0) / started (rule 1) micro-batches by bin, prefix-summed into out_done
//   rule 0:   scale_hi[b] = largest s_n and total_hi[b] = largest T_n among the rows whose TOTAL falls into bin b.  A row
//             with total bin b > k still runs at threshold k (its time is theta_{n,k}); with b <= k it has finished (T_n):
//                 step_k = max( fl32(S * tau_k), max_{b <= k} total_hi[b] ) + T^c,
//             S = largest s_n over bins b > k (tau_k >= 0; rounding is monotone) or the smallest s_n of all rows
//             (tau_k < 0: then every row still runs and s * tau_k decreases with s).
//   rule 1:   fin_hi[a] = largest finish time among the micro-batches whose START falls into bin a; step_k is the
//             prefix maximum (the same point updates as in the other kernels, with the row's own bins).
// Positive floats order like their bit patterns, so the maxima and the minimum are integer atomics; -1 marks "none".
// A plain kernel (ordinary 16-byte loads of the thread's own row, no staging): bound by instruction issue, not by HBM.
// ------------------------------------------------------------------------------------------
constexpr int kScaledThreads = 256;
constexpr int kScaledGroup = 16;  // samples of a row held in registers at a time

__host__ __device__ inline int scaled_lut_cells(int K) { return min(kLutCellsMax, 4 * K); }
__host__ __device__ inline size_t scaled_smem_bytes(int K)
{
    return sizeof(int) * (size_t)(5 * (K + 4) + 16) + (((size_t)(scaled_lut_cells(K) + 1) * sizeof(unsigned short) + 15) & ~(size_t)15);
}

template <int RULE>
__global__ void __launch_bounds__(kScaledThreads)
dc_sweep_scaled(const float *__restrict__ lat, const float *__restrict__ taus, const float *__restrict__ scale, long long T, int N,
                int M, int K, float t_comm, float *out_step, int32_t *out_done, float *out_sync)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *tau_s = reinterpret_cast<float *>(smem_raw);      // K + 1 (tau_s[K] = +inf)
    int *hist = reinterpret_cast<int *>(tau_s + (K + 4));     // K + 2 (bins 0..K)
    int *a_hi = hist + (K + 4);                               // rule 0: scale_hi bits, rule 1: fin_hi bits
    int *b_hi = a_hi + (K + 4);                               // rule 0: total_hi bits
    int *above = b_hi + (K + 4);                              // rule 0: largest scale over bins > k (bits), -1 if none
    int *misc = above + (K + 4);                              // [0] smallest scale bits, [1] largest total bits
    int *meta = misc + 8;                                     // the lookup table's parameters (build_lut)
    unsigned short *lut = reinterpret_cast<unsigned short *>(meta + 8);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool vec4 = (M % 4 == 0) && ((reinterpret_cast<uintptr_t>(lat) & 15) == 0);
    for (int k = tid; k < K; k += blockDim.x) tau_s[k] = taus[k];
    if (tid == 0) {
        misc[0] = 0x7f800000;                    // +inf
        tau_s[K] = __int_as_float(0x7f800000);  // sentinel: nothing reaches it
    }
    __syncthreads();
    {  // the smallest scale is the same for every trial: one reduction per block
        int lo = 0x7f800000;
        for (int n = tid; n < N; n += blockDim.x) lo = min(lo, __float_as_int(scale[n]));
        lo = __reduce_min_sync(0xffffffffu, lo);
        if (lane == 0) atomicMin(&misc[0], lo);
    }
    // The table over equal cells of the common thresholds' range that the other kernels use.  Here it only proposes
    // where to look: a running sum P of a row with scale s is looked up at P / s, and the row's own thresholds
    // fl32(s * tau_k) decide from there by exact comparisons, forward and backward.
    const unsigned C = (unsigned)scaled_lut_cells(K);
    {
        SweepParams lp;
        lp.K = K;
        lp.lut_cells = (int)C;
        SmemTail ls;
        ls.tau_s = tau_s;
        ls.meta = meta;
        ls.lut = lut;
        build_lut(lp, ls, tid, blockDim.x);  // ends with __syncthreads()
    }
    const float lut_lo = __int_as_float(meta[1]), lut_scale = __int_as_float(meta[2]);
    // j(P) = #{k : fl32(s tau_k) <= P} for one row; fl32(s tau_k) is non-decreasing in k
    // The proposal is settled in one step without a branch when it is off by at most one threshold (always, unless a
    // cell holds several thresholds or P / s rounds across a cell border); the loops are the general case.
    auto bin_of = [&](float P, float s, float inv_s) -> int {
        int j = lut[lut_cell(__fmul_rn(P, inv_s), lut_lo, lut_scale, C)] >> 2;   // 0..K
        const bool up = P >= __fmul_rn(s, tau_s[j]);                              // tau_s[K] = +inf
        j += up ? 1 : 0;
        // the neighbour on the other side: theta_j if the step was taken, theta_{j-1} if not
        const float other = __fmul_rn(s, tau_s[up ? min(j, K) : max(j - 1, 0)]);
        const bool settled = up ? (P < other || j >= K) : (P >= other || j == 0);
        if (!settled) {
            while (j < K && P >= __fmul_rn(s, tau_s[j])) ++j;
            while (j > 0 && P < __fmul_rn(s, tau_s[j - 1])) --j;
        }
        return j;
    };

    for (long long t = blockIdx.x; t < T; t += gridDim.x) {
        for (int j = tid; j <= K + 1; j += blockDim.x) {
            hist[j] = 0;
            a_hi[j] = RULE == 0 ? -1 : 0;
            b_hi[j] = -1;
        }
        if (tid == 0) misc[1] = 0;
        __syncthreads();
        int total_hi_bits = 0;  // largest total among this thread's rows
        for (int n0 = 0; n0 < N; n0 += blockDim.x) {  // (uniform trip count: the warp votes below need every lane)
            const int n = n0 + tid;
            const bool valid = n < N;
            const float s = valid ? scale[n] : 1.0f;
            const float inv_s = __fdividef(1.0f, s);
            // rows without a worker behind them add zeros and sit below a first threshold of +inf
            const float first = valid ? __fmul_rn(s, tau_s[0]) : __int_as_float(0x7f800000);
            const float *row = lat + ((size_t)t * N + (valid ? n : 0)) * M;
            float P = 0.0f;
            int in_bin0 = 0;        // bin 0 (where most rows spend their first micro-batches) is counted in registers
            float fin_bin0 = 0.0f;  // rule 1: largest finish time among the micro-batches that start in bin 0
            int last_bin = valid ? bin_of(0.0f, s, inv_s) : 0;  // bin of the running sum so far
            for (int m0 = 0; m0 < M; m0 += kScaledGroup) {
                const int ns = min(kScaledGroup, M - m0);  // the same for every lane
                float x[kScaledGroup];
                if (vec4) {  // rows of whole 16-byte quads on a 16-byte aligned base (ns is a multiple of 4 then)
                    const float4 *row4 = reinterpret_cast<const float4 *>(row + m0);
#pragma unroll
                    for (int q = 0; q < kScaledGroup / 4; ++q) {
                        const float4 v = (valid && 4 * q < ns) ? __ldg(row4 + q) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                        x[4 * q] = v.x;
                        x[4 * q + 1] = v.y;
                        x[4 * q + 2] = v.z;
                        x[4 * q + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kScaledGroup; ++i) x[i] = (valid && i < ns) ? __ldg(row + m0 + i) : 0.0f;
                }
#pragma unroll
                for (int i = 0; i < kScaledGroup; ++i) {  // running sums, strictly left to right (missing samples add 0)
                    P = __fadd_rn(P, x[i]);
                    x[i] = P;
                }
#pragma unroll
                for (int q = 0; q < kScaledGroup / 4; ++q) {
                    if (4 * q >= ns) break;
                    const int nq = min(4, ns - 4 * q);
                    // every lane still below its first threshold (and so was everything before): these samples are bin 0
                    if (__all_sync(0xffffffffu, x[4 * q + 3] < first && last_bin == 0)) {
                        in_bin0 += nq;
                        fin_bin0 = x[4 * q + 3];
                        continue;
                    }
                    if (valid) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (e < nq) {
                                const float Pm = x[4 * q + e];
                                const int here = bin_of(Pm, s, inv_s);
                                const int bin = RULE == 0 ? here : last_bin;
                                last_bin = here;
                                if (bin == 0) {
                                    ++in_bin0;
                                    fin_bin0 = Pm;  // (running sums never decrease)
                                } else {
                                    atomicAdd(&hist[bin], 1);
                                    if (RULE == 1) atomicMax(&a_hi[bin], __float_as_int(Pm));
                                }
                            }
                        }
                    }
                }
            }
            if (valid) {
                if (in_bin0 > 0) {
                    atomicAdd(&hist[0], in_bin0);
                    if (RULE == 1) atomicMax(&a_hi[0], __float_as_int(fin_bin0));
                }
                total_hi_bits = max(total_hi_bits, __float_as_int(P));
            }
            if (RULE == 0 && valid) {  // (merging the lanes of a bin first, by a warp match, measured slower than these)
                atomicMax(&a_hi[last_bin], __float_as_int(s));
                atomicMax(&b_hi[last_bin], __float_as_int(P));
            }
        }
        total_hi_bits = __reduce_max_sync(0xffffffffu, total_hi_bits);
        if (lane == 0) atomicMax(&misc[1], total_hi_bits);
        __syncthreads();
        if (warp == 0) {
            float *step_row = out_step + t * K;
            int32_t *done_row = out_done + t * K;
            if (RULE == 0) {
                // above[k] = largest scale among bins k+1 .. K, from the top down, 32 thresholds at a time
                int carry = -1;
                for (int k0 = ((K - 1) / 32) * 32; k0 >= 0; k0 -= 32) {
                    const int k = k0 + lane;
                    int v = (k < K) ? a_hi[k + 1] : -1;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int u = __shfl_down_sync(0xffffffffu, v, o);
                        if (lane + o < 32) v = max(v, u);
                    }
                    v = max(v, carry);
                    if (k < K) above[k] = v;
                    carry = __shfl_sync(0xffffffffu, v, 0);
                }
                __syncwarp();
            }
            int count_carry = 0, hi_carry = RULE == 0 ? -1 : 0;
            const float s_min = __int_as_float(misc[0]);
            for (int k0 = 0; k0 < K; k0 += 32) {
                const int k = k0 + lane;
                const int h = (k < K) ? hist[k] : 0;
                const int incl = warp_inclusive_scan(h, lane);
                int hi = (k < K) ? (RULE == 0 ? b_hi[k] : a_hi[k]) : (RULE == 0 ? -1 : 0);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int u = __shfl_up_sync(0xffffffffu, hi, o);
                    if (lane >= o) hi = max(hi, u);
                }
                hi = max(hi, hi_carry);
                if (k < K) {
                    done_row[k] = count_carry + incl;
                    float step;
                    if (RULE == 0) {
                        const float tau = tau_s[k];
                        // workers still running at this threshold: all of them when tau < 0, else those in bins above k
                        const bool running = tau < 0.0f || above[k] >= 0;
                        const float run_time = __fmul_rn(tau < 0.0f ? s_min : __int_as_float(above[k]), tau);
                        const bool finished = hi >= 0;
                        const float fin_time = __int_as_float(hi);
                        step = running ? (finished ? fmaxf(run_time, fin_time) : run_time) : fin_time;
                    } else {
                        step = __int_as_float(hi);
                    }
                    step_row[k] = __fadd_rn(step, t_comm);
                }
                count_carry += __shfl_sync(0xffffffffu, incl, 31);
                hi_carry = __shfl_sync(0xffffffffu, hi, 31);
            }
            if (lane == 0 && out_sync != nullptr) out_sync[t] = __fadd_rn(__int_as_float(misc[1]), t_comm);
        }
        __syncthreads();
    }
}

}  // namespace
