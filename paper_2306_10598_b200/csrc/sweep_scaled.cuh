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
// theta_{n,k} is non-decreasing in k (rounding is monotone) and a row's running sums never decrease, so a row's bin
// j = #{k : theta_{n,k} <= P} only moves forward: a cursor that is advanced by exact comparisons with s_n * tau_k.
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
// A plain kernel (ordinary loads, no staging): this entry point is about the rule, not about bandwidth.
// ------------------------------------------------------------------------------------------
constexpr int kScaledThreads = 256;

__host__ __device__ inline size_t scaled_smem_bytes(int K) { return sizeof(int) * (size_t)(5 * (K + 4) + 8); }

template <int RULE>
__global__ void __launch_bounds__(kScaledThreads)
dc_sweep_scaled(const float *__restrict__ lat, const float *__restrict__ taus, const float *__restrict__ scale, long long T, int N,
                int M, int K, float t_comm, float *out_step, int32_t *out_done, float *out_sync)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *tau_s = reinterpret_cast<float *>(smem_raw);      // K + 1 (tau_s[K] unused)
    int *hist = reinterpret_cast<int *>(tau_s + (K + 4));     // K + 2 (bins 0..K)
    int *a_hi = hist + (K + 4);                               // rule 0: scale_hi bits, rule 1: fin_hi bits
    int *b_hi = a_hi + (K + 4);                               // rule 0: total_hi bits
    int *above = b_hi + (K + 4);                              // rule 0: largest scale over bins > k (bits), -1 if none
    int *misc = above + (K + 4);                              // [0] smallest scale bits, [1] largest total bits
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool vec4 = (M % 4 == 0) && ((reinterpret_cast<uintptr_t>(lat) & 15) == 0);
    for (int k = tid; k < K; k += blockDim.x) tau_s[k] = taus[k];
    __syncthreads();

    for (long long t = blockIdx.x; t < T; t += gridDim.x) {
        for (int j = tid; j <= K + 1; j += blockDim.x) {
            hist[j] = 0;
            a_hi[j] = RULE == 0 ? -1 : 0;
            b_hi[j] = -1;
        }
        if (tid == 0) {
            misc[0] = 0x7f800000;  // +inf
            misc[1] = 0;
        }
        __syncthreads();
        for (int n = tid; n < N; n += blockDim.x) {
            const float s = scale[n];
            const float *row = lat + ((size_t)t * N + n) * M;
            float P = 0.0f;
            int j = 0;  // bin of the running sum so far: thresholds 0..j-1 are <= it
            while (j < K && 0.0f >= __fmul_rn(s, tau_s[j])) ++j;
            int in_bin0 = 0;        // bin 0 (where most rows spend their first micro-batches) is counted in registers
            float fin_bin0 = 0.0f;  // rule 1: largest finish time among the micro-batches that start in bin 0
            auto one_sample = [&](float x) {
                const int start_bin = j;
                P = __fadd_rn(P, x);
                while (j < K && P >= __fmul_rn(s, tau_s[j])) ++j;
                const int bin = RULE == 0 ? j : start_bin;
                if (bin == 0) {
                    ++in_bin0;
                    fin_bin0 = P;  // (running sums never decrease)
                } else {
                    atomicAdd(&hist[bin], 1);
                    if (RULE == 1) atomicMax(&a_hi[bin], __float_as_int(P));
                }
            };
            if (vec4) {  // rows of whole 16-byte quads on a 16-byte aligned base: four samples per load
                const float4 *row4 = reinterpret_cast<const float4 *>(row);
                for (int q = 0; q < M / 4; ++q) {
                    const float4 v = __ldg(row4 + q);
                    one_sample(v.x);
                    one_sample(v.y);
                    one_sample(v.z);
                    one_sample(v.w);
                }
            } else {
                for (int m = 0; m < M; ++m) one_sample(__ldg(row + m));
            }
            if (in_bin0 > 0) {
                atomicAdd(&hist[0], in_bin0);
                if (RULE == 1) atomicMax(&a_hi[0], __float_as_int(fin_bin0));
            }
            if (RULE == 0) {
                atomicMax(&a_hi[j], __float_as_int(s));
                atomicMax(&b_hi[j], __float_as_int(P));
                atomicMin(&misc[0], __float_as_int(s));
            }
            atomicMax(&misc[1], __float_as_int(P));
        }
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
