// Trial reduction, tau*, the closed-form companion, group merging, input checks and the read probe.
// Part of dropcompute.cu (one translation unit, included there in this order); everything is internal.
#pragma once

namespace {

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

// Data precondition check: counts latencies that are negative, NaN or infinite, rows (one worker's M latencies)
// of good values whose left-to-right fp32 sum is not finite, and thresholds that are NaN or smaller than their
// predecessor.
__global__ void __launch_bounds__(256)
dc_check_kernel(const float *__restrict__ lat, unsigned long long total, unsigned long long rows, int M,
                const float *__restrict__ taus, int K, unsigned long long *counters)
{
    unsigned long long bad = 0;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const float x = lat[i];
        if (!(x >= 0.0f) || !(x <= 3.402823466e38f)) ++bad;
    }
    for (unsigned long long r = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; r < rows; r += stride) {
        float P = 0.0f;
        bool good = true;
        for (int m = 0; m < M; ++m) {
            const float x = lat[r * (unsigned long long)M + m];
            good = good && (x >= 0.0f) && (x <= 3.402823466e38f);
            P = __fadd_rn(P, x);
        }
        if (good && !(P <= 3.402823466e38f)) ++bad;
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

}  // namespace
