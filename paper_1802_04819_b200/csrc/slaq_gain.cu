// Marginal gains: expand every job's fitted curve into the predicted loss reduction of its
// n-th core, n = 1..max_cores_per_job (the objective Loss_j(a_j, t) - Loss_j(a_j, t+T) of
// "Scheduling Based on Quality Improvements", differenced in a_j).
//
// An iteration on n cores takes t(n) = s + w/n seconds, so an epoch of T seconds runs
// m(n) = T n / (s n + w) iterations; in window coordinates that is X_n = m(n) / span ahead
// of the newest point, and R(n) = f(0) - f(X_n).  g(n) = R(n) - R(n-1) is evaluated without
// cancellation (divisions by Newton reciprocals: a gain is good to a few ulp), clamped to +0
// where it is not a positive finite number, and made non-increasing in n by a running minimum.  One warp per job; the row is written once,
// coalesced, and its keys feed the first histogram of the threshold selection.
#include <math_constants.h>

#include "slaq_internal.cuh"
#include "slaq_gain_curve.cuh"

namespace slaq {

namespace {

using namespace gaincurve;

constexpr int kWarpsPerBlock = 8;

// Slopes of the upper concave envelope of the points (n, R(n)), n = 0..cap, written over the row
// (row[n-1] holds the clamped difference R(n) - R(n-1) on entry).  One thread walks the row: a stack
// of envelope vertices, a point leaving it when it lies on or below the chord from the vertex
// before it to the new point.  Rows that need this are rare (the fit is not convex ahead).
__device__ void envelope_of_row(double* row, int cap, unsigned short* stack) {
    double run = 0.0;
    for (int n = 1; n <= cap; ++n) {   // differences -> R(n) in place
        run += row[n - 1];
        row[n - 1] = run;
    }
    auto R = [&](int n) { return n == 0 ? 0.0 : row[n - 1]; };
    int top = 0;
    for (int n = 0; n <= cap; ++n) {
        while (top >= 2) {
            const int a = stack[top - 2], b = stack[top - 1];
            if ((R(b) - R(a)) * (double)(n - b) <= (R(n) - R(b)) * (double)(b - a)) --top;
            else break;
        }
        stack[top++] = (unsigned short)n;
    }
    // slopes, written from the right so that R(a) of each segment is still in place when it is read
    for (int v = top - 1; v >= 1; --v) {
        const int a = stack[v - 1], b = stack[v];
        const double slope = (R(b) - R(a)) / (double)(b - a);
        for (int n = b; n > a; --n) row[n - 1] = slope;
    }
}

// kOptions: the instantiation that knows the two options of the prediction (the plain one carries none of
// their code).  options: bit 0 = rows become the slopes of the concave envelope of R(n) instead of a
// running minimum; target-loss hints are read per job.
template <bool kOptions>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
gain_kernel(JobArrays job, FitArrays fit, int max_jobs, int cap, double T, int first_unit, double* __restrict__ gain,
            unsigned long long* __restrict__ hist0, int options) {
    __shared__ unsigned int sh_hist[kRadixBins];
    __shared__ unsigned short sh_stack[kOptions ? kWarpsPerBlock : 1][kOptions ? kMaxCoresLimit + 1 : 1];
    const bool envelope = kOptions && (options & 1) != 0;
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * kWarpsPerBlock;
    for (int j = blockIdx.x * kWarpsPerBlock + warp; j < max_jobs; j += warps_total) {
        const bool active = job.count[j] > 0;
        bool no_time = false;
        const Curve c = load_curve(job, fit, j, max_jobs, T, &no_time);
        if (no_time && lane == 0) fit.status[j] = SLAQ_JOB_NO_TIME;
        // A target-loss hint caps the predicted reduction at (newest loss - target) / M.
        double reduction_cap = CUDART_INF;
        if (kOptions && c.kind != 3) {
            const double target = job.target[j];
            const double M = fit.largest[j];
            if (finite_d(target) && M > 0.0) {
                const int ring = job.cap[j];
                int at = job.head[j] - 1;
                at += at < 0 ? ring : 0;
                const double newest = index_ok(at, ring, kErrStorage, job.err_word) ? job.row[j][at] : 0.0;
                reduction_cap = __ddiv_rn(fmax(newest - target, 0.0), M);
            }
        }
        if (kOptions && (envelope || reduction_cap < CUDART_INF)) {
            // General path (options in use): the row is completed in memory first, then read back for the cap
            // and the histogram.
            double* row = gain + (size_t)j * cap;
            double prev = CUDART_INF, carry_min = CUDART_INF;
            int rises = 0;
            for (int base = 0; base < cap; base += 32) {
                const int n = base + lane + 1;
                double g = CUDART_INF;
                if (n <= cap) g = c.kind == 3 ? 0.0 : raw_gain(c, n);
                if (envelope) {
                    double left = __shfl_up_sync(kFull, g, 1);
                    if (lane == 0) left = prev;
                    rises |= (n <= cap && g > left) ? 1 : 0;
                    prev = __shfl_sync(kFull, g, 31);
                } else {
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double up = __shfl_up_sync(kFull, g, o);
                        if (lane >= o) g = fmin(g, up);
                    }
                    g = fmin(g, carry_min);
                    carry_min = __shfl_sync(kFull, g, 31);
                }
                if (n <= cap && index_ok((long long)j * cap + (n - 1), (long long)max_jobs * cap, kErrGain, job.err_word))
                    row[n - 1] = g;
            }
            __syncwarp();
            if (envelope && __any_sync(kFull, rises)) {
                if (lane == 0) envelope_of_row(row, cap, sh_stack[warp]);
                __syncwarp();
            }
            double before = 0.0;   // uncapped reduction of the cores before this chunk
            for (int base = 0; base < cap; base += 32) {
                const int n = base + lane + 1;
                double g = n <= cap ? row[n - 1] : 0.0;
                if (reduction_cap < CUDART_INF) {
                    double incl = g;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double up = __shfl_up_sync(kFull, incl, o);
                        if (lane >= o) incl += up;
                    }
                    const double left = reduction_cap - (before + (incl - g));
                    before += __shfl_sync(kFull, incl, 31);
                    g = left > 0.0 ? fmin(g, left) : 0.0;
                    if (n <= cap) row[n - 1] = g;
                }
                const bool counted = active && n <= cap && n >= first_unit;
                const unsigned digit = (unsigned)((unsigned long long)__double_as_longlong(g) >> (64 - kRadixBits));
                const unsigned live = __ballot_sync(kFull, counted);
                if (counted) {
                    const unsigned peers = __match_any_sync(live, digit);
                    if ((int)(__ffs(peers) - 1) == lane && index_ok(digit, kRadixBins, kErrBin, job.err_word))
                        atomicAdd(&sh_hist[digit], (unsigned)__popc(peers));
                }
            }
            continue;
        }
        double carry = CUDART_INF;   // running minimum of the gains before this chunk
        for (int base = 0; base < cap; base += 32) {
            const int n = base + lane + 1;
            double g = CUDART_INF;
            if (n <= cap) g = c.kind == 3 ? 0.0 : raw_gain(c, n);
            // inclusive running minimum over n; most chunks fall already (convex fits), which one look at the
            // left neighbour shows
            double left = __shfl_up_sync(kFull, g, 1);
            if (lane == 0) left = carry;
            if (!__all_sync(kFull, n > cap || !(g > left))) {
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double up = __shfl_up_sync(kFull, g, o);
                    if (lane >= o) g = fmin(g, up);
                }
                g = fmin(g, carry);
            }
            carry = __shfl_sync(kFull, g, 31);
            const bool counted = active && n <= cap && n >= first_unit;
            if (n <= cap && index_ok((long long)j * cap + (n - 1), (long long)max_jobs * cap, kErrGain, job.err_word))
                gain[(size_t)j * cap + (n - 1)] = g;
            const unsigned digit = (unsigned)((unsigned long long)__double_as_longlong(g) >> (64 - kRadixBits));
            // lanes with the same digit add once: a row is nearly constant in its top bits, and often the whole
            // chunk shares one digit
            const unsigned live = __ballot_sync(kFull, counted);
            if (live) {
                const unsigned first_digit = __shfl_sync(kFull, digit, __ffs(live) - 1);
                if (__all_sync(kFull, !counted || digit == first_digit)) {
                    if (lane == __ffs(live) - 1 && index_ok(digit, kRadixBins, kErrBin, job.err_word))
                        atomicAdd(&sh_hist[digit], (unsigned)__popc(live));
                } else if (counted) {
                    const unsigned peers = __match_any_sync(live, digit);
                    if ((int)(__ffs(peers) - 1) == lane && index_ok(digit, kRadixBins, kErrBin, job.err_word))
                        atomicAdd(&sh_hist[digit], (unsigned)__popc(peers));
                }
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) {
        const unsigned v = sh_hist[i];
        if (v) atomicAdd(&hist0[i], (unsigned long long)v);
    }
}

__global__ void time_model_kernel(JobArrays job, int max_jobs, double* out_s, double* out_w) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= max_jobs) return;
    double s = CUDART_NAN, w = CUDART_NAN;
    (void)time_law(job, j, max_jobs, s, w);   // leaves NaN where the job has neither a fixed law nor samples
    out_s[j] = s;
    out_w[j] = w;
}

}  // namespace

int launch_gain(slaq_handle* h, double epoch_seconds, int first_unit) {
    int blocks = h->sm_count * 4;
    const int needed = (h->max_jobs + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > needed) blocks = needed;
    const auto kernel = (h->gain_envelope || h->n_hinted > 0) ? gain_kernel<true> : gain_kernel<false>;
    kernel<<<blocks, kWarpsPerBlock * 32, 0, h->stream>>>(h->job, h->fit, h->max_jobs, h->max_cores, epoch_seconds,
                                                         first_unit, h->gain, h->scratch.hist, h->gain_envelope ? 1 : 0);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("gain kernel launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return 1;
}

int launch_time_model(slaq_handle* h, double* d_s, double* d_w) {
    const int threads = 256, blocks = (h->max_jobs + threads - 1) / threads;
    time_model_kernel<<<blocks, threads, 0, h->stream>>>(h->job, h->max_jobs, d_s, d_w);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("time model kernel launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return 1;
}

}  // namespace slaq
