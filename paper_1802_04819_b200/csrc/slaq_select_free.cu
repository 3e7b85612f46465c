// Allocation without a gain table: the same global top-C selection as slaq_alloc.cu, but the gains
// are evaluated where they are needed instead of being written out for every (job, core count).
//
// A job's marginal gains fall with its core count, so everything the selection asks of a row can be
// answered by a binary search over n with the gain of the n-th core evaluated in closed form:
//   - the histogram of the leading key digit needs only the positions at which the row crosses a
//     digit boundary (a row spans a few binades at most);
//   - once the threshold's leading digit is known, each row contributes one contiguous segment of
//     candidates; only those are evaluated and appended (unordered) to one flat list, on which the
//     remaining digits of the threshold are found by an ordinary radix select;
//   - per job, the gains above and at the threshold are counted from its segment again, and the
//     predicted reduction at the allocation sums the job's first a_j gains.
// The effective gain of the n-th core is min(g(1), g(n)): the running minimum of a sequence that
// rises and then falls (a fit that is concave near the newest point, convex later), and the sequence
// itself where it only falls.  Rounding can leave wiggles of an ulp in such a sequence; the search
// treats the row as ordered, every candidate is evaluated explicitly and its key kept inside the
// chosen digit, and both the histogram and the per-job counts use the same search positions, so
// the cores handed out add up exactly and a gain is misplaced only within an ulp of the threshold.
#include <math_constants.h>

#include "slaq_internal.cuh"
#include "slaq_gain_curve.cuh"

namespace slaq {

namespace {

using namespace gaincurve;

constexpr int kThreads = 256;
constexpr int kTopShift = 64 - kRadixBits;

__host__ __device__ inline int pass_shift(int pass) {
    return pass < kRadixPasses - 1 ? 64 - kRadixBits * (pass + 1) : 0;
}
__host__ __device__ inline int pass_bits(int pass) {
    return pass < kRadixPasses - 1 ? kRadixBits : 64 - kRadixBits * (kRadixPasses - 1);
}

struct Row {
    Curve c;
    double g1;   // gain of the first core: no later core counts for more
};

__device__ __forceinline__ unsigned long long key_of(const Row& r, int n) {
    const double g = n == 1 ? r.g1 : fmin(r.g1, raw_gain(r.c, n));
    return (unsigned long long)__double_as_longlong(g);
}

// First n in [lo, hi + 1] whose key lies below `bound`, the keys taken as non-increasing in n.
__device__ int first_below(const Row& r, int lo, int hi, unsigned long long bound) {
    int a = lo, b = hi + 1;
    while (a < b) {
        const int mid = (a + b) >> 1;
        if (key_of(r, mid) < bound) b = mid;
        else a = mid + 1;
    }
    return a;
}

// The row cut into runs of equal leading digit, from the largest gains down: run i starts at `pos`,
// is attributed the digit of the key found there, and ends before the first later n whose key lies
// below that digit's lowest key.  Digits fall strictly from run to run.  f(pos, next, digit) is called
// per run and stops the walk by returning false.  Every kernel that needs these positions walks the
// row with this one routine, so they always agree.
template <class F>
__device__ void walk_runs(const Row& r, int first_unit, int cap, F f) {
    int pos = first_unit;
    while (pos <= cap) {
        const unsigned digit = (unsigned)(key_of(r, pos) >> kTopShift);
        const int next = digit == 0 ? cap + 1 : first_below(r, pos + 1, cap, (unsigned long long)digit << kTopShift);
        if (!f(pos, next, digit)) return;
        pos = next;
    }
}

__device__ bool load_row(const JobArrays& job, const FitArrays& fit, int j, int max_jobs, double T, Row& r) {
    bool no_time = false;
    r.c = load_curve(job, fit, j, max_jobs, T, &no_time);
    if (no_time) fit.status[j] = SLAQ_JOB_NO_TIME;
    r.g1 = r.c.kind == 3 ? 0.0 : raw_gain(r.c, 1);
    return job.count[j] > 0;
}

// Leading-digit histogram of every active row's gains n = first_unit..cap, one thread per job.
__global__ void __launch_bounds__(kThreads)
free_hist0_kernel(JobArrays job, FitArrays fit, int max_jobs, int cap, double T, int first_unit,
                  unsigned long long* __restrict__ hist0) {
    __shared__ unsigned int sh_hist[kRadixBins];
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < max_jobs; j += gridDim.x * blockDim.x) {
        Row r;
        if (!load_row(job, fit, j, max_jobs, T, r) || first_unit > cap) continue;
        walk_runs(r, first_unit, cap, [&](int pos, int next, unsigned digit) {
            if (index_ok(digit, kRadixBins, kErrBin, job.err_word)) atomicAdd(&sh_hist[digit], (unsigned)(next - pos));
            return true;
        });
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) {
        const unsigned v = sh_hist[i];
        if (v) atomicAdd(&hist0[i], (unsigned long long)v);
    }
}

// Each row's candidates (keys whose leading digit is the threshold's) form the segment [lo, hi) of n;
// their keys go to the flat list, clamped into the digit.  seg_lo / seg_hi keep the segment.
__global__ void __launch_bounds__(kThreads)
free_candidates_kernel(JobArrays job, FitArrays fit, int max_jobs, int cap, double T, int first_unit,
                       const SelectState* __restrict__ sel, int32_t* __restrict__ seg_lo, int32_t* __restrict__ seg_hi,
                       unsigned long long* __restrict__ list, unsigned long long* __restrict__ list_len,
                       long long list_cap) {
    if (sel->done) return;
    const unsigned long long top = sel->prefix >> kTopShift;
    const unsigned long long bin_lo = top << kTopShift, bin_hi = bin_lo | ((1ull << kTopShift) - 1ull);
    const int lane = threadIdx.x & 31;
    for (int j0 = blockIdx.x * blockDim.x + threadIdx.x - lane; j0 < max_jobs; j0 += gridDim.x * blockDim.x) {
        const int j = j0 + lane;
        int lo = first_unit, hi = first_unit;
        Row r;
        const bool live = j < max_jobs && load_row(job, fit, j, max_jobs, T, r) && first_unit <= cap;
        if (live) {
            lo = hi = cap + 1;               // no run at or below the threshold's digit: the whole row lies above
            walk_runs(r, first_unit, cap, [&](int pos, int next, unsigned digit) {
                if (digit > top) return true;
                lo = pos;
                hi = digit == top ? next : pos;
                return false;
            });
            seg_lo[j] = lo;
            seg_hi[j] = hi;
        } else if (j < max_jobs) {
            seg_lo[j] = seg_hi[j] = first_unit;
        }
        // the warp reserves one range of the list for all its candidates
        const int mine = live ? hi - lo : 0;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += up;
        }
        const int total = __shfl_sync(kFull, incl, 31);
        unsigned long long base = 0;
        if (lane == 31 && total > 0) base = atomicAdd(list_len, (unsigned long long)total);
        base = __shfl_sync(kFull, base, 31) + (unsigned long long)(incl - mine);
        for (int n = lo; n < lo + mine; ++n) {
            unsigned long long k = key_of(r, n);
            k = k < bin_lo ? bin_lo : (k > bin_hi ? bin_hi : k);
            const long long at = (long long)base + (n - lo);
            if (index_ok(at, list_cap, kErrGain, job.err_word)) list[at] = k;
        }
    }
}

// One digit of the threshold from the flat list: histogram of digit `pass` over the entries that agree
// with the prefix found so far; the last block to finish picks the bin (as the table's passes do).
__global__ void __launch_bounds__(kThreads)
free_flat_pass_kernel(const unsigned long long* __restrict__ list, const unsigned long long* __restrict__ list_len,
                      int pass, unsigned long long* __restrict__ hist_all, SelectState* sel, unsigned int* ticket) {
    __shared__ unsigned int sh_hist[kRadixBins];
    __shared__ unsigned long long sh_scan[kThreads + 1];
    __shared__ bool is_last;
    if (sel->done) return;
    unsigned long long* hist = hist_all + (size_t)pass * kRadixBins;
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    const unsigned long long prefix = sel->prefix;
    const int shift = pass_shift(pass), bits = pass_bits(pass);
    const int above_shift = pass_shift(pass - 1);        // the digits above this one must equal the prefix's
    const unsigned long long n = *list_len;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (unsigned long long)gridDim.x * blockDim.x) {
        const unsigned long long k = list[i];
        if ((k >> above_shift) == (prefix >> above_shift))
            atomicAdd(&sh_hist[(unsigned)(k >> shift) & ((1u << bits) - 1u)], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) {
        const unsigned v = sh_hist[i];
        if (v) atomicAdd(&hist[i], (unsigned long long)v);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(&ticket[1 + pass], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // pick the bin: walk the bins from the top until what is still wanted is covered
    const int t = threadIdx.x, nbins = 1 << bits;
    const int per = (kRadixBins + kThreads - 1) / kThreads;
    unsigned long long mine = 0;
    for (int k = 0; k < per; ++k) {
        const int b = nbins - 1 - (t * per + k);
        if (b >= 0) mine += __ldcg(&hist[b]);
    }
    sh_scan[t] = mine;
    __syncthreads();
    if (t == 0) {
        unsigned long long run = 0;
        for (int i = 0; i < kThreads; ++i) {
            const unsigned long long v = sh_scan[i];
            sh_scan[i] = run;
            run += v;
        }
    }
    __syncthreads();
    const long long want = sel->want;
    __syncthreads();
    unsigned long long above = sh_scan[t];
    for (int k = 0; k < per; ++k) {
        const int b = nbins - 1 - (t * per + k);
        if (b < 0) break;
        const unsigned long long c = __ldcg(&hist[b]);
        if (above < (unsigned long long)want && (unsigned long long)want <= above + c) {
            sel->prefix |= (unsigned long long)b << shift;   // exactly one thread gets here
            sel->want = want - (long long)above;
        }
        above += c;
    }
}

// Per job: gains above the threshold and equal to it, from the job's segment (evaluated again, with
// the same clamp); block sums of the ties for the prefix over job ids.
__global__ void __launch_bounds__(kThreads)
free_count_kernel(JobArrays job, FitArrays fit, int max_jobs, int cap, double T, int first_unit,
                  const SelectState* __restrict__ sel, int32_t* __restrict__ gt, int32_t* __restrict__ eq,
                  long long* __restrict__ block_eq) {
    __shared__ int sh_eq[kThreads / 32];
    const bool none_wanted = sel->done != 0;
    const unsigned long long tau = sel->prefix;
    const unsigned long long top = tau >> kTopShift;
    const unsigned long long bin_lo = top << kTopShift, bin_hi = bin_lo | ((1ull << kTopShift) - 1ull);
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    int my_gt = 0, my_eq = 0;
    if (j < max_jobs && !none_wanted) {
        const int lo = gt[j], hi = eq[j];    // the segment left by the candidates kernel
        if (lo < hi) {
            Row r;
            load_row(job, fit, j, max_jobs, T, r);
            for (int n = lo; n < hi; ++n) {
                unsigned long long k = key_of(r, n);
                k = k < bin_lo ? bin_lo : (k > bin_hi ? bin_hi : k);
                my_gt += k > tau ? 1 : 0;
                my_eq += k == tau ? 1 : 0;
            }
        }
        my_gt += lo - first_unit;            // everything in front of the segment is larger
    }
    if (j < max_jobs) {
        gt[j] = my_gt;
        eq[j] = my_eq;
    }
    int eq_sum = my_eq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) eq_sum += __shfl_xor_sync(kFull, eq_sum, o);
    if ((threadIdx.x & 31) == 0) sh_eq[threadIdx.x >> 5] = eq_sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long total = 0;
        for (int w = 0; w < kThreads / 32; ++w) total += sh_eq[w];
        block_eq[blockIdx.x] = total;
    }
}

// a_j from the counts and the tie prefix; the predicted reduction at a_j sums the job's first a_j
// gains with a running minimum, exactly as a row of the gain table is formed.
__global__ void __launch_bounds__(kThreads)
free_finalise_kernel(JobArrays job, FitArrays fit, int max_jobs, int cap, double T, int floor_units,
                     const SelectState* __restrict__ sel, const int32_t* __restrict__ gt,
                     const int32_t* __restrict__ eq, const long long* __restrict__ block_prefix,
                     int32_t* __restrict__ alloc, double* __restrict__ reduction, int32_t* __restrict__ out_alloc,
                     long long* counters) {
    __shared__ long long sh_pre[kThreads];
    const int t = threadIdx.x;
    const int j = blockIdx.x * blockDim.x + t;
    const int my_eq = j < max_jobs ? eq[j] : 0;
    sh_pre[t] = my_eq;
    __syncthreads();
    for (int o = 1; o < kThreads; o <<= 1) {
        const long long v = t >= o ? sh_pre[t - o] : 0;
        __syncthreads();
        sh_pre[t] += v;
        __syncthreads();
    }
    const long long before = block_prefix[blockIdx.x] + sh_pre[t] - my_eq;
    int a = 0;
    long long ties_taken = 0;
    const bool live = j < max_jobs && job.count[j] > 0;
    if (live) {
        long long take = sel->want - before;
        take = take < 0 ? 0 : (take > my_eq ? my_eq : take);
        a = floor_units + gt[j] + (int)take;
        a = a < 0 ? 0 : (a > cap ? cap : a);
        ties_taken = take;
    }
    if (j < max_jobs) {
        alloc[j] = a;
        if (out_alloc) out_alloc[j] = a;
        if (live) job.last_alloc[j] = a;
        double R = 0.0;
        if (live && a > 0) {
            Row r;
            load_row(job, fit, j, max_jobs, T, r);
            double run = CUDART_INF;
            for (int n = 1; n <= a; ++n) {
                run = fmin(run, n == 1 ? r.g1 : raw_gain(r.c, n));
                R += run;
            }
        }
        reduction[j] = R;
    }
    __syncthreads();
    sh_pre[t] = ((long long)a << 20) | ties_taken;
    __syncthreads();
    for (int o = kThreads / 2; o > 0; o >>= 1) {
        if (t < o) sh_pre[t] += sh_pre[t + o];
        __syncthreads();
    }
    if (t == 0) {
        atomicAdd((unsigned long long*)&counters[6], (unsigned long long)(sh_pre[0] >> 20));
        atomicAdd((unsigned long long*)&counters[7], (unsigned long long)(sh_pre[0] & ((1ll << 20) - 1)));
    }
}

__global__ void free_init_kernel(SelectState* sel, long long want, unsigned long long* list_len) {
    sel->prefix = want > 0 ? 0ull : ~0ull;
    sel->want = want > 0 ? want : 0;
    sel->done = want > 0 ? 0 : 1;
    *list_len = 0;
}

}  // namespace

// The kernels the table path shares: pick of the first digit and the scan of the block tie sums.
int launch_pick_first(slaq_handle* h);
int launch_scan_blocks(slaq_handle* h, int blocks);

// Predict + allocate without the gain table.  `want` = units beyond the floor among n >= first_unit.
int launch_allocate_free(slaq_handle* h, double T, long long want, int first_unit, int32_t* d_out_alloc) {
    const int J = h->max_jobs, cap = h->max_cores;
    cudaStream_t st = h->stream;
    int launches = 0;
    unsigned long long* list = reinterpret_cast<unsigned long long*>(h->gain);   // the table's memory holds the candidates
    unsigned long long* list_len = reinterpret_cast<unsigned long long*>(h->scratch.counters + 15);
    const long long list_cap = (long long)J * h->cap_alloc;
    const int blocks_jobs = (J + kThreads - 1) / kThreads;
    int grid = h->sm_count * 8;
    if (grid > blocks_jobs) grid = blocks_jobs;
    free_init_kernel<<<1, 1, 0, st>>>(h->scratch.sel, want, list_len);
    free_hist0_kernel<<<grid, kThreads, 0, st>>>(h->job, h->fit, J, cap, T, first_unit, h->scratch.hist);
    launches += 2;
    int k = launch_pick_first(h);
    if (k < 0) return -1;
    launches += k;
    free_candidates_kernel<<<grid, kThreads, 0, st>>>(h->job, h->fit, J, cap, T, first_unit, h->scratch.sel, h->scratch.gt,
                                                     h->scratch.eq, list, list_len, list_cap);
    ++launches;
    const int flat_grid = h->sm_count * 4;
    for (int pass = 1; pass < kRadixPasses; ++pass) {
        free_flat_pass_kernel<<<flat_grid, kThreads, 0, st>>>(list, list_len, pass, h->scratch.hist, h->scratch.sel,
                                                             h->scratch.ticket);
        ++launches;
    }
    free_count_kernel<<<blocks_jobs, kThreads, 0, st>>>(h->job, h->fit, J, cap, T, first_unit, h->scratch.sel,
                                                       h->scratch.gt, h->scratch.eq, h->scratch.block_eq);
    ++launches;
    if ((k = launch_scan_blocks(h, blocks_jobs)) < 0) return -1;
    launches += k;
    free_finalise_kernel<<<blocks_jobs, kThreads, 0, st>>>(h->job, h->fit, J, cap, T, first_unit - 1, h->scratch.sel,
                                                          h->scratch.gt, h->scratch.eq, h->scratch.block_eq, h->alloc,
                                                          h->reduction, d_out_alloc, h->scratch.counters);
    ++launches;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("table-free allocation kernels launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return launches;
}

}  // namespace slaq
