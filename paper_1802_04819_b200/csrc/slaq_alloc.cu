// Allocation: the greedy loop of "Scheduling Based on Quality Improvements" as a global
// top-C selection.
//
// The paper starts every job at one core and then gives one core at a time to the job
// whose next core has the largest predicted gain.  Gain rows are non-increasing in n, so
// that loop hands out exactly the `want` largest gains beyond the floor, and among equal
// gains it serves (job id ascending, n ascending).  Here: a most-significant-digit-first
// radix select over the 64-bit patterns of the gains (all >= +0, so the IEEE pattern
// orders like the value) finds the threshold tau and how many gains equal to tau are
// still wanted - after the first two passes it reads only the short segment of each row
// that still agrees with the threshold's leading digits; then per job  a_j = floor + #{g > tau} + clamp(wanted - P_j, 0, #{g = tau})
// with P_j the number of gains equal to tau in jobs with a lower id.
#include <math_constants.h>

#include "slaq_internal.cuh"

namespace slaq {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kSelectThreads = 256;
constexpr int kJobsPerBlock = 256;   // count / finalise kernels: 8 warps x 32 jobs

__host__ __device__ inline int pass_shift(int pass) {
    return pass < kRadixPasses - 1 ? 64 - kRadixBits * (pass + 1) : 0;
}
__host__ __device__ inline int pass_bits(int pass) {
    return pass < kRadixPasses - 1 ? kRadixBits : 64 - kRadixBits * (kRadixPasses - 1);
}

// After the histogram of `pass` is complete: walk the bins from the top until `want`
// units are covered, extend the threshold prefix by that bin and keep what is still
// wanted inside it.  Called by every thread of one block of kSelectThreads threads;
// sh holds kSelectThreads + 1 entries.
__device__ void pick_bin(const unsigned long long* hist, int pass, SelectState* sel, unsigned long long* sh) {
    const int t = threadIdx.x;
    const int nbins = 1 << pass_bits(pass);
    const int per = (kRadixBins + kSelectThreads - 1) / kSelectThreads;   // bins per thread, from the top down
    unsigned long long mine = 0;
    for (int k = 0; k < per; ++k) {
        const int b = nbins - 1 - (t * per + k);
        if (b >= 0) mine += __ldcg(&hist[b]);
    }
    sh[t] = mine;
    __syncthreads();
    if (t == 0) {   // exclusive prefix over threads
        unsigned long long run = 0;
        for (int i = 0; i < kSelectThreads; ++i) {
            const unsigned long long v = sh[i];
            sh[i] = run;
            run += v;
        }
        sh[kSelectThreads] = run;
    }
    __syncthreads();
    const long long want = sel->want;
    const bool done = sel->done != 0;
    __syncthreads();
    if (done) return;
    unsigned long long above = sh[t];
    for (int k = 0; k < per; ++k) {
        const int b = nbins - 1 - (t * per + k);
        if (b < 0) break;
        const unsigned long long c = __ldcg(&hist[b]);
        if (above < (unsigned long long)want && (unsigned long long)want <= above + c) {
            sel->prefix |= (unsigned long long)b << pass_shift(pass);   // exactly one thread gets here
            sel->want = want - (long long)above;
        }
        above += c;
    }
}

// Rows are non-increasing, so the candidates of a row whose leading digits equal the threshold
// prefix found so far form one contiguous segment [seg_lo, seg_hi) of the row.  Pass p narrows every
// segment by the bin chosen for digit p - 1 (elements with a larger digit lie before it, with a smaller
// one behind it) and histograms digit p over what is left; from the second pass on only the
// segments are read.  The last block to finish picks the bin of digit p.
__global__ void __launch_bounds__(kSelectThreads)
select_pass_kernel(const double* __restrict__ gain, const int32_t* __restrict__ count, int max_jobs, int cap,
                   int first_unit, int pass, unsigned long long* __restrict__ hist_all, SelectState* sel,
                   unsigned int* ticket, int32_t* __restrict__ seg_lo, int32_t* __restrict__ seg_hi, int do_pick,
                   int32_t* err_word) {
    __shared__ unsigned int sh_hist[kRadixBins];
    __shared__ unsigned long long sh_scan[kSelectThreads + 1];
    __shared__ bool is_last;
    unsigned long long* hist = hist_all + (size_t)pass * kRadixBins;
    if (sel->done) return;   // uniform over the grid: nothing is wanted
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    const unsigned long long prefix = sel->prefix;
    const int shift = pass_shift(pass), bits = pass_bits(pass);
    const int prev_shift = pass_shift(pass - 1), prev_bits = pass_bits(pass - 1);
    const unsigned prev_bin = (unsigned)(prefix >> prev_shift) & ((1u << prev_bits) - 1u);
    const unsigned long long* keys = reinterpret_cast<const unsigned long long*>(gain);
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * (kSelectThreads / 32);
    // a warp takes 32 rows at a time: each lane looks up one row's segment, then the warp walks the
    // rows whose segment is not empty (after the second pass most are)
    for (int j0 = (blockIdx.x * (kSelectThreads / 32) + (threadIdx.x >> 5)) * 32; j0 < max_jobs; j0 += warps_total * 32) {
        const int mine = j0 + lane;
        int my_lo = first_unit - 1, my_hi = cap;      // 0-based positions n - 1
        bool live = mine < max_jobs && count[mine] > 0;
        if (live && pass > 1) {
            my_lo = seg_lo[mine];
            my_hi = seg_hi[mine];
#ifdef SLAQ_DEBUG_BOUNDS
            if (my_lo < first_unit - 1 || my_hi > cap || my_lo > my_hi) {   // not a segment of this row: skip it
                if (err_word) atomicOr(err_word, kErrSegment);
                my_lo = my_hi = first_unit - 1;
            }
#endif
        }
        unsigned todo = __ballot_sync(kFull, live && my_lo < my_hi);
        while (todo) {
            const int r = __ffs(todo) - 1;
            todo &= todo - 1;
            const int j = j0 + r;
            const int lo = __shfl_sync(kFull, my_lo, r), hi = __shfl_sync(kFull, my_hi, r);
            int above = 0, same = 0;
            auto take = [&](unsigned long long key, bool in) {
                const unsigned d_prev = (unsigned)(key >> prev_shift) & ((1u << prev_bits) - 1u);
                const bool match = in && d_prev == prev_bin;
                above += __popc(__ballot_sync(kFull, in && d_prev > prev_bin));
                same += __popc(__ballot_sync(kFull, match));
                const unsigned bin = (unsigned)(key >> shift) & ((1u << bits) - 1u);
                if (match && index_ok(bin, kRadixBins, kErrBin, err_word)) atomicAdd(&sh_hist[bin], 1u);
            };
            auto fetch = [&](int i) -> unsigned long long {
                return (i < hi && index_ok((long long)j * cap + i, (long long)max_jobs * cap, kErrGain, err_word))
                           ? keys[(size_t)j * cap + i] : 0ull;
            };
            if (hi - lo <= 128) {
                // a segment of up to four chunks (a whole row of the first table-wide pass): all its loads are
                // issued before the first is used, so that a warp keeps four of them in flight instead of one
                unsigned long long k4[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) k4[c] = fetch(lo + 32 * c + lane);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (lo + 32 * c < hi) take(k4[c], lo + 32 * c + lane < hi);
            } else {
                for (int base = lo; base < hi; base += 32) take(fetch(base + lane), base + lane < hi);
            }
            if (lane == r) {
                my_lo = lo + above;
                my_hi = lo + above + same;
            }
        }
        if (live) {
            seg_lo[mine] = my_lo;
            seg_hi[mine] = my_hi;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) {
        const unsigned v = sh_hist[i];
        if (v) atomicAdd(&hist[i], (unsigned long long)v);
    }
    if (!do_pick) return;   // the histogram is completed elsewhere (summed over GPUs) before the bin is picked
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(&ticket[1 + pass], 1u) == gridDim.x - 1;
    __syncthreads();
    if (is_last) {
        __threadfence();
        pick_bin(hist, pass, sel, sh_scan);
    }
}

// The first histogram is complete when this starts (it was filled by an earlier kernel).
__global__ void __launch_bounds__(kSelectThreads) pick_first_kernel(unsigned long long* hist_all, SelectState* sel) {
    __shared__ unsigned long long sh_scan[kSelectThreads + 1];
    pick_bin(hist_all, 0, sel, sh_scan);
}

// Pick the bin of any pass from a histogram that is complete when the kernel starts.
__global__ void __launch_bounds__(kSelectThreads)
pick_pass_kernel(unsigned long long* hist_all, int pass, SelectState* sel) {
    __shared__ unsigned long long sh_scan[kSelectThreads + 1];
    if (sel->done) return;
    pick_bin(hist_all + (size_t)pass * kRadixBins, pass, sel, sh_scan);
}

__global__ void init_select_kernel(SelectState* sel, long long want) {
    sel->prefix = want > 0 ? 0ull : ~0ull;   // nothing wanted: a threshold above every gain
    sel->want = want > 0 ? want : 0;
    sel->done = want > 0 ? 0 : 1;
}

// Histogram of the first digit when the gain rows were not written by the gain kernel.
__global__ void __launch_bounds__(kSelectThreads)
first_hist_kernel(const double* __restrict__ gain, const int32_t* __restrict__ count, int max_jobs, int cap,
                  int first_unit, unsigned long long* __restrict__ hist0, int32_t* err_word) {
    __shared__ unsigned int sh_hist[kRadixBins];
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    const unsigned long long* keys = reinterpret_cast<const unsigned long long*>(gain);
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * (kSelectThreads / 32);
    for (int j = blockIdx.x * (kSelectThreads / 32) + (threadIdx.x >> 5); j < max_jobs; j += warps_total) {
        if (count[j] <= 0) continue;
        for (int n = first_unit + lane; n <= cap; n += 32)
            if (index_ok((long long)j * cap + (n - 1), (long long)max_jobs * cap, kErrGain, err_word))
                atomicAdd(&sh_hist[(unsigned)(keys[(size_t)j * cap + (n - 1)] >> (64 - kRadixBits))], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadixBins; i += blockDim.x) {
        const unsigned v = sh_hist[i];
        if (v) atomicAdd(&hist0[i], (unsigned long long)v);
    }
}

// Per job: how many candidate gains lie above the threshold and how many equal it.  The segments
// left by the last pass hold the candidates that agree with the threshold in all but the last digit;
// one more narrowing by that digit's bin gives the gains equal to the threshold, and everything in
// front of them is larger.  gt / eq overwrite seg_lo / seg_hi in place.
__global__ void __launch_bounds__(256)
count_kernel(const double* __restrict__ gain, const int32_t* __restrict__ count, int max_jobs, int cap, int first_unit,
             const SelectState* __restrict__ sel, int32_t* __restrict__ gt, int32_t* __restrict__ eq,
             long long* __restrict__ block_eq, int32_t* err_word) {
    __shared__ int sh_eq[8];
    const bool none_wanted = sel->done != 0;
    const unsigned long long tau = sel->prefix;
    constexpr int last = kRadixPasses - 1;
    const unsigned last_bin = (unsigned)(tau >> pass_shift(last)) & ((1u << pass_bits(last)) - 1u);
    const unsigned long long* keys = reinterpret_cast<const unsigned long long*>(gain);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // each lane owns one of the warp's 32 rows; the warp walks the rows whose segment is not empty
    const int mine = blockIdx.x * kJobsPerBlock + warp * 32 + lane;
    const bool live = mine < max_jobs && count[mine] > 0 && !none_wanted;
    int my_lo = 0, my_hi = 0;
    if (live) {
        my_lo = gt[mine];    // segment [lo, hi) written by the last pass
        my_hi = eq[mine];
#ifdef SLAQ_DEBUG_BOUNDS
        if (my_lo < first_unit - 1 || my_hi > cap || my_lo > my_hi) {
            if (err_word) atomicOr(err_word, kErrSegment);
            my_lo = my_hi = first_unit - 1;
        }
#endif
    }
    int my_gt = live ? my_lo - (first_unit - 1) : 0, my_eq = 0;
    unsigned todo = __ballot_sync(kFull, live && my_lo < my_hi);
    while (todo) {
        const int r = __ffs(todo) - 1;
        todo &= todo - 1;
        const int j = blockIdx.x * kJobsPerBlock + warp * 32 + r;
        const int lo = __shfl_sync(kFull, my_lo, r), hi = __shfl_sync(kFull, my_hi, r);
        int above = 0, same = 0;
        for (int base = lo; base < hi; base += 32) {
            const int i = base + lane;
            const bool in = i < hi;
            unsigned long long key = 0;
            if (in && index_ok((long long)j * cap + i, (long long)max_jobs * cap, kErrGain, err_word))
                key = keys[(size_t)j * cap + i];
            const unsigned d = (unsigned)(key >> pass_shift(last)) & ((1u << pass_bits(last)) - 1u);
            above += __popc(__ballot_sync(kFull, in && d > last_bin));
            same += __popc(__ballot_sync(kFull, in && d == last_bin));
        }
        if (lane == r) {
            my_gt += above;
            my_eq = same;
        }
    }
    if (mine < max_jobs) {
        gt[mine] = my_gt;
        eq[mine] = my_eq;
    }
    int eq_sum = my_eq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) eq_sum += __shfl_xor_sync(kFull, eq_sum, o);
    if (lane == 0) sh_eq[warp] = eq_sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long total = 0;
        for (int w = 0; w < 8; ++w) total += sh_eq[w];
        block_eq[blockIdx.x] = total;
    }
}

// Exclusive prefix sum of block_eq[0..n), one block of 1024 threads; block_eq[n] receives the total.
__global__ void __launch_bounds__(1024) scan_blocks_kernel(long long* block_eq, int n) {
    __shared__ long long sh[1024];
    const int t = threadIdx.x;
    const int per = (n + 1023) / 1024;
    const int lo = min(t * per, n), hi = min(lo + per, n);
    long long sum = 0;
    for (int i = lo; i < hi; ++i) sum += block_eq[i];
    sh[t] = sum;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {   // inclusive scan
        const long long v = t >= o ? sh[t - o] : 0;
        __syncthreads();
        sh[t] += v;
        __syncthreads();
    }
    long long run = sh[t] - sum;
    for (int i = lo; i < hi; ++i) {
        const long long v = block_eq[i];
        block_eq[i] = run;
        run += v;
    }
    __syncthreads();
    if (t == 1023) block_eq[n] = sh[1023];
}

// a_j from the counts, the predicted reduction at a_j, and the allocation becomes the job's core count.
__global__ void __launch_bounds__(256)
finalise_kernel(const double* __restrict__ gain, const int32_t* __restrict__ count, int max_jobs, int cap, int floor_units,
                const SelectState* __restrict__ sel, const int32_t* __restrict__ gt, const int32_t* __restrict__ eq,
                const long long* __restrict__ block_prefix, int32_t* __restrict__ alloc, double* __restrict__ reduction,
                int32_t* __restrict__ last_alloc, int32_t* __restrict__ out_alloc, long long* counters,
                long long ties_before, const long long* __restrict__ d_ties_before, int32_t* err_word) {
    __shared__ long long sh_pre[kJobsPerBlock];
    if (d_ties_before) ties_before += *d_ties_before;   // the count held by lower shards, left on the device by the caller
    const int t = threadIdx.x;
    const int j0 = blockIdx.x * kJobsPerBlock;
    const int jt = j0 + t;
    const int my_eq = jt < max_jobs ? eq[jt] : 0;
    sh_pre[t] = my_eq;
    __syncthreads();
    for (int o = 1; o < kJobsPerBlock; o <<= 1) {
        const long long v = t >= o ? sh_pre[t - o] : 0;
        __syncthreads();
        sh_pre[t] += v;
        __syncthreads();
    }
    // ties in jobs with a lower id (ties_before: those held by lower-numbered shards of the same cluster)
    const long long before = ties_before + block_prefix[blockIdx.x] + sh_pre[t] - my_eq;
    int a = 0;
    long long ties_taken = 0;
    if (jt < max_jobs && count[jt] > 0) {
        long long take = sel->want - before;
        take = take < 0 ? 0 : (take > my_eq ? my_eq : take);
        a = floor_units + gt[jt] + (int)take;
        ties_taken = take;
#ifdef SLAQ_DEBUG_BOUNDS
        if (a < 0 || a > cap) {   // an allocation outside 0..cap would read past the row below
            if (err_word) atomicOr(err_word, kErrSegment);
            a = a < 0 ? 0 : cap;
        }
#endif
    }
    if (jt < max_jobs) {
        alloc[jt] = a;
        if (out_alloc) out_alloc[jt] = a;
        if (count[jt] > 0) last_alloc[jt] = a;
    }
    // block totals for the statistics: cores handed out and ties taken, both at most 1024 per job
    __syncthreads();
    sh_pre[t] = ((long long)a << 20) | ties_taken;
    __syncthreads();
    for (int o = kJobsPerBlock / 2; o > 0; o >>= 1) {
        if (t < o) sh_pre[t] += sh_pre[t + o];
        __syncthreads();
    }
    if (t == 0) {
        atomicAdd((unsigned long long*)&counters[6], (unsigned long long)(sh_pre[0] >> 20));
        atomicAdd((unsigned long long*)&counters[7], (unsigned long long)(sh_pre[0] & ((1ll << 20) - 1)));
    }
    // predicted reduction at the allocation: the job's first a_j gains.  Most jobs get a few cores: their own thread
    // adds them in order (all threads of the block load at once); a row with more than 32 is left to its warp.
    const int warp = t >> 5, lane = t & 31;
    const bool mine = jt < max_jobs;
    if (mine && a <= 32) {
        double R = 0.0;
        const double* row = gain + (size_t)jt * cap;
        for (int n = 0; n < a; ++n) R += row[n];
        reduction[jt] = R;
    }
    unsigned big = __ballot_sync(kFull, mine && a > 32);
    while (big) {
        const int r = __ffs(big) - 1;
        big &= big - 1;
        const int j = j0 + warp * 32 + r;
        const int aj = __shfl_sync(kFull, a, r);
        double R = 0.0;
        for (int n = lane; n < aj; n += 32) R += gain[(size_t)j * cap + n];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) R += __shfl_xor_sync(kFull, R, o);
        if (lane == 0) reduction[j] = R;
    }
}

}  // namespace

// Selection + counts + allocation on the gain rows held by the handle.  `want` = units to
// hand out beyond the floor among gains n >= first_unit.  hist0_ready: the first histogram
// was already accumulated (by the gain kernel).
int launch_allocate(slaq_handle* h, long long want, int first_unit, bool hist0_ready, int32_t* d_out_alloc) {
    int launches = 0;
    const int J = h->max_jobs, cap = h->max_cores;
    cudaStream_t st = h->stream;
    int grid = h->sm_count * 8;
    const int needed = (J + (kSelectThreads / 32) - 1) / (kSelectThreads / 32);
    if (grid > needed) grid = needed;
    init_select_kernel<<<1, 1, 0, st>>>(h->scratch.sel, want);
    ++launches;
    if (!hist0_ready) {
        first_hist_kernel<<<grid, kSelectThreads, 0, st>>>(h->gain, h->job.count, J, cap, first_unit, h->scratch.hist,
                                                          h->err_word);
        ++launches;
    }
    pick_first_kernel<<<1, kSelectThreads, 0, st>>>(h->scratch.hist, h->scratch.sel);
    ++launches;
    for (int pass = 1; pass < kRadixPasses; ++pass) {
        select_pass_kernel<<<grid, kSelectThreads, 0, st>>>(h->gain, h->job.count, J, cap, first_unit, pass,
                                                           h->scratch.hist, h->scratch.sel, h->scratch.ticket,
                                                           h->scratch.gt, h->scratch.eq, 1, h->err_word);
        ++launches;
    }
    const int blocks = (J + kJobsPerBlock - 1) / kJobsPerBlock;
    count_kernel<<<blocks, 256, 0, st>>>(h->gain, h->job.count, J, cap, first_unit, h->scratch.sel, h->scratch.gt,
                                         h->scratch.eq, h->scratch.block_eq, h->err_word);
    scan_blocks_kernel<<<1, 1024, 0, st>>>(h->scratch.block_eq, blocks);
    finalise_kernel<<<blocks, 256, 0, st>>>(h->gain, h->job.count, J, cap, first_unit - 1, h->scratch.sel, h->scratch.gt,
                                            h->scratch.eq, h->scratch.block_eq, h->alloc, h->reduction,
                                            h->job.last_alloc, d_out_alloc, h->scratch.counters, 0, nullptr, h->err_word);
    launches += 3;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("allocation kernels launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return launches;
}

// The two small steps the table-free selection (slaq_select_free.cu) shares with this file.
int launch_pick_first(slaq_handle* h) {
    pick_first_kernel<<<1, kSelectThreads, 0, h->stream>>>(h->scratch.hist, h->scratch.sel);
    return 1;
}
int launch_scan_blocks(slaq_handle* h, int blocks) {
    scan_blocks_kernel<<<1, 1024, 0, h->stream>>>(h->scratch.block_eq, blocks);
    return 1;
}

// ---- one cluster sharded over several GPUs: the same kernels, driven step by step so that the
// histograms can be summed over the shards between the steps ----

static int check_launch(slaq_handle* h, const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return 0;
    h->err = std::string(what) + ": " + cudaGetErrorString(e);
    return -1;
}

// Pick the bin of `pass` from its (summed) histogram; pass 0 first sets what is wanted over all shards.
int launch_shard_pick(slaq_handle* h, int pass, long long want) {
    int launches = 0;
    if (pass == 0) {
        init_select_kernel<<<1, 1, 0, h->stream>>>(h->scratch.sel, want);
        ++launches;
    }
    pick_pass_kernel<<<1, kSelectThreads, 0, h->stream>>>(h->scratch.hist, pass, h->scratch.sel);
    ++launches;
    return check_launch(h, "shard pick") ? -1 : launches;
}

// Narrow this shard's segments by the bin of digit pass - 1 and histogram digit `pass` locally.
int launch_shard_pass(slaq_handle* h, int pass, int first_unit) {
    const int J = h->max_jobs;
    int grid = h->sm_count * 8;
    const int needed = (J + (kSelectThreads / 32) - 1) / (kSelectThreads / 32);
    if (grid > needed) grid = needed;
    select_pass_kernel<<<grid, kSelectThreads, 0, h->stream>>>(h->gain, h->job.count, J, h->max_cores, first_unit, pass,
                                                              h->scratch.hist, h->scratch.sel, h->scratch.ticket,
                                                              h->scratch.gt, h->scratch.eq, 0, h->err_word);
    return check_launch(h, "shard pass") ? -1 : 1;
}

// Per-job counts of this shard; *d_total points at the shard's number of gains equal to the threshold.
int launch_shard_count(slaq_handle* h, int first_unit, const long long** d_total) {
    const int J = h->max_jobs;
    const int blocks = (J + kJobsPerBlock - 1) / kJobsPerBlock;
    count_kernel<<<blocks, 256, 0, h->stream>>>(h->gain, h->job.count, J, h->max_cores, first_unit, h->scratch.sel,
                                                h->scratch.gt, h->scratch.eq, h->scratch.block_eq, h->err_word);
    scan_blocks_kernel<<<1, 1024, 0, h->stream>>>(h->scratch.block_eq, blocks);
    *d_total = h->scratch.block_eq + blocks;
    return check_launch(h, "shard count") ? -1 : 2;
}

int launch_shard_finalise(slaq_handle* h, int first_unit, long long ties_before, const long long* d_ties_before,
                          int32_t* d_out_alloc) {
    const int J = h->max_jobs;
    const int blocks = (J + kJobsPerBlock - 1) / kJobsPerBlock;
    finalise_kernel<<<blocks, 256, 0, h->stream>>>(h->gain, h->job.count, J, h->max_cores, first_unit - 1, h->scratch.sel,
                                                   h->scratch.gt, h->scratch.eq, h->scratch.block_eq, h->alloc,
                                                   h->reduction, h->job.last_alloc, d_out_alloc, h->scratch.counters,
                                                   ties_before, d_ties_before, h->err_word);
    return check_launch(h, "shard finalise") ? -1 : 1;
}

// ---------------------------------------------------------------------------------
// Allocation without any device allocation: the same kernels, their scratch in a static
// device array that ships with the library image.
// ---------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxJobs = 32768;
constexpr int kStaticBlocks = kStaticMaxJobs / kJobsPerBlock;

// Everything the selection and the per-job counts write besides the caller's outputs.
struct StaticScratch {
    unsigned long long hist[kRadixPasses * kRadixBins];   // cleared every call
    unsigned int ticket[8];                               // cleared every call
    SelectState sel;                                      // rewritten every call
    long long counters[16];                               // cleared every call
    long long block_eq[kStaticBlocks + 2];                // fully rewritten before it is read
    int32_t gt[kStaticMaxJobs];                           // fully rewritten before it is read
    int32_t eq[kStaticMaxJobs];
    int32_t every_row_active[kStaticMaxJobs];             // set to 1 every call
    int32_t cores_now[kStaticMaxJobs];                    // sink for the "current core count" the kernels keep
};

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

__global__ void fill_ones_kernel(int32_t* v, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) v[i] = 1;
}

// Device address of g_static_scratch on the current device, looked up once per device.
// In host code the array's name only stands for the symbol; kernels need this address.
int static_scratch_for_current_device(StaticScratch** out) {
    constexpr int kMaxDevices = 64;
    static StaticScratch* cache[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SLAQ_E_CUDA;
    StaticScratch* p = __atomic_load_n(&cache[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return SLAQ_E_CUDA;
        p = static_cast<StaticScratch*>(addr);
        __atomic_store_n(&cache[dev], p, __ATOMIC_RELEASE);   // every thread finds the same address
    }
    *out = p;
    return SLAQ_OK;
}

}  // namespace

}  // namespace slaq

extern "C" int slaq_allocate_static(const double* d_gain, int32_t n_jobs, int32_t max_cores_per_job,
                                    int64_t total_cores, int32_t* d_out_alloc, double* d_out_reduction,
                                    void* cuda_stream) {
    using namespace slaq;
    if (!d_gain || !d_out_alloc || !d_out_reduction || n_jobs < 1 || max_cores_per_job < 1 || total_cores < 0)
        return SLAQ_E_ARG;
    if (n_jobs > kStaticMaxJobs || max_cores_per_job > kMaxCoresLimit) return SLAQ_E_RANGE;
    StaticScratch* sc = nullptr;
    const int rc = static_scratch_for_current_device(&sc);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int J = n_jobs, cap = max_cores_per_job;
    const int floor_units = total_cores >= J ? 1 : 0, first_unit = floor_units + 1;
    const long long usable = total_cores < (long long)J * cap ? total_cores : (long long)J * cap;
    const long long want = usable - (long long)J * floor_units;

    // the array keeps the previous call's contents: clear what the kernels accumulate into
    if (cudaMemsetAsync(sc->hist, 0, sizeof sc->hist, st) != cudaSuccess) return SLAQ_E_CUDA;
    if (cudaMemsetAsync(sc->ticket, 0, sizeof sc->ticket, st) != cudaSuccess) return SLAQ_E_CUDA;
    if (cudaMemsetAsync(sc->counters, 0, sizeof sc->counters, st) != cudaSuccess) return SLAQ_E_CUDA;
    fill_ones_kernel<<<(J + 255) / 256, 256, 0, st>>>(sc->every_row_active, J);
    init_select_kernel<<<1, 1, 0, st>>>(&sc->sel, want);

    int sm_count = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    int grid = sm_count * 8;
    const int needed = (J + (kSelectThreads / 32) - 1) / (kSelectThreads / 32);
    if (grid > needed) grid = needed;
    first_hist_kernel<<<grid, kSelectThreads, 0, st>>>(d_gain, sc->every_row_active, J, cap, first_unit, sc->hist, nullptr);
    pick_first_kernel<<<1, kSelectThreads, 0, st>>>(sc->hist, &sc->sel);
    for (int pass = 1; pass < kRadixPasses; ++pass)
        select_pass_kernel<<<grid, kSelectThreads, 0, st>>>(d_gain, sc->every_row_active, J, cap, first_unit, pass,
                                                           sc->hist, &sc->sel, sc->ticket, sc->gt, sc->eq, 1, nullptr);
    const int blocks = (J + kJobsPerBlock - 1) / kJobsPerBlock;
    count_kernel<<<blocks, 256, 0, st>>>(d_gain, sc->every_row_active, J, cap, first_unit, &sc->sel, sc->gt, sc->eq,
                                         sc->block_eq, nullptr);
    scan_blocks_kernel<<<1, 1024, 0, st>>>(sc->block_eq, blocks);
    finalise_kernel<<<blocks, 256, 0, st>>>(d_gain, sc->every_row_active, J, cap, floor_units, &sc->sel, sc->gt, sc->eq,
                                            sc->block_eq, d_out_alloc, d_out_reduction, sc->cores_now, nullptr,
                                            sc->counters, 0, nullptr, nullptr);
    if (cudaGetLastError() != cudaSuccess) return SLAQ_E_CUDA;
    if (total_cores < J) return SLAQ_W_OVERSUBSCRIBED;
    if (total_cores > (long long)J * cap) return SLAQ_W_UNDERFILLED;
    return SLAQ_OK;
}
