// C ABI of the library: handle, state updates (append / bulk load / time law / removal),
// the scheduling epoch, and read-back of results.  The contract is in include/slaq.h.
#include <math_constants.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "slaq_internal.cuh"

using namespace slaq;

namespace {

constexpr size_t kAlign = 256;

struct Bump {
    char* base;
    size_t off = 0;
    template <class T>
    T* take(size_t n) {
        off = (off + kAlign - 1) / kAlign * kAlign;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

// Lay every device array out inside one workspace; with base == nullptr only the size is computed.
size_t layout(slaq_handle* h, char* base, int32_t J, int32_t Hmax, int32_t cap) {
    Bump b{base};
    const size_t Js = (size_t)J;
    double* ring = b.take<double>(Js * Hmax);
    double* wtab = b.take<double>(Hmax);
    JobArrays job;
    job.row = b.take<double*>(Js);
    job.cap = b.take<int32_t>(Js);
    job.head = b.take<int32_t>(Js);
    job.count = b.take<int32_t>(Js);
    job.k_last = b.take<int64_t>(Js);
    job.m_seen = b.take<double>(Js);
    job.tm = b.take<double>(8 * Js);
    job.s_set = b.take<double>(Js);
    job.w_set = b.take<double>(Js);
    job.last_alloc = b.take<int32_t>(Js);
    job.target = b.take<double>(Js);
    FitArrays fit;
    fit.status = b.take<int32_t>(Js);
    fit.family = b.take<int8_t>(Js);
    fit.params = b.take<double>(4 * Js);
    fit.residual = b.take<double>(2 * Js);
    fit.sweeps = b.take<int32_t>(2 * Js);
    fit.largest = b.take<double>(Js);
    fit.span = b.take<double>(Js);
    fit.both = b.take<double>(8 * Js);
    fit.mask = b.take<uint8_t>(Js);
    fit.k_fit = b.take<int64_t>(Js);
    fit.warm_p = b.take<double>(8 * Js);
    fit.warm_mask = b.take<uint8_t>(Js);
    fit.warm_k = b.take<int64_t>(Js);
    fit.warm_span = b.take<double>(Js);
    fit.warm_scale = b.take<double>(Js);
    Scratch sc;
    sc.hist = b.take<unsigned long long>((size_t)kRadixPasses * kRadixBins);
    const size_t zero_from = b.off - sizeof(unsigned long long) * (size_t)kRadixPasses * kRadixBins;
    sc.ticket = b.take<unsigned int>(kTickets);
    sc.sel = b.take<SelectState>(1);
    sc.counters = b.take<long long>(16);
    sc.bucket = b.take<int32_t>((size_t)Hmax + 1);
    sc.zero_bytes = b.off - zero_from;
    sc.gt = b.take<int32_t>(Js);
    sc.eq = b.take<int32_t>(Js);
    sc.block_eq = b.take<long long>(Js / 256 + 2);
    sc.order = b.take<int32_t>(Js);
    sc.start = b.take<int32_t>((size_t)Hmax + 1);
    sc.cursor = b.take<int32_t>((size_t)Hmax + 1);
    Staging st;
    st.ids = b.take<int32_t>(Js);
    st.losses = b.take<double>(Js);
    st.times = b.take<double>(Js);
    st.cores = b.take<int32_t>(Js);
    st.offsets = b.take<int64_t>(Js + 1);
    st.k_last = b.take<int64_t>(Js);
    st.m_seen = b.take<double>(Js);
    double* gain = b.take<double>(Js * cap);
    int32_t* alloc = b.take<int32_t>(Js);
    double* reduction = b.take<double>(Js);
    int32_t* err_word = b.take<int32_t>(4);
    job.max_jobs = J;
    job.ring_lo = ring;
    job.ring_hi = ring ? ring + Js * Hmax : nullptr;
    job.packed_lo = job.packed_hi = nullptr;
    job.err_word = err_word;
    if (h && base) {
        h->ring_pool = ring;
        h->wtab = wtab;
        h->job = job;
        h->fit = fit;
        h->scratch = sc;
        h->stage = st;
        h->gain = gain;
        h->alloc = alloc;
        h->reduction = reduction;
        h->err_word = err_word;
    }
    return (b.off + kAlign - 1) / kAlign * kAlign;
}

int fail(slaq_handle* h, int code, const std::string& msg) {
    if (h) h->err = msg;
    return code;
}

int cuda_fail(slaq_handle* h, cudaError_t e, const char* what) {
    return fail(h, SLAQ_E_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define CK(call, what)                                            \
    do {                                                          \
        const cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(h, e_, what);     \
    } while (0)

// (Re)initialise jobs: all of them (ids == nullptr) or the listed ones.
__global__ void init_jobs_kernel(JobArrays job, FitArrays fit, double* ring, int max_jobs, int max_hist,
                                 const int32_t* ids, int n, int32_t* alloc, double* reduction) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int j = ids ? ids[i] : i;
    if (j < 0 || j >= max_jobs) return;
    job.row[j] = ring + (size_t)j * max_hist;
    job.cap[j] = max_hist;
    job.head[j] = 0;
    job.count[j] = 0;
    job.k_last[j] = -1;
    job.m_seen[j] = -CUDART_INF;
    const size_t J = (size_t)max_jobs;
    for (int k = 0; k < 6; ++k) job.tm[k * J + j] = 0.0;
    job.tm[6 * J + j] = CUDART_INF;
    job.tm[7 * J + j] = -CUDART_INF;
    job.s_set[j] = CUDART_NAN;
    job.w_set[j] = CUDART_NAN;
    job.last_alloc[j] = 1;
    job.target[j] = CUDART_NAN;
    fit.status[j] = SLAQ_JOB_INACTIVE;
    fit.family[j] = -1;
    for (int k = 0; k < 4; ++k) fit.params[4 * (size_t)j + k] = CUDART_NAN;
    fit.residual[2 * (size_t)j] = fit.residual[2 * (size_t)j + 1] = CUDART_INF;
    fit.sweeps[2 * (size_t)j] = fit.sweeps[2 * (size_t)j + 1] = 0;
    fit.largest[j] = CUDART_NAN;
    fit.span[j] = 1.0;
    fit.mask[j] = 0;
    fit.warm_mask[j] = 0;
    alloc[j] = 0;
    reduction[j] = 0.0;
}

// One new iteration per listed job: ring write, iteration index, largest reduction seen,
// and the sums of the iteration-time law (booked at the given or the current core count).
// checked: the arrays come straight from the caller's device memory, unseen by the host - an id out of range,
// a job without any loss yet, a loss or time that is not finite or a core count below 1 sets kErrInput and
// that entry is skipped.
__global__ void append_kernel(JobArrays job, FitArrays fit, int max_jobs, int n, const int32_t* ids,
                              const double* losses, const double* times, const int32_t* cores, int checked) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int j = ids[i];
    if (j < 0 || j >= max_jobs) {
        if (checked) atomicOr(job.err_word, kErrInput);
        return;
    }
    const double loss = losses[i];
    if (checked) {
        const bool bad = !(fabs(loss) <= 1.7976931348623157e308) || job.count[j] <= 0 ||
                         (times && !(fabs(times[i]) <= 1.7976931348623157e308)) || (times && cores && cores[i] < 1);
        if (bad) {
            atomicOr(job.err_word, kErrInput);
            return;
        }
    }
    double* row = job.row[j];
    const int cap = job.cap[j];
    int head = job.head[j];
    const int count = job.count[j];
#ifdef SLAQ_DEBUG_BOUNDS
    {   // the ring lies inside one of the pools and the write position inside the ring
        const bool in_ring = row >= job.ring_lo && row + cap <= job.ring_hi;
        const bool in_packed = job.packed_lo && row >= job.packed_lo && row + cap <= job.packed_hi;
        if (!(in_ring || in_packed) || head < 0 || head >= cap || count < 0 || count > cap) {
            atomicOr(job.err_word, kErrStorage);
            return;
        }
    }
#endif
    if (count > 0) {
        const double prev = row[head == 0 ? cap - 1 : head - 1];
        const double seen = job.m_seen[j], drop = prev - loss;
        job.m_seen[j] = drop > seen ? drop : seen;
    }
    row[head] = loss;
    head = head + 1 == cap ? 0 : head + 1;
    job.head[j] = head;
    job.count[j] = count < cap ? count + 1 : cap;
    job.k_last[j] += 1;
    // the history changes: what the last epoch fitted becomes the next fit's starting point
    const uint8_t fitted = fit.mask[j];
    fit.warm_mask[j] = fitted;
    if (fitted) {
        for (int k = 0; k < 8; ++k) fit.warm_p[8 * (size_t)j + k] = fit.both[8 * (size_t)j + k];
        fit.warm_k[j] = fit.k_fit[j];
        fit.warm_span[j] = fit.span[j];
        fit.warm_scale[j] = fit.largest[j];
    }
    if (times) {
        int nc = cores ? cores[i] : job.last_alloc[j];
        if (nc < 1) nc = 1;
        const double t = times[i], nn = (double)nc, u = __ddiv_rn(1.0, nn);
        const size_t J = (size_t)max_jobs;
        double* tm = job.tm + j;
        tm[0] = __dadd_rn(tm[0], 1.0);
        tm[J] = __dadd_rn(tm[J], u);
        tm[2 * J] = __dadd_rn(tm[2 * J], __dmul_rn(u, u));
        tm[3 * J] = __dadd_rn(tm[3 * J], t);
        tm[4 * J] = __dadd_rn(tm[4 * J], __dmul_rn(u, t));
        tm[5 * J] = __dadd_rn(tm[5 * J], __dmul_rn(t, nn));
        tm[6 * J] = fmin(tm[6 * J], u);
        tm[7 * J] = fmax(tm[7 * J], u);
    }
}

// Bulk load: one warp per listed job copies (ring mode) or adopts (packed mode) its row.
__global__ void load_kernel(JobArrays job, FitArrays fit, double* ring, int max_jobs, int max_hist, int n,
                            const int32_t* ids,
                            const int64_t* offsets, const double* src, const int64_t* k_last, const double* m_seen,
                            int packed) {
    const int slot = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (slot >= n) return;
    const int j = ids[slot];
    if (j < 0 || j >= max_jobs) return;
    const int64_t lo = offsets[slot], hi = offsets[slot + 1];
    int64_t H = hi - lo;
    if (H > max_hist) H = max_hist;   // keep the newest points
    const double* from = src + (hi - H);
    double* row = ring + (size_t)j * max_hist;
    int cap = max_hist;
    if (packed && H > 0) {
        row = const_cast<double*>(from);
        cap = (int)H;
    } else {
        for (int i = lane; i < H; i += 32)
            if (index_ok((row - job.ring_lo) + i, job.ring_hi - job.ring_lo, kErrStorage, job.err_word)) row[i] = from[i];
    }
    if (lane == 0) {
        job.row[j] = row;
        job.cap[j] = cap;
        job.head[j] = (int)(H % cap);
        job.count[j] = (int)H;
        job.k_last[j] = H > 0 ? k_last[slot] : -1;
        job.m_seen[j] = m_seen ? m_seen[slot] : -CUDART_INF;
        fit.mask[j] = 0;        // a replaced history has no earlier fit to start from
        fit.warm_mask[j] = 0;
    }
}

// Export: one warp per job copies its window, oldest point first, to out[offsets[j] ..].
__global__ void export_windows_kernel(JobArrays job, int max_jobs, const int64_t* offsets, double* out) {
    const int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (j >= max_jobs) return;
    const int H = job.count[j], cap = job.cap[j];
    if (H <= 0 || H > cap) return;
    const double* row = job.row[j];
    int oldest = job.head[j] - H;
    if (oldest < 0) oldest += cap;
    const int64_t base = offsets[j];
    for (int i = lane; i < H; i += 32) {
        int pos = oldest + i;
        pos -= pos >= cap ? cap : 0;
        if (index_ok(pos, cap, kErrStorage, job.err_word)) out[base + i] = row[pos];
    }
}

__global__ void set_time_kernel(JobArrays job, int max_jobs, int n, const int32_t* ids, const double* s,
                                const double* w) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int j = ids[i];
    if (j < 0 || j >= max_jobs) return;
    job.s_set[j] = s[i];
    job.w_set[j] = w[i];
}

__global__ void set_target_kernel(JobArrays job, int max_jobs, int n, const int32_t* ids, const double* targets) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int j = ids[i];
    if (j < 0 || j >= max_jobs) return;
    job.target[j] = targets[i];
}

// Kernels and copies go to the current device: it must be the one the handle lives on.
int check_device(slaq_handle* h) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(h, SLAQ_E_CUDA, "cudaGetDevice failed");
    if (dev != h->device) return fail(h, SLAQ_E_ARG, "the handle was created on another device than the current one");
    return SLAQ_OK;
}

int check_ids(slaq_handle* h, int32_t n, const int32_t* ids, bool forbid_dups) {
    if (const int rc = check_device(h)) return rc;
    if (n < 0) return fail(h, SLAQ_E_ARG, "negative count");
    if (n > 0 && !ids) return fail(h, SLAQ_E_ARG, "job_ids is null");
    if (n > h->max_jobs) return fail(h, SLAQ_E_ARG, "more entries than job ids");
    if (++h->stamp_epoch == 0) {
        std::fill(h->stamp.begin(), h->stamp.end(), 0u);
        h->stamp_epoch = 1;
    }
    for (int32_t i = 0; i < n; ++i) {
        const int32_t j = ids[i];
        if (j < 0 || j >= h->max_jobs) return fail(h, SLAQ_E_RANGE, "job id outside 0..max_jobs-1");
        if (forbid_dups) {
            if (h->stamp[j] == h->stamp_epoch) return fail(h, SLAQ_E_ARG, "a job id is listed twice in one call");
            h->stamp[j] = h->stamp_epoch;
        }
    }
    return SLAQ_OK;
}

int ensure_weights(slaq_handle* h) {
    if (h->wtab_gamma == h->gamma) return SLAQ_OK;
    std::vector<double> tab((size_t)h->max_hist);
    for (int m = 0; m < h->max_hist; ++m) tab[m] = std::pow(h->gamma, (double)m);
    CK(cudaMemcpyAsync(h->wtab, tab.data(), tab.size() * sizeof(double), cudaMemcpyHostToDevice, h->stream),
       "upload weight table");
    CK(cudaStreamSynchronize(h->stream), "upload weight table");
    h->wtab_gamma = h->gamma;
    return SLAQ_OK;
}

int check_device_errors(slaq_handle* h) {
    int32_t word = 0;
    CK(cudaMemcpyAsync(&word, h->err_word, sizeof word, cudaMemcpyDeviceToHost, h->stream), "read error word");
    CK(cudaStreamSynchronize(h->stream), "read error word");
    if (word != 0) {
        std::string what = "a kernel found an inconsistency:";
        if (word & kErrWindow) what += " a window longer than its ring;";
        if (word & kErrStorage) what += " a position outside a job's storage;";
        if (word & kErrShared) what += " an offset outside a shared-memory slice;";
        if (word & kErrGain) what += " an entry outside the gain table;";
        if (word & kErrSegment) what += " a candidate segment outside its row;";
        if (word & kErrBin) what += " a histogram bin out of range;";
        if (word & kErrJob) what += " a job id out of range;";
        if (word & kErrInput) what += " slaq_append_losses_device was given an id out of range, a job without losses, a value that is not finite or a core count below 1 (those entries were skipped);";
        cudaMemsetAsync(h->err_word, 0, sizeof word, h->stream);   // reported once: the next epoch starts clean
        return fail(h, SLAQ_E_CUDA, what);
    }
    return SLAQ_OK;
}

// Device scratch for calls that move caller data of a size unknown at creation (a bulk load into
// rings, the normalisation export): owned by the handle, grown when a call needs more, kept for
// the next call, released by slaq_destroy.  The stream must be idle when it grows.
int ensure_call_buffer(slaq_handle* h, size_t bytes, void** out) {
    if (bytes > h->call_buf_bytes) {
        CK(cudaStreamSynchronize(h->stream), "sync before growing the call buffer");
        if (h->call_buf) cudaFree(h->call_buf);
        h->call_buf = nullptr;
        h->call_buf_bytes = 0;
        const size_t want = (bytes + kAlign - 1) / kAlign * kAlign;
        const cudaError_t e = cudaMalloc(&h->call_buf, want);
        if (e != cudaSuccess) {
            h->call_buf = nullptr;
            return fail(h, SLAQ_E_NOMEM, std::string("cudaMalloc of the call buffer: ") + cudaGetErrorString(e));
        }
        h->call_buf_bytes = want;
    }
    *out = h->call_buf;
    return SLAQ_OK;
}

int create_common(slaq_handle* h, int32_t max_jobs, int32_t max_hist, int32_t cap, void* ws, size_t bytes) {
    h->max_jobs = max_jobs;
    h->max_hist = max_hist;
    h->cap_alloc = cap;
    h->max_cores = cap;
    CK(cudaGetDevice(&h->device), "cudaGetDevice");
    cudaDeviceProp prop;
    CK(cudaGetDeviceProperties(&prop, h->device), "cudaGetDeviceProperties");
    h->sm_count = prop.multiProcessorCount;
    const size_t need = layout(nullptr, nullptr, max_jobs, max_hist, cap);
    if (ws) {
        if (bytes < need) return fail(h, SLAQ_E_NOMEM, "workspace smaller than slaq_workspace_bytes()");
        if (reinterpret_cast<uintptr_t>(ws) % kAlign) return fail(h, SLAQ_E_ARG, "workspace is not 256-byte aligned");
        h->ws = ws;
        h->owns_ws = false;
    } else {
        const cudaError_t e = cudaMalloc(&h->ws, need);
        if (e != cudaSuccess) {
            h->ws = nullptr;
            return fail(h, SLAQ_E_NOMEM, std::string("cudaMalloc of the workspace: ") + cudaGetErrorString(e));
        }
        h->owns_ws = true;
    }
    h->ws_bytes = need;
    layout(h, static_cast<char*>(h->ws), max_jobs, max_hist, cap);
    h->active.assign((size_t)max_jobs, 0);
    h->stamp.assign((size_t)max_jobs, 0u);
    h->in_packed.assign((size_t)max_jobs, 0);
    h->hinted.assign((size_t)max_jobs, 0);
    for (auto& ev : h->ev) CK(cudaEventCreate(&ev), "cudaEventCreate");
    CK(cudaMemsetAsync(h->scratch.hist, 0, h->scratch.zero_bytes, h->stream), "clear scratch");
    CK(cudaMemsetAsync(h->err_word, 0, 16, h->stream), "clear error word");
    const int threads = 256;
    init_jobs_kernel<<<(max_jobs + threads - 1) / threads, threads, 0, h->stream>>>(
        h->job, h->fit, h->ring_pool, max_jobs, max_hist, nullptr, max_jobs, h->alloc, h->reduction);
    CK(cudaGetLastError(), "init kernel");
    CK(cudaStreamSynchronize(h->stream), "init kernel");
    return SLAQ_OK;
}

bool sizes_ok(int32_t max_jobs, int32_t max_hist, int32_t cap) {
    return max_jobs >= 1 && max_hist >= 4 && max_hist <= kMaxHistLimit && cap >= 1 && cap <= kMaxCoresLimit;
}

int do_append(slaq_handle* h, int32_t n, const int32_t* ids, const double* losses, const double* times,
              const int32_t* cores) {
    if (!h) return SLAQ_E_ARG;
    if (n > 0 && !losses) return fail(h, SLAQ_E_ARG, "losses is null");
    if (const int dc = check_device(h)) return dc;
    if (n < 0) return fail(h, SLAQ_E_ARG, "negative count");
    if (n > 0 && !ids) return fail(h, SLAQ_E_ARG, "job_ids is null");
    if (n > h->max_jobs) return fail(h, SLAQ_E_ARG, "more entries than job ids");
    cudaStream_t st = h->stream;
    // The copies into the staging arrays go first: from pinned memory they run while the host
    // checks the arguments below.  Nothing reads the staging arrays unless the checks pass.
    if (n > 0) {
        CK(cudaMemcpyAsync(h->stage.ids, ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st), "copy job ids");
        CK(cudaMemcpyAsync(h->stage.losses, losses, sizeof(double) * n, cudaMemcpyHostToDevice, st), "copy losses");
        if (times)
            CK(cudaMemcpyAsync(h->stage.times, times, sizeof(double) * n, cudaMemcpyHostToDevice, st), "copy times");
        if (times && cores)
            CK(cudaMemcpyAsync(h->stage.cores, cores, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st), "copy cores");
    }
    int bad = check_ids(h, n, ids, true);
    for (int32_t i = 0; i < n && !bad; ++i) {
        if (!std::isfinite(losses[i])) bad = fail(h, SLAQ_E_NONFINITE, "a loss is not finite");
        else if (times && !std::isfinite(times[i])) bad = fail(h, SLAQ_E_NONFINITE, "an iteration time is not finite");
        else if (cores && cores[i] < 1) bad = fail(h, SLAQ_E_ARG, "cores_used must be at least 1");
    }
    if (bad) {
        cudaStreamSynchronize(st);   // the caller's buffers are free again; the state is untouched
        return bad;
    }
    if (n == 0) return SLAQ_OK;
    const int threads = 256;
    append_kernel<<<(n + threads - 1) / threads, threads, 0, st>>>(
        h->job, h->fit, h->max_jobs, n, h->stage.ids, h->stage.losses, times ? h->stage.times : nullptr,
        (times && cores) ? h->stage.cores : nullptr, 0);
    CK(cudaGetLastError(), "append kernel");
    CK(cudaStreamSynchronize(st), "append");   // the caller may reuse its buffers
    if (h->n_active < h->max_jobs) {   // nothing to do once every id is active
        for (int32_t i = 0; i < n; ++i) {
            if (!h->active[ids[i]]) {
                h->active[ids[i]] = 1;
                h->n_active += 1;
            }
        }
    }
    return SLAQ_OK;
}

int do_load(slaq_handle* h, int32_t n, const int32_t* ids, const int64_t* offsets, const double* losses,
            const int64_t* k_last, const double* m_seen, bool packed) {
    if (!h) return SLAQ_E_ARG;
    if (n > 0 && (!offsets || !losses || !k_last)) return fail(h, SLAQ_E_ARG, "offsets, losses or k_last is null");
    const int rc = check_ids(h, n, ids, true);
    if (rc) return rc;
    if (n == 0) return SLAQ_OK;
    if (offsets[0] < 0) return fail(h, SLAQ_E_ARG, "offsets must start at or above 0");
    for (int32_t i = 0; i < n; ++i)
        if (offsets[i + 1] < offsets[i]) return fail(h, SLAQ_E_ARG, "offsets must not decrease");
    const int64_t lo = offsets[0], total = offsets[n] - lo;
    for (int64_t i = 0; i < total; ++i)
        if (!std::isfinite(losses[lo + i])) return fail(h, SLAQ_E_NONFINITE, "a loss is not finite");
    if (m_seen)
        for (int32_t i = 0; i < n; ++i)
            if (std::isnan(m_seen[i]) || m_seen[i] == INFINITY)
                return fail(h, SLAQ_E_NONFINITE, "m_seen must be a number below +infinity");
    cudaStream_t st = h->stream;
    double* d_src = nullptr;
    double* old_pool = nullptr;
    if (packed) {
        // The new pool is allocated before anything changes, so a failed allocation leaves the handle
        // as it was.  Jobs of the old pool that are listed again are re-pointed by the load kernel and
        // keep their time sums, time law and core count; those that are not listed lose their
        // storage with the old pool and are reset to inactive.
        double* new_pool = nullptr;
        if (total > 0) {
            const cudaError_t e = cudaMalloc(&new_pool, sizeof(double) * (size_t)total);
            if (e != cudaSuccess)
                return fail(h, SLAQ_E_NOMEM, std::string("cudaMalloc of the packed pool: ") + cudaGetErrorString(e));
        }
        if (h->packed_pool) {
            std::vector<int32_t> gone;
            for (int32_t j = 0; j < h->max_jobs; ++j)
                if (h->in_packed[j] && h->stamp[j] != h->stamp_epoch) gone.push_back(j);   // check_ids stamped the listed ids
            const int32_t m = (int32_t)gone.size();
            if (m > 0) {
                cudaError_t e = cudaMemcpyAsync(h->stage.ids, gone.data(), sizeof(int32_t) * m, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess) {
                    init_jobs_kernel<<<(m + 255) / 256, 256, 0, st>>>(h->job, h->fit, h->ring_pool, h->max_jobs,
                                                                      h->max_hist, h->stage.ids, m, h->alloc, h->reduction);
                    e = cudaGetLastError();
                }
                if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // `gone` is read by the copy until here
                if (e != cudaSuccess) {
                    cudaFree(new_pool);
                    return cuda_fail(h, e, "release jobs of the earlier packed load");
                }
                for (int32_t j : gone) {
                    h->in_packed[j] = 0;
                    if (h->hinted[j]) {
                        h->hinted[j] = 0;
                        h->n_hinted -= 1;
                    }
                    if (h->active[j]) {
                        h->active[j] = 0;
                        h->n_active -= 1;
                    }
                }
            }
            old_pool = h->packed_pool;   // still referenced by the re-listed jobs until the load kernel has run
        }
        h->packed_pool = new_pool;
        h->packed_len = (size_t)total;
        h->job.packed_lo = new_pool;
        h->job.packed_hi = new_pool ? new_pool + total : nullptr;
        d_src = new_pool;
    } else if (total > 0) {
        void* buf = nullptr;
        if (const int rc_buf = ensure_call_buffer(h, sizeof(double) * (size_t)total, &buf)) return rc_buf;
        d_src = static_cast<double*>(buf);
    }
    int status = SLAQ_OK;
    {
        cudaError_t e = cudaSuccess;
        if (total > 0) e = cudaMemcpyAsync(d_src, losses + lo, sizeof(double) * (size_t)total, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage.ids, ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st);
        std::vector<int64_t> rel((size_t)n + 1);
        for (int32_t i = 0; i <= n; ++i) rel[i] = offsets[i] - lo;
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(h->stage.offsets, rel.data(), sizeof(int64_t) * (n + 1), cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage.k_last, k_last, sizeof(int64_t) * n, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && m_seen)
            e = cudaMemcpyAsync(h->stage.m_seen, m_seen, sizeof(double) * n, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) {
            const int threads = 256, warps = threads / 32;
            load_kernel<<<(n + warps - 1) / warps, threads, 0, st>>>(
                h->job, h->fit, h->ring_pool, h->max_jobs, h->max_hist, n, h->stage.ids, h->stage.offsets, d_src,
                h->stage.k_last, m_seen ? h->stage.m_seen : nullptr, packed ? 1 : 0);
            e = cudaGetLastError();
        }
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // `rel` and the caller's buffers are free again
        if (e != cudaSuccess) status = cuda_fail(h, e, "bulk load");
    }
    if (old_pool) cudaFree(old_pool);   // the stream is idle: nothing points into the old pool any more
    if (status) return status;
    for (int32_t i = 0; i < n; ++i) {
        const bool now = offsets[i + 1] > offsets[i];
        h->in_packed[ids[i]] = (packed && now) ? 1 : 0;
        if (now != (h->active[ids[i]] != 0)) {
            h->active[ids[i]] = now ? 1 : 0;
            h->n_active += now ? 1 : -1;
        }
    }
    return SLAQ_OK;
}

// Without a gain table: only the plain prediction (no envelope, no target-loss hints) has its gains in closed form.
bool epoch_is_table_free(const slaq_handle* h, bool only_allocate) {
    return !only_allocate && h->selection == 1 && !h->gain_envelope && h->n_hinted == 0;
}

// The launches of one epoch, put on h->stream in order.  Returns the number of kernels or -1.
// with_events: the stage boundaries are marked with the handle's events (left out of a captured
// graph: events recorded by a graph cannot be timed).
int enqueue_epoch(slaq_handle* h, double T, int64_t want, int floor_units, int32_t* d_out, bool only_allocate,
                  bool with_events) {
    cudaStream_t st = h->stream;
    int launches = 0, k;
    if (with_events && cudaEventRecord(h->ev[0], st) != cudaSuccess) return -1;
    if (cudaMemsetAsync(h->scratch.hist, 0, h->scratch.zero_bytes, st) != cudaSuccess) return -1;
    if (!only_allocate) {
        if ((k = launch_fit(h)) < 0) return -1;
        launches += k;
    }
    if (with_events && cudaEventRecord(h->ev[1], st) != cudaSuccess) return -1;
    const bool table_free = epoch_is_table_free(h, only_allocate);
    if (!only_allocate && !table_free) {
        if ((k = launch_gain(h, T, floor_units + 1)) < 0) return -1;
        launches += k;
    }
    if (with_events && cudaEventRecord(h->ev[2], st) != cudaSuccess) return -1;
    if (table_free) k = launch_allocate_free(h, T, want, floor_units + 1, d_out);
    else k = launch_allocate(h, want, floor_units + 1, !only_allocate, d_out);
    if (k < 0) return -1;
    launches += k;
    if (with_events && cudaEventRecord(h->ev[3], st) != cudaSuccess) return -1;
    return launches;
}

// Everything the epoch's launches depend on besides device data: a graph captured for one
// key is replayed only for the same key.
std::vector<long long> epoch_key(const slaq_handle* h, double T, int64_t want, int floor_units, const int32_t* d_out,
                                 bool only_allocate) {
    long long t_bits, g_bits;
    std::memcpy(&t_bits, &T, sizeof t_bits);
    std::memcpy(&g_bits, &h->gamma, sizeof g_bits);
    return {t_bits, (long long)want, floor_units, (long long)(uintptr_t)d_out, only_allocate ? 1 : 0, h->n_active,
            h->max_cores, h->lm_trials, h->min_fit_points, h->warm_start ? 1 : 0, (long long)h->fit_slice_bytes,
            (long long)h->fit_cluster_jobs, g_bits, h->gain_envelope ? 1 : 0, h->selection, h->n_hinted,
            (long long)(uintptr_t)h->job.packed_lo, (long long)(uintptr_t)h->job.packed_hi};
}

int run_epoch(slaq_handle* h, double T, int64_t C, int32_t* d_out, bool only_allocate) {
    if (!only_allocate && !(T > 0.0 && std::isfinite(T))) return fail(h, SLAQ_E_ARG, "epoch_seconds must be positive");
    if (C < 0) return fail(h, SLAQ_E_ARG, "total_cores must not be negative");
    if (const int dc = check_device(h)) return dc;
    const int rc = ensure_weights(h);
    if (rc) return rc;
    const int64_t active = h->n_active, cap = h->max_cores;
    const int floor_units = C >= active ? 1 : 0;
    const int64_t usable = std::min<int64_t>(C, active * cap);
    const int64_t want = usable - active * floor_units;
    cudaStream_t st = h->stream;

    bool graph_ok = h->epoch_graph == 1 || (h->epoch_graph < 0 && h->max_jobs <= kGraphAutoJobs);
    if (graph_ok) {   // not while the caller captures this stream into a graph of its own
        cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &status) != cudaSuccess || status != cudaStreamCaptureStatusNone) graph_ok = false;
        if (!graph_ok) cudaGetLastError();
    }
    int launches = -1;
    h->last_epoch_was_graph = false;
    if (graph_ok) {
        const std::vector<long long> key = epoch_key(h, T, want, floor_units, d_out, only_allocate);
        if (h->graph_exec && key == h->graph_key) {
            CK(cudaEventRecord(h->ev[0], st), "event");
            CK(cudaGraphLaunch(h->graph_exec, st), "launch epoch graph");
            CK(cudaEventRecord(h->ev[3], st), "event");
            launches = h->graph_launches;
            h->last_epoch_was_graph = true;
        } else if (key == h->seen_key) {   // the second call in a row with this key: capture, then replay
            if (!h->capture_stream)
                CK(cudaStreamCreateWithFlags(&h->capture_stream, cudaStreamNonBlocking), "create capture stream");
            CK(cudaStreamBeginCapture(h->capture_stream, cudaStreamCaptureModeRelaxed), "begin capture");
            h->stream = h->capture_stream;
            const int n = enqueue_epoch(h, T, want, floor_units, d_out, only_allocate, false);
            h->stream = st;
            cudaGraph_t graph = nullptr;
            const cudaError_t e_end = cudaStreamEndCapture(h->capture_stream, &graph);
            if (n >= 0 && e_end == cudaSuccess && graph) {
                if (h->graph_exec) {
                    cudaGraphExecDestroy(h->graph_exec);
                    h->graph_exec = nullptr;
                }
                const cudaError_t e_inst = cudaGraphInstantiate(&h->graph_exec, graph, 0);
                cudaGraphDestroy(graph);
                if (e_inst == cudaSuccess) {
                    h->graph_key = key;
                    h->graph_launches = n;
                    CK(cudaEventRecord(h->ev[0], st), "event");
                    CK(cudaGraphLaunch(h->graph_exec, st), "launch epoch graph");
                    CK(cudaEventRecord(h->ev[3], st), "event");
                    launches = n;
                    h->last_epoch_was_graph = true;
                } else {
                    h->graph_exec = nullptr;
                    cudaGetLastError();
                }
            } else {
                if (graph) cudaGraphDestroy(graph);
                cudaGetLastError();
                if (n < 0) return SLAQ_E_CUDA;
            }
        }
        h->seen_key = key;
    }
    if (launches < 0) {
        launches = enqueue_epoch(h, T, want, floor_units, d_out, only_allocate, true);
        if (launches < 0) {
            if (h->err.empty()) h->err = "an epoch launch failed";
            return SLAQ_E_CUDA;
        }
    }
    h->have_epoch = true;
    h->last_launches = launches;
    h->last_cores = usable;
    // whether h->gain holds this epoch's rows (plain launches and a replayed graph alike), and what a later
    // request for them has to be predicted for
    h->gain_table_current = !epoch_is_table_free(h, only_allocate);
    h->last_T = T;
    h->last_first_unit = floor_units + 1;
    if (active > 0 && C < active) return SLAQ_W_OVERSUBSCRIBED;
    if (C > active * cap) return SLAQ_W_UNDERFILLED;
    return SLAQ_OK;
}

template <class T>
int fetch(slaq_handle* h, T* host, const T* dev, size_t n, const char* what) {
    if (!host) return SLAQ_OK;
    CK(cudaMemcpyAsync(host, dev, sizeof(T) * n, cudaMemcpyDeviceToHost, h->stream), what);
    return SLAQ_OK;
}

}  // namespace

extern "C" {

size_t slaq_workspace_bytes(int32_t max_jobs, int32_t max_hist, int32_t max_cores_per_job) {
    if (!sizes_ok(max_jobs, max_hist, max_cores_per_job)) return 0;
    return layout(nullptr, nullptr, max_jobs, max_hist, max_cores_per_job);
}

int slaq_create_in(void* dev_ws, size_t bytes, int32_t max_jobs, int32_t max_hist, int32_t max_cores_per_job,
                   slaq_t** out) {
    if (!out) return SLAQ_E_ARG;
    *out = nullptr;
    if (!sizes_ok(max_jobs, max_hist, max_cores_per_job)) return SLAQ_E_ARG;
    slaq_handle* h = new (std::nothrow) slaq_handle();
    if (!h) return SLAQ_E_NOMEM;
    const int rc = create_common(h, max_jobs, max_hist, max_cores_per_job, dev_ws, bytes);
    if (rc < 0) {
        slaq_destroy(h);
        return rc;
    }
    *out = h;
    return SLAQ_OK;
}

int slaq_create(int32_t max_jobs, int32_t max_hist, slaq_t** out) {
    return slaq_create_in(nullptr, 0, max_jobs, max_hist, 64, out);
}

int slaq_destroy(slaq_t* h) {
    if (!h) return SLAQ_OK;
    if (h->ws) cudaStreamSynchronize(h->stream);
    for (auto& ev : h->ev)
        if (ev) cudaEventDestroy(ev);
    if (h->graph_exec) cudaGraphExecDestroy(h->graph_exec);
    if (h->capture_stream) cudaStreamDestroy(h->capture_stream);
    if (h->packed_pool) cudaFree(h->packed_pool);
    if (h->call_buf) cudaFree(h->call_buf);
    if (h->owns_ws && h->ws) cudaFree(h->ws);
    delete h;
    return SLAQ_OK;
}

const char* slaq_last_error(const slaq_t* h) { return h ? h->err.c_str() : "null handle"; }

int slaq_set_stream(slaq_t* h, void* cuda_stream) {
    if (!h) return SLAQ_E_ARG;
    CK(cudaStreamSynchronize(h->stream), "sync old stream");
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    return SLAQ_OK;
}

int slaq_set_param(slaq_t* h, int key, double value) {
    if (!h) return SLAQ_E_ARG;
    switch (key) {
        case SLAQ_P_GAMMA:
            if (!(value > 0.0 && value <= 1.0)) return fail(h, SLAQ_E_ARG, "gamma must lie in (0, 1]");
            h->gamma = value;
            return SLAQ_OK;
        case SLAQ_P_LM_TRIALS:
            if (!(value >= 0 && value <= 1000)) return fail(h, SLAQ_E_ARG, "trials must lie in 0..1000");
            h->lm_trials = (int32_t)value;
            return SLAQ_OK;
        case SLAQ_P_MAX_CORES_PER_JOB:
            if (!(value >= 1 && value <= kMaxCoresLimit)) return fail(h, SLAQ_E_ARG, "max cores per job must lie in 1..1024");
            if ((int32_t)value > h->cap_alloc)
                return fail(h, SLAQ_E_RANGE, "max cores per job beyond what the handle was created for");
            h->max_cores = (int32_t)value;
            return SLAQ_OK;
        case SLAQ_P_MIN_FIT_POINTS:
            if (!(value >= 4 && value <= kMaxHistLimit)) return fail(h, SLAQ_E_ARG, "min fit points must be at least 4");
            h->min_fit_points = (int32_t)value;
            return SLAQ_OK;
        case SLAQ_P_FIT_SLICE_BYTES:
            if (!(value >= 8192 && value <= 200 * 1024)) return fail(h, SLAQ_E_ARG, "fit slice must lie in 8 KB..200 KB");
            h->fit_slice_bytes = (size_t)value;
            return SLAQ_OK;
        case SLAQ_P_WARM_START:
            if (!(value == 0.0 || value == 1.0)) return fail(h, SLAQ_E_ARG, "warm start must be 0 or 1");
            h->warm_start = value != 0.0;
            return SLAQ_OK;
        case SLAQ_P_FIT_CLUSTER_JOBS:
            if (!(value >= 0.0 && value <= 1e15)) return fail(h, SLAQ_E_ARG, "cluster jobs must not be negative");
            h->fit_cluster_jobs = (int64_t)value;
            return SLAQ_OK;
        case SLAQ_P_EPOCH_GRAPH:
            if (!(value == -1.0 || value == 0.0 || value == 1.0)) return fail(h, SLAQ_E_ARG, "epoch graph must be -1, 0 or 1");
            h->epoch_graph = (int)value;
            return SLAQ_OK;
        case SLAQ_P_GAIN_ENVELOPE:
            if (!(value == 0.0 || value == 1.0)) return fail(h, SLAQ_E_ARG, "gain envelope must be 0 or 1");
            h->gain_envelope = value != 0.0;
            return SLAQ_OK;
        case SLAQ_P_SELECTION:
            if (!(value == 0.0 || value == 1.0)) return fail(h, SLAQ_E_ARG, "selection must be 0 or 1");
            h->selection = (int)value;
            return SLAQ_OK;
        default:
            return fail(h, SLAQ_E_ARG, "unknown parameter key");
    }
}

int slaq_get_param(const slaq_t* h, int key, double* out_value) {
    if (!h || !out_value) return SLAQ_E_ARG;
    switch (key) {
        case SLAQ_P_GAMMA: *out_value = h->gamma; return SLAQ_OK;
        case SLAQ_P_LM_TRIALS: *out_value = h->lm_trials; return SLAQ_OK;
        case SLAQ_P_MAX_CORES_PER_JOB: *out_value = h->max_cores; return SLAQ_OK;
        case SLAQ_P_MIN_FIT_POINTS: *out_value = h->min_fit_points; return SLAQ_OK;
        case SLAQ_P_FIT_SLICE_BYTES: *out_value = (double)h->fit_slice_bytes; return SLAQ_OK;
        case SLAQ_P_WARM_START: *out_value = h->warm_start ? 1.0 : 0.0; return SLAQ_OK;
        case SLAQ_P_FIT_CLUSTER_JOBS: *out_value = (double)h->fit_cluster_jobs; return SLAQ_OK;
        case SLAQ_P_EPOCH_GRAPH: *out_value = (double)h->epoch_graph; return SLAQ_OK;
        case SLAQ_P_GAIN_ENVELOPE: *out_value = h->gain_envelope ? 1.0 : 0.0; return SLAQ_OK;
        case SLAQ_P_SELECTION: *out_value = (double)h->selection; return SLAQ_OK;
        default: return SLAQ_E_ARG;
    }
}

int slaq_append_losses(slaq_t* h, int32_t n, const int32_t* job_ids, const double* losses, const double* iter_times) {
    return do_append(h, n, job_ids, losses, iter_times, nullptr);
}

int slaq_append_losses_ex(slaq_t* h, int32_t n, const int32_t* job_ids, const double* losses, const double* iter_times,
                          const int32_t* cores_used) {
    return do_append(h, n, job_ids, losses, iter_times, cores_used);
}

int slaq_append_losses_device(slaq_t* h, int32_t n, const int32_t* d_job_ids, const double* d_losses,
                               const double* d_iter_times, const int32_t* d_cores_used) {
    if (!h) return SLAQ_E_ARG;
    if (const int dc = check_device(h)) return dc;
    if (n < 0) return fail(h, SLAQ_E_ARG, "negative count");
    if (n > h->max_jobs) return fail(h, SLAQ_E_ARG, "more entries than job ids");
    if (n > 0 && (!d_job_ids || !d_losses)) return fail(h, SLAQ_E_ARG, "job_ids or losses is null");
    if (d_cores_used && !d_iter_times) return fail(h, SLAQ_E_ARG, "cores_used without iter_times");
    if (n == 0) return SLAQ_OK;
    const int threads = 256;
    append_kernel<<<(n + threads - 1) / threads, threads, 0, h->stream>>>(h->job, h->fit, h->max_jobs, n, d_job_ids, d_losses,
                                                                        d_iter_times, d_cores_used, 1);
    CK(cudaGetLastError(), "append kernel");
    return SLAQ_OK;
}

int slaq_load_histories(slaq_t* h, int32_t n_jobs, const int32_t* job_ids, const int64_t* offsets, const double* losses,
                        const int64_t* k_last, const double* m_seen) {
    return do_load(h, n_jobs, job_ids, offsets, losses, k_last, m_seen, false);
}

int slaq_load_histories_packed(slaq_t* h, int32_t n_jobs, const int32_t* job_ids, const int64_t* offsets,
                               const double* losses, const int64_t* k_last, const double* m_seen) {
    return do_load(h, n_jobs, job_ids, offsets, losses, k_last, m_seen, true);
}

int slaq_set_time_model(slaq_t* h, int32_t n, const int32_t* job_ids, const double* s, const double* w) {
    if (!h) return SLAQ_E_ARG;
    if (n > 0 && (!s || !w)) return fail(h, SLAQ_E_ARG, "s or w is null");
    const int rc = check_ids(h, n, job_ids, true);
    if (rc) return rc;
    for (int32_t i = 0; i < n; ++i)
        if (!(std::isfinite(s[i]) && std::isfinite(w[i]) && s[i] >= 0.0 && w[i] > 0.0))
            return fail(h, SLAQ_E_ARG, "time law needs finite s >= 0 and w > 0");
    if (n == 0) return SLAQ_OK;
    cudaStream_t st = h->stream;
    CK(cudaMemcpyAsync(h->stage.ids, job_ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st), "copy job ids");
    CK(cudaMemcpyAsync(h->stage.losses, s, sizeof(double) * n, cudaMemcpyHostToDevice, st), "copy s");
    CK(cudaMemcpyAsync(h->stage.times, w, sizeof(double) * n, cudaMemcpyHostToDevice, st), "copy w");
    const int threads = 256;
    set_time_kernel<<<(n + threads - 1) / threads, threads, 0, st>>>(h->job, h->max_jobs, n, h->stage.ids, h->stage.losses,
                                                                    h->stage.times);
    CK(cudaGetLastError(), "time law kernel");
    CK(cudaStreamSynchronize(st), "time law");
    return SLAQ_OK;
}

int slaq_set_target_loss(slaq_t* h, int32_t n, const int32_t* job_ids, const double* targets) {
    if (!h) return SLAQ_E_ARG;
    if (n > 0 && !targets) return fail(h, SLAQ_E_ARG, "targets is null");
    const int rc = check_ids(h, n, job_ids, true);
    if (rc) return rc;
    for (int32_t i = 0; i < n; ++i)
        if (std::isinf(targets[i])) return fail(h, SLAQ_E_NONFINITE, "a target loss must be a number, or NaN for none");
    if (n == 0) return SLAQ_OK;
    cudaStream_t st = h->stream;
    CK(cudaMemcpyAsync(h->stage.ids, job_ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st), "copy job ids");
    CK(cudaMemcpyAsync(h->stage.losses, targets, sizeof(double) * n, cudaMemcpyHostToDevice, st), "copy targets");
    const int threads = 256;
    set_target_kernel<<<(n + threads - 1) / threads, threads, 0, st>>>(h->job, h->max_jobs, n, h->stage.ids, h->stage.losses);
    CK(cudaGetLastError(), "target kernel");
    CK(cudaStreamSynchronize(st), "targets");
    for (int32_t i = 0; i < n; ++i) {
        const uint8_t now = std::isnan(targets[i]) ? 0 : 1;
        h->n_hinted += (int32_t)now - (int32_t)h->hinted[job_ids[i]];
        h->hinted[job_ids[i]] = now;
    }
    return SLAQ_OK;
}

int slaq_remove_jobs(slaq_t* h, int32_t n, const int32_t* job_ids) {
    if (!h) return SLAQ_E_ARG;
    const int rc = check_ids(h, n, job_ids, false);
    if (rc) return rc;
    if (n == 0) return SLAQ_OK;
    cudaStream_t st = h->stream;
    CK(cudaMemcpyAsync(h->stage.ids, job_ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st), "copy job ids");
    const int threads = 256;
    init_jobs_kernel<<<(n + threads - 1) / threads, threads, 0, st>>>(h->job, h->fit, h->ring_pool, h->max_jobs,
                                                                     h->max_hist, h->stage.ids, n, h->alloc, h->reduction);
    CK(cudaGetLastError(), "remove kernel");
    CK(cudaStreamSynchronize(st), "remove");
    for (int32_t i = 0; i < n; ++i) {
        h->in_packed[job_ids[i]] = 0;
        if (h->hinted[job_ids[i]]) {
            h->hinted[job_ids[i]] = 0;
            h->n_hinted -= 1;
        }
        if (h->active[job_ids[i]]) {
            h->active[job_ids[i]] = 0;
            h->n_active -= 1;
        }
    }
    return SLAQ_OK;
}

int slaq_schedule_device(slaq_t* h, double epoch_seconds, int64_t total_cores, int32_t* d_out_alloc) {
    if (!h) return SLAQ_E_ARG;
    return run_epoch(h, epoch_seconds, total_cores, d_out_alloc, false);
}

int slaq_schedule(slaq_t* h, double epoch_seconds, int64_t total_cores, int32_t* out_alloc) {
    if (!h) return SLAQ_E_ARG;
    if (!out_alloc) return fail(h, SLAQ_E_ARG, "out_alloc is null");
    const int rc = run_epoch(h, epoch_seconds, total_cores, nullptr, false);
    if (rc < 0) return rc;
    CK(cudaMemcpyAsync(out_alloc, h->alloc, sizeof(int32_t) * (size_t)h->max_jobs, cudaMemcpyDeviceToHost, h->stream),
       "copy allocation");
    const int ec = check_device_errors(h);   // its synchronisation also completes the copy above
    return ec ? ec : rc;
}

int slaq_set_gains(slaq_t* h, const double* gain) {
    if (!h || !gain) return SLAQ_E_ARG;
    CK(cudaMemcpyAsync(h->gain, gain, sizeof(double) * (size_t)h->max_jobs * h->max_cores, cudaMemcpyHostToDevice,
                       h->stream),
       "copy gains");
    CK(cudaStreamSynchronize(h->stream), "copy gains");
    return SLAQ_OK;
}

int slaq_allocate_only(slaq_t* h, int64_t total_cores, int32_t* out_alloc) {
    if (!h) return SLAQ_E_ARG;
    if (!out_alloc) return fail(h, SLAQ_E_ARG, "out_alloc is null");
    const int rc = run_epoch(h, 1.0, total_cores, nullptr, true);
    if (rc < 0) return rc;
    CK(cudaMemcpyAsync(out_alloc, h->alloc, sizeof(int32_t) * (size_t)h->max_jobs, cudaMemcpyDeviceToHost, h->stream),
       "copy allocation");
    CK(cudaStreamSynchronize(h->stream), "copy allocation");
    return rc;
}

// ---- one cluster sharded over several GPUs ----

int slaq_get_active_count(slaq_t* h, int32_t* out_active) {
    if (!h || !out_active) return SLAQ_E_ARG;
    *out_active = h->n_active;
    return SLAQ_OK;
}

int slaq_shard_predict(slaq_t* h, double epoch_seconds, int32_t with_floor) {
    if (!h) return SLAQ_E_ARG;
    if (!(epoch_seconds > 0.0 && std::isfinite(epoch_seconds))) return fail(h, SLAQ_E_ARG, "epoch_seconds must be positive");
    if (const int dc = check_device(h)) return dc;
    const int rc = ensure_weights(h);
    if (rc) return rc;
    cudaStream_t st = h->stream;
    int launches = 0, k;
    h->shard_first_unit = with_floor ? 2 : 1;
    h->last_epoch_was_graph = false;
    CK(cudaMemsetAsync(h->scratch.hist, 0, h->scratch.zero_bytes, st), "clear scratch");
    CK(cudaEventRecord(h->ev[0], st), "event");
    if ((k = launch_fit(h)) < 0) return SLAQ_E_CUDA;
    launches += k;
    CK(cudaEventRecord(h->ev[1], st), "event");
    if ((k = launch_gain(h, epoch_seconds, h->shard_first_unit)) < 0) return SLAQ_E_CUDA;
    launches += k;
    CK(cudaEventRecord(h->ev[2], st), "event");
    CK(cudaEventRecord(h->ev[3], st), "event");
    h->have_epoch = true;
    h->last_launches = launches;
    h->gain_table_current = true;
    h->last_T = epoch_seconds;
    h->last_first_unit = h->shard_first_unit;
    return SLAQ_OK;
}

int slaq_shard_histogram(slaq_t* h, int32_t pass, uint64_t* d_hist, int32_t import_it) {
    if (!h || !d_hist) return SLAQ_E_ARG;
    if (pass < 0 || pass >= kRadixPasses) return fail(h, SLAQ_E_ARG, "pass outside 0..5");
    unsigned long long* mine = h->scratch.hist + (size_t)pass * kRadixBins;
    const size_t bytes = sizeof(unsigned long long) * kRadixBins;
    if (import_it)
        CK(cudaMemcpyAsync(mine, d_hist, bytes, cudaMemcpyDeviceToDevice, h->stream), "import histogram");
    else
        CK(cudaMemcpyAsync(d_hist, mine, bytes, cudaMemcpyDeviceToDevice, h->stream), "export histogram");
    return SLAQ_OK;
}

int slaq_shard_pick(slaq_t* h, int32_t pass, int64_t want) {
    if (!h) return SLAQ_E_ARG;
    if (pass < 0 || pass >= kRadixPasses) return fail(h, SLAQ_E_ARG, "pass outside 0..5");
    const int k = launch_shard_pick(h, pass, want);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    return SLAQ_OK;
}

int slaq_shard_pass(slaq_t* h, int32_t pass) {
    if (!h) return SLAQ_E_ARG;
    if (pass < 1 || pass >= kRadixPasses) return fail(h, SLAQ_E_ARG, "pass outside 1..5");
    const int k = launch_shard_pass(h, pass, h->shard_first_unit);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    return SLAQ_OK;
}

int slaq_shard_count(slaq_t* h, int64_t* out_local_ties) {
    if (!h || !out_local_ties) return SLAQ_E_ARG;
    const long long* d_total = nullptr;
    const int k = launch_shard_count(h, h->shard_first_unit, &d_total);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    long long total = 0;
    CK(cudaMemcpyAsync(&total, d_total, sizeof total, cudaMemcpyDeviceToHost, h->stream), "read tie count");
    CK(cudaStreamSynchronize(h->stream), "read tie count");
    *out_local_ties = total;
    return SLAQ_OK;
}

int slaq_shard_count_device(slaq_t* h, int64_t* d_out_local_ties) {
    if (!h || !d_out_local_ties) return SLAQ_E_ARG;
    const long long* d_total = nullptr;
    const int k = launch_shard_count(h, h->shard_first_unit, &d_total);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    CK(cudaMemcpyAsync(d_out_local_ties, d_total, sizeof(long long), cudaMemcpyDeviceToDevice, h->stream), "export tie count");
    return SLAQ_OK;
}

int slaq_shard_finalise_device(slaq_t* h, const int64_t* d_ties_before, int32_t* out_alloc) {
    if (!h) return SLAQ_E_ARG;
    if (!out_alloc || !d_ties_before) return fail(h, SLAQ_E_ARG, "out_alloc or d_ties_before is null");
    const int k = launch_shard_finalise(h, h->shard_first_unit, 0, reinterpret_cast<const long long*>(d_ties_before), nullptr);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    CK(cudaEventRecord(h->ev[3], h->stream), "event");
    CK(cudaMemcpyAsync(out_alloc, h->alloc, sizeof(int32_t) * (size_t)h->max_jobs, cudaMemcpyDeviceToHost, h->stream),
       "copy allocation");
    return check_device_errors(h);
}

int slaq_shard_finalise(slaq_t* h, int64_t ties_before, int32_t* out_alloc) {
    if (!h) return SLAQ_E_ARG;
    if (!out_alloc) return fail(h, SLAQ_E_ARG, "out_alloc is null");
    if (ties_before < 0) return fail(h, SLAQ_E_ARG, "ties_before must not be negative");
    const int k = launch_shard_finalise(h, h->shard_first_unit, ties_before, nullptr, nullptr);
    if (k < 0) return SLAQ_E_CUDA;
    h->last_launches += k;
    CK(cudaEventRecord(h->ev[3], h->stream), "event");
    CK(cudaMemcpyAsync(out_alloc, h->alloc, sizeof(int32_t) * (size_t)h->max_jobs, cudaMemcpyDeviceToHost, h->stream),
       "copy allocation");
    return check_device_errors(h);
}

int slaq_get_predictions(slaq_t* h, double* out_reduction, double* out_gain, int8_t* out_family, double* out_params,
                         double* out_residual, int32_t* out_status, int32_t* out_sweeps, double* out_largest) {
    if (!h) return SLAQ_E_ARG;
    if (!h->have_epoch) return fail(h, SLAQ_E_ARG, "no epoch has been scheduled yet");
    const size_t J = (size_t)h->max_jobs;
    int rc = 0;
    if (out_gain && !h->gain_table_current) {   // the last epoch ran without a table: write the rows now
        if (launch_gain(h, h->last_T, h->last_first_unit) < 0) return SLAQ_E_CUDA;
        h->gain_table_current = true;
    }
    if ((rc = fetch(h, out_reduction, h->reduction, J, "copy reductions"))) return rc;
    if ((rc = fetch(h, out_gain, h->gain, J * h->max_cores, "copy gains"))) return rc;
    if ((rc = fetch(h, out_family, h->fit.family, J, "copy families"))) return rc;
    if ((rc = fetch(h, out_params, h->fit.params, 4 * J, "copy parameters"))) return rc;
    if ((rc = fetch(h, out_residual, h->fit.residual, 2 * J, "copy residuals"))) return rc;
    if ((rc = fetch(h, out_status, h->fit.status, J, "copy status"))) return rc;
    if ((rc = fetch(h, out_sweeps, h->fit.sweeps, 2 * J, "copy sweeps"))) return rc;
    if ((rc = fetch(h, out_largest, h->fit.largest, J, "copy largest reductions"))) return rc;
    CK(cudaStreamSynchronize(h->stream), "copy predictions");
    return SLAQ_OK;
}

int slaq_get_normalised(slaq_t* h, int32_t n, const int32_t* job_ids, int64_t capacity, int64_t* out_offsets,
                        double* out_changes, double* out_levels, double* out_largest) {
    if (!h) return SLAQ_E_ARG;
    int rc = check_ids(h, n, job_ids, false);
    if (rc) return rc;
    if ((rc = ensure_weights(h))) return rc;
    if (n == 0) {
        if (out_offsets) out_offsets[0] = 0;
        return SLAQ_OK;
    }
    cudaStream_t st = h->stream;
    std::vector<int32_t> counts((size_t)h->max_jobs);
    CK(cudaMemcpyAsync(counts.data(), h->job.count, sizeof(int32_t) * counts.size(), cudaMemcpyDeviceToHost, st),
       "read window lengths");
    CK(cudaStreamSynchronize(st), "read window lengths");
    std::vector<int64_t> offs((size_t)n + 1, 0);
    for (int32_t i = 0; i < n; ++i) offs[i + 1] = offs[i] + counts[job_ids[i]];
    const int64_t total = offs[n];
    if ((out_changes || out_levels) && total > capacity) return fail(h, SLAQ_E_RANGE, "output capacity too small");
    if (out_offsets) std::memcpy(out_offsets, offs.data(), sizeof(int64_t) * (n + 1));
    // one handle-owned buffer: [n] largest, then [total] changes and [total] levels
    void* buf = nullptr;
    const size_t n_pad = ((size_t)n + 31) / 32 * 32;
    if ((rc = ensure_call_buffer(h, sizeof(double) * (n_pad + 2 * (size_t)total), &buf))) return rc;
    double* d_largest = static_cast<double*>(buf);
    double* d_changes = total > 0 ? d_largest + n_pad : nullptr;
    double* d_levels = total > 0 ? d_changes + total : nullptr;
    int status = SLAQ_OK;
    cudaError_t e = cudaMemcpyAsync(h->stage.ids, job_ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(h->stage.offsets, offs.data(), sizeof(int64_t) * (n + 1), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && launch_normalise_export(h, n, h->stage.offsets, d_changes, d_levels, d_largest) < 0)
        status = SLAQ_E_CUDA;
    if (e == cudaSuccess && status == SLAQ_OK) {
        if (out_changes && total > 0)
            e = cudaMemcpyAsync(out_changes, d_changes, sizeof(double) * (size_t)total, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess && out_levels && total > 0)
            e = cudaMemcpyAsync(out_levels, d_levels, sizeof(double) * (size_t)total, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess && out_largest)
            e = cudaMemcpyAsync(out_largest, d_largest, sizeof(double) * n, cudaMemcpyDeviceToHost, st);
    }
    const cudaError_t e2 = cudaStreamSynchronize(st);
    if (e == cudaSuccess) e = e2;
    if (e != cudaSuccess) status = cuda_fail(h, e, "normalised export");
    return status;
}

int slaq_get_time_model(slaq_t* h, double* out_s, double* out_w) {
    if (!h || !out_s || !out_w) return SLAQ_E_ARG;
    // the staging arrays hold one double per job each: they serve as the kernel's output
    if (launch_time_model(h, h->stage.losses, h->stage.times) < 0) return SLAQ_E_CUDA;
    const size_t J = (size_t)h->max_jobs;
    CK(cudaMemcpyAsync(out_s, h->stage.losses, sizeof(double) * J, cudaMemcpyDeviceToHost, h->stream), "copy s");
    CK(cudaMemcpyAsync(out_w, h->stage.times, sizeof(double) * J, cudaMemcpyDeviceToHost, h->stream), "copy w");
    CK(cudaStreamSynchronize(h->stream), "copy time law");
    return SLAQ_OK;
}

int slaq_get_fit_state(slaq_t* h, double* out_params, uint8_t* out_mask, int64_t* out_k, double* out_span,
                       double* out_scale) {
    if (!h || !out_params || !out_mask || !out_k || !out_span || !out_scale) return SLAQ_E_ARG;
    if (const int rc = check_device(h)) return rc;
    const size_t J = (size_t)h->max_jobs;
    int rc;
    if ((rc = fetch(h, out_params, h->fit.both, 8 * J, "copy fitted parameters"))) return rc;
    if ((rc = fetch(h, out_mask, h->fit.mask, J, "copy fit masks"))) return rc;
    if ((rc = fetch(h, out_k, h->fit.k_fit, J, "copy fit iteration indices"))) return rc;
    if ((rc = fetch(h, out_span, h->fit.span, J, "copy fit spans"))) return rc;
    if ((rc = fetch(h, out_scale, h->fit.largest, J, "copy fit scales"))) return rc;
    CK(cudaStreamSynchronize(h->stream), "copy fit state");
    return SLAQ_OK;
}

int slaq_set_fit_state(slaq_t* h, const double* params, const uint8_t* mask, const int64_t* k, const double* span,
                       const double* scale) {
    if (!h || !params || !mask || !k || !span || !scale) return SLAQ_E_ARG;
    if (const int rc = check_device(h)) return rc;
    const size_t J = (size_t)h->max_jobs;
    for (size_t j = 0; j < J; ++j) {
        if (!mask[j]) continue;
        if (mask[j] > 3) return fail(h, SLAQ_E_ARG, "fit mask above 3");
        if (!h->active[j]) return fail(h, SLAQ_E_ARG, "fit state for a job without losses");
        if (!(span[j] > 0.0 && std::isfinite(span[j]) && scale[j] > 0.0 && std::isfinite(scale[j])))
            return fail(h, SLAQ_E_ARG, "fit state needs a positive finite span and scale");
    }
    cudaStream_t st = h->stream;
    const cudaMemcpyKind up = cudaMemcpyHostToDevice;
    CK(cudaMemcpyAsync(h->fit.both, params, sizeof(double) * 8 * J, up, st), "copy fitted parameters");
    CK(cudaMemcpyAsync(h->fit.warm_p, params, sizeof(double) * 8 * J, up, st), "copy fitted parameters");
    CK(cudaMemcpyAsync(h->fit.mask, mask, sizeof(uint8_t) * J, up, st), "copy fit masks");
    CK(cudaMemcpyAsync(h->fit.warm_mask, mask, sizeof(uint8_t) * J, up, st), "copy fit masks");
    CK(cudaMemcpyAsync(h->fit.k_fit, k, sizeof(int64_t) * J, up, st), "copy fit iteration indices");
    CK(cudaMemcpyAsync(h->fit.warm_k, k, sizeof(int64_t) * J, up, st), "copy fit iteration indices");
    CK(cudaMemcpyAsync(h->fit.span, span, sizeof(double) * J, up, st), "copy fit spans");
    CK(cudaMemcpyAsync(h->fit.warm_span, span, sizeof(double) * J, up, st), "copy fit spans");
    CK(cudaMemcpyAsync(h->fit.largest, scale, sizeof(double) * J, up, st), "copy fit scales");
    CK(cudaMemcpyAsync(h->fit.warm_scale, scale, sizeof(double) * J, up, st), "copy fit scales");
    CK(cudaStreamSynchronize(st), "copy fit state");
    return SLAQ_OK;
}

// ---- the whole scheduler state as one host blob ----

namespace {

constexpr uint64_t kStateMagic = 0x51414c5345544154ull;   // "TATESLAQ" read as little-endian bytes
constexpr uint32_t kStateVersion = 1;

struct StateHeader {
    uint64_t magic;
    uint32_t version;
    int32_t max_jobs;
    int32_t max_hist;      // longest window in the blob
    int32_t reserved;
    int64_t total_points;
    uint64_t bytes;        // size of the whole blob
};

// The per-job arrays of a blob, in order, each entry count given per job; all 8-byte aligned
// because every block's size is a multiple of 8 (max_jobs is padded to a multiple of 8 entries).
struct StateLayout {
    size_t J8;             // max_jobs rounded up to a multiple of 8
    size_t off_count, off_k_last, off_m_seen, off_tm, off_s_set, off_w_set, off_last_alloc, off_target;
    size_t off_both, off_mask, off_k_fit, off_span, off_largest;
    size_t off_warm_p, off_warm_mask, off_warm_k, off_warm_span, off_warm_scale;
    size_t off_offsets, off_losses, bytes;
};

StateLayout state_layout(int32_t max_jobs, int64_t total_points) {
    StateLayout L;
    L.J8 = ((size_t)max_jobs + 7) / 8 * 8;
    size_t o = sizeof(StateHeader);
    auto take = [&](size_t bytes) { const size_t at = o; o += (bytes + 7) / 8 * 8; return at; };
    L.off_count = take(4 * L.J8);
    L.off_k_last = take(8 * L.J8);
    L.off_m_seen = take(8 * L.J8);
    L.off_tm = take(8 * 8 * (size_t)max_jobs);
    L.off_s_set = take(8 * L.J8);
    L.off_w_set = take(8 * L.J8);
    L.off_last_alloc = take(4 * L.J8);
    L.off_target = take(8 * L.J8);
    L.off_both = take(8 * 8 * L.J8);
    L.off_mask = take(L.J8);
    L.off_k_fit = take(8 * L.J8);
    L.off_span = take(8 * L.J8);
    L.off_largest = take(8 * L.J8);
    L.off_warm_p = take(8 * 8 * L.J8);
    L.off_warm_mask = take(L.J8);
    L.off_warm_k = take(8 * L.J8);
    L.off_warm_span = take(8 * L.J8);
    L.off_warm_scale = take(8 * L.J8);
    L.off_offsets = take(8 * ((size_t)max_jobs + 1));
    L.off_losses = take(8 * (size_t)total_points);
    L.bytes = o;
    return L;
}

int read_counts(slaq_handle* h, std::vector<int32_t>& counts, int64_t* total, int32_t* longest) {
    counts.resize((size_t)h->max_jobs);
    CK(cudaMemcpyAsync(counts.data(), h->job.count, sizeof(int32_t) * counts.size(), cudaMemcpyDeviceToHost, h->stream),
       "read window lengths");
    CK(cudaStreamSynchronize(h->stream), "read window lengths");
    *total = 0;
    *longest = 0;
    for (int32_t c : counts) {
        *total += c > 0 ? c : 0;
        *longest = std::max(*longest, c);
    }
    return SLAQ_OK;
}

}  // namespace

int slaq_export_state_bytes(slaq_t* h, size_t* out_bytes) {
    if (!h || !out_bytes) return SLAQ_E_ARG;
    if (const int rc = check_device(h)) return rc;
    std::vector<int32_t> counts;
    int64_t total = 0;
    int32_t longest = 0;
    if (const int rc = read_counts(h, counts, &total, &longest)) return rc;
    *out_bytes = state_layout(h->max_jobs, total).bytes;
    return SLAQ_OK;
}

int slaq_export_state(slaq_t* h, void* out_blob, size_t capacity) {
    if (!h || !out_blob) return SLAQ_E_ARG;
    if (const int rc = check_device(h)) return rc;
    std::vector<int32_t> counts;
    int64_t total = 0;
    int32_t longest = 0;
    if (const int rc = read_counts(h, counts, &total, &longest)) return rc;
    const StateLayout L = state_layout(h->max_jobs, total);
    if (capacity < L.bytes) return fail(h, SLAQ_E_RANGE, "blob capacity below slaq_export_state_bytes()");
    char* blob = static_cast<char*>(out_blob);
    std::memset(blob, 0, L.bytes);
    StateHeader hd{kStateMagic, kStateVersion, h->max_jobs, longest, 0, total, (uint64_t)L.bytes};
    std::memcpy(blob, &hd, sizeof hd);
    const size_t J = (size_t)h->max_jobs;
    int64_t* offsets = reinterpret_cast<int64_t*>(blob + L.off_offsets);
    offsets[0] = 0;
    for (size_t j = 0; j < J; ++j) offsets[j + 1] = offsets[j] + (counts[j] > 0 ? counts[j] : 0);
    cudaStream_t st = h->stream;
    const cudaMemcpyKind down = cudaMemcpyDeviceToHost;
    std::memcpy(blob + L.off_count, counts.data(), 4 * J);
    CK(cudaMemcpyAsync(blob + L.off_k_last, h->job.k_last, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_m_seen, h->job.m_seen, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_tm, h->job.tm, 8 * 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_s_set, h->job.s_set, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_w_set, h->job.w_set, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_last_alloc, h->job.last_alloc, 4 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_target, h->job.target, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_both, h->fit.both, 8 * 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_mask, h->fit.mask, J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_k_fit, h->fit.k_fit, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_span, h->fit.span, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_largest, h->fit.largest, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_warm_p, h->fit.warm_p, 8 * 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_warm_mask, h->fit.warm_mask, J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_warm_k, h->fit.warm_k, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_warm_span, h->fit.warm_span, 8 * J, down, st), "export state");
    CK(cudaMemcpyAsync(blob + L.off_warm_scale, h->fit.warm_scale, 8 * J, down, st), "export state");
    if (total > 0) {
        void* buf = nullptr;
        if (const int rc = ensure_call_buffer(h, 8 * (size_t)total, &buf)) return rc;
        CK(cudaMemcpyAsync(h->stage.offsets, offsets, 8 * (J + 1), cudaMemcpyHostToDevice, st), "export state");
        const int threads = 256, warps = threads / 32;
        export_windows_kernel<<<(h->max_jobs + warps - 1) / warps, threads, 0, st>>>(h->job, h->max_jobs, h->stage.offsets,
                                                                                  static_cast<double*>(buf));
        CK(cudaGetLastError(), "export kernel");
        CK(cudaMemcpyAsync(blob + L.off_losses, buf, 8 * (size_t)total, down, st), "export state");
    }
    CK(cudaStreamSynchronize(st), "export state");
    return SLAQ_OK;
}

int slaq_import_state(slaq_t* h, const void* blob_in, size_t bytes) {
    if (!h || !blob_in) return SLAQ_E_ARG;
    if (const int rc = check_device(h)) return rc;
    const char* blob = static_cast<const char*>(blob_in);
    StateHeader hd;
    if (bytes < sizeof hd) return fail(h, SLAQ_E_ARG, "state blob shorter than its header");
    std::memcpy(&hd, blob, sizeof hd);
    if (hd.magic != kStateMagic || hd.version != kStateVersion) return fail(h, SLAQ_E_ARG, "not a state blob of this library version");
    if (hd.max_jobs != h->max_jobs) return fail(h, SLAQ_E_RANGE, "state blob of a handle with another number of job ids");
    if (hd.max_hist > h->max_hist) return fail(h, SLAQ_E_RANGE, "state blob holds windows longer than this handle's max_hist");
    if (hd.total_points < 0) return fail(h, SLAQ_E_ARG, "state blob: negative point count");
    const StateLayout L = state_layout(hd.max_jobs, hd.total_points);
    if (hd.bytes != L.bytes || bytes < L.bytes) return fail(h, SLAQ_E_ARG, "state blob is truncated or its sizes disagree");
    const size_t J = (size_t)h->max_jobs;
    const int32_t* counts = reinterpret_cast<const int32_t*>(blob + L.off_count);
    const int64_t* offsets = reinterpret_cast<const int64_t*>(blob + L.off_offsets);
    const int64_t* k_last = reinterpret_cast<const int64_t*>(blob + L.off_k_last);
    const double* m_seen = reinterpret_cast<const double*>(blob + L.off_m_seen);
    const uint8_t* mask = reinterpret_cast<const uint8_t*>(blob + L.off_mask);
    const uint8_t* warm_mask = reinterpret_cast<const uint8_t*>(blob + L.off_warm_mask);
    if (offsets[0] != 0 || offsets[J] != hd.total_points) return fail(h, SLAQ_E_ARG, "state blob: offsets disagree with the point count");
    for (size_t j = 0; j < J; ++j) {
        const int64_t H = offsets[j + 1] - offsets[j];
        if (H < 0 || H > h->max_hist || H != (counts[j] > 0 ? counts[j] : 0))
            return fail(h, SLAQ_E_ARG, "state blob: a window length disagrees with its offsets");
        if (std::isnan(m_seen[j]) || m_seen[j] == INFINITY) return fail(h, SLAQ_E_NONFINITE, "state blob: m_seen must be a number below +infinity");
        if (mask[j] > 3 || warm_mask[j] > 3) return fail(h, SLAQ_E_ARG, "state blob: fit mask above 3");
    }
    // everything the handle holds goes; then the windows come in as a bulk load into rings (which checks the losses)
    cudaStream_t st = h->stream;
    {
        const int threads = 256;
        init_jobs_kernel<<<(h->max_jobs + threads - 1) / threads, threads, 0, st>>>(
            h->job, h->fit, h->ring_pool, h->max_jobs, h->max_hist, nullptr, h->max_jobs, h->alloc, h->reduction);
        CK(cudaGetLastError(), "import: reset kernel");
        CK(cudaStreamSynchronize(st), "import: reset");
        std::fill(h->active.begin(), h->active.end(), 0);
        std::fill(h->in_packed.begin(), h->in_packed.end(), 0);
        std::fill(h->hinted.begin(), h->hinted.end(), 0);
        h->n_hinted = 0;
        h->n_active = 0;
        if (h->packed_pool) {
            cudaFree(h->packed_pool);
            h->packed_pool = nullptr;
            h->packed_len = 0;
            h->job.packed_lo = h->job.packed_hi = nullptr;
        }
        h->have_epoch = false;
    }
    std::vector<int32_t> ids(J);
    for (size_t j = 0; j < J; ++j) ids[j] = (int32_t)j;
    const int rc = do_load(h, h->max_jobs, ids.data(), offsets, reinterpret_cast<const double*>(blob + L.off_losses), k_last,
                           m_seen, false);
    if (rc) return rc;
    const cudaMemcpyKind up = cudaMemcpyHostToDevice;
    CK(cudaMemcpyAsync(h->job.tm, blob + L.off_tm, 8 * 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->job.s_set, blob + L.off_s_set, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->job.w_set, blob + L.off_w_set, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->job.last_alloc, blob + L.off_last_alloc, 4 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->job.target, blob + L.off_target, 8 * J, up, st), "import state");
    {
        const double* target = reinterpret_cast<const double*>(blob + L.off_target);
        for (size_t j = 0; j < J; ++j)
            if (!std::isnan(target[j])) {
                h->hinted[j] = 1;
                h->n_hinted += 1;
            }
    }
    CK(cudaMemcpyAsync(h->fit.both, blob + L.off_both, 8 * 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.mask, blob + L.off_mask, J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.k_fit, blob + L.off_k_fit, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.span, blob + L.off_span, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.largest, blob + L.off_largest, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.warm_p, blob + L.off_warm_p, 8 * 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.warm_mask, blob + L.off_warm_mask, J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.warm_k, blob + L.off_warm_k, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.warm_span, blob + L.off_warm_span, 8 * J, up, st), "import state");
    CK(cudaMemcpyAsync(h->fit.warm_scale, blob + L.off_warm_scale, 8 * J, up, st), "import state");
    CK(cudaStreamSynchronize(st), "import state");
    return SLAQ_OK;
}

int slaq_get_fit_phase_cycles(slaq_t* h, int64_t* out_cycles) {
    if (!h || !out_cycles) return SLAQ_E_ARG;
    if (!h->have_epoch) return fail(h, SLAQ_E_ARG, "no epoch has been scheduled yet");
    long long counters[16];
    CK(cudaMemcpyAsync(counters, h->scratch.counters, sizeof counters, cudaMemcpyDeviceToHost, h->stream), "copy counters");
    CK(cudaStreamSynchronize(h->stream), "copy phase cycles");
    for (int i = 0; i < 6; ++i) out_cycles[i] = counters[8 + i];
    return SLAQ_OK;
}

int slaq_get_stats(slaq_t* h, slaq_stats* out) {
    if (!h || !out) return SLAQ_E_ARG;
    if (!h->have_epoch) return fail(h, SLAQ_E_ARG, "no epoch has been scheduled yet");
    std::memset(out, 0, sizeof *out);
    long long counters[16];
    SelectState sel;
    CK(cudaMemcpyAsync(counters, h->scratch.counters, sizeof counters, cudaMemcpyDeviceToHost, h->stream), "copy counters");
    CK(cudaMemcpyAsync(&sel, h->scratch.sel, sizeof sel, cudaMemcpyDeviceToHost, h->stream), "copy selection state");
    CK(cudaStreamSynchronize(h->stream), "copy statistics");
    CK(cudaEventElapsedTime(&out->ms_total, h->ev[0], h->ev[3]), "event time");
    if (!h->last_epoch_was_graph) {   // a replayed graph has no stage boundaries to time
        CK(cudaEventElapsedTime(&out->ms_fit, h->ev[0], h->ev[1]), "event time");
        CK(cudaEventElapsedTime(&out->ms_gain, h->ev[1], h->ev[2]), "event time");
        CK(cudaEventElapsedTime(&out->ms_alloc, h->ev[2], h->ev[3]), "event time");
    }
    out->launches = h->last_launches;
    out->active_jobs = h->n_active;
    out->points = counters[0];
    out->model_sweeps = counters[1];
    out->fitted_jobs = (int32_t)counters[2];
    out->sublinear_wins = (int32_t)counters[3];
    out->exponential_wins = (int32_t)counters[4];
    out->fallback_jobs = (int32_t)counters[5];
    out->nonconvex_fits = (int32_t)counters[14];
    out->cores_handed_out = counters[6];
    out->tie_units = counters[7];
    double tau = 0.0;
    if (sel.prefix != ~0ull) std::memcpy(&tau, &sel.prefix, sizeof tau);
    out->threshold = tau;
    return SLAQ_OK;
}

}  // extern "C"
