// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "slaq.h"
#include "slaq_bounds.cuh"

namespace slaq {

constexpr int kMaxHistLimit = 6000;   // one warp stages a whole window in shared memory
constexpr int kMaxCoresLimit = 1024;
constexpr int kRadixBits = 11;
constexpr int kRadixBins = 1 << kRadixBits;
constexpr int kRadixPasses = 6;       // 11 + 11 + 11 + 11 + 11 + 9 bits, most significant first
constexpr int kMaxFitClasses = 8;     // window-length classes of the fit (one launch each)
constexpr int kFitQueueBase = 8;      // ticket[kFitQueueBase + c]: work queue head of class c
constexpr int kTickets = 16;
constexpr int kGraphAutoJobs = 20000;  // handles up to this size replay the epoch as a CUDA graph unless told otherwise

// Device-side state of one job, structure of arrays (index = job id).
struct JobArrays {
    double** row;        // start of the job's window storage (ring of `cap` slots)
    int32_t* cap;        // slots in the ring
    int32_t* head;       // slot the next loss goes to
    int32_t* count;      // stored losses, 0 = inactive
    int64_t* k_last;     // iteration index of the newest loss
    double* m_seen;      // largest one-step reduction seen so far (-inf: none)
    double* tm;          // [8][max_jobs]: count, sum u, sum u^2, sum t, sum u t, sum t n, min u, max u (u = 1/cores)
    double* s_set;       // fixed time law (NaN: use the estimate)
    double* w_set;
    int32_t* last_alloc; // core count of the last epoch (1 before any)
    double* target;      // hint of the loss the job will end at (NaN: none)
    // extents, read by the bounds build only
    int32_t max_jobs;
    const double* ring_lo;     // the ring pool [ring_lo, ring_hi)
    const double* ring_hi;
    const double* packed_lo;   // the packed pool (both null while there is none)
    const double* packed_hi;
    int32_t* err_word;
};

// What the fit leaves for the later stages, one entry per job.
struct FitArrays {
    int32_t* status;     // SLAQ_JOB_*
    int8_t* family;      // 0, 1 or -1
    double* params;      // [max_jobs][4]; linear-extrapolation kinds keep (rho, r_cap) in slots 0, 1
    double* residual;    // [max_jobs][2]
    int32_t* sweeps;     // [max_jobs][2]
    double* largest;     // M
    double* span;        // max(H-1, 1)
    // Both families' end points of the last epoch, in that epoch's window coordinates
    // (span, largest and k_fit say which), and the copy the next fit may start from.  A
    // job's copy is refreshed when its history changes, so an epoch repeated without new
    // losses starts from the same point and gives the same result.
    double* both;        // [max_jobs][8]: family I (a, b, c, d), family II (alpha, beta, c, unused)
    uint8_t* mask;       // bit 0 / 1: family I / II ended with a finite residual
    int64_t* k_fit;      // index of the newest iteration at that fit
    double* warm_p;      // [max_jobs][8]
    uint8_t* warm_mask;
    int64_t* warm_k;
    double* warm_span;
    double* warm_scale;
};

// Running state of the radix select.
struct SelectState {
    unsigned long long prefix;       // bits of the threshold key found so far
    long long want;                  // units still to take inside the current candidate set
    int done;                        // nothing is wanted: the threshold lies above every gain
};

// Scratch of one epoch; [hist, hist + zero_bytes) is cleared at the start of every epoch.
struct Scratch {
    unsigned long long* hist;        // [kRadixPasses][kRadixBins]
    unsigned int* ticket;            // [kTickets]: block-completion counter per radix pass, work queue per fit class
    SelectState* sel;
    long long* counters;             // [16] statistics accumulated by kernels
    size_t zero_bytes;
    int32_t* gt;                     // per job: during the passes the start of its candidate segment, then gains above the threshold
    int32_t* eq;                     // per job: during the passes the end of its segment, then gains equal to the threshold
    long long* block_eq;             // per block of the count kernel: sum of eq
    int32_t* bucket;                 // [max_hist + 1] jobs per window length (inside the cleared region)
    int32_t* order;                  // job ids, longest window first (fit kernel work list)
    int32_t* start;                  // [max_hist + 1] start[h] = jobs with a window longer than h
    int32_t* cursor;                 // [max_hist + 1] scatter positions of the counting sort
};

struct Staging {
    int32_t* ids;
    double* losses;
    double* times;
    int32_t* cores;
    int64_t* offsets;
    int64_t* k_last;
    double* m_seen;
};

}  // namespace slaq

struct slaq_handle {
    int device = 0;
    int32_t max_jobs = 0, max_hist = 0, cap_alloc = 0;   // cap_alloc: gain columns the buffers were sized for
    int32_t max_cores = 64;
    double gamma = 0.9;
    int32_t lm_trials = 20, min_fit_points = 4;
    size_t fit_slice_bytes = 13824;       // shared memory one warp of the fit kernel may use (parked sums, up to 52 rows of 32 points, a spare row)
    bool warm_start = false;              // fits start from the last epoch's parameters where there are some
    int selection = 0;                    // 0: selection over the written gain table, 1: gains evaluated on demand, no table
    bool gain_table_current = false;      // h->gain holds the rows of the last epoch
    double last_T = 0.0;                  // what the last epoch's gains were predicted for
    int last_first_unit = 2;
    std::vector<uint8_t> hinted;          // host mirror: job has a target-loss hint
    int32_t n_hinted = 0;
    bool gain_envelope = false;           // gain rows are slopes of the concave envelope of R(n), not a running minimum
    int64_t fit_cluster_jobs = 0;         // active jobs the lanes per job are chosen for (0: this handle's own)
    cudaStream_t stream = nullptr;
    bool owns_ws = false;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    double* ring_pool = nullptr;      // [max_jobs][max_hist]
    double* packed_pool = nullptr;    // separate allocation made by slaq_load_histories_packed
    size_t packed_len = 0;
    void* call_buf = nullptr;         // scratch of calls that move caller data of any size (grown on demand, kept)
    size_t call_buf_bytes = 0;
    double* wtab = nullptr;           // gamma^m, m = 0..max_hist-1
    double wtab_gamma = -1.0;
    slaq::JobArrays job;
    slaq::FitArrays fit;
    slaq::Scratch scratch;
    slaq::Staging stage;
    double* gain = nullptr;           // [max_jobs][max_cores]
    int32_t* alloc = nullptr;
    double* reduction = nullptr;
    int32_t* err_word = nullptr;      // device error flags set by kernels
    cudaEvent_t ev[4] = {};
    bool have_epoch = false;
    int32_t last_launches = 0;
    int64_t last_cores = 0;
    int sm_count = 148;
    std::vector<uint8_t> active;      // host mirror: job has at least one loss
    std::vector<uint32_t> stamp;      // host: duplicate detection
    std::vector<uint8_t> in_packed;   // host: job's row lives in the packed pool
    uint32_t stamp_epoch = 0;
    int32_t n_active = 0;
    int shard_first_unit = 2;         // set by slaq_shard_predict for the steps that follow
    // The epoch as a CUDA graph: what the captured launches depended on, the instantiated graph,
    // and the stream the capture runs on (the caller's stream may be the legacy default stream,
    // which cannot capture).
    int epoch_graph = -1;             // 0 never, 1 always, -1: for handles of at most kGraphAutoJobs jobs
    std::vector<long long> graph_key, seen_key;
    cudaGraphExec_t graph_exec = nullptr;
    cudaStream_t capture_stream = nullptr;
    int32_t graph_launches = 0;
    bool last_epoch_was_graph = false;
    std::string err;
};

namespace slaq {

// kernel launchers: each returns the number of kernels it launched, or -1 after setting h->err
int launch_fit(slaq_handle* h);
int launch_gain(slaq_handle* h, double epoch_seconds, int first_unit);
int launch_allocate(slaq_handle* h, long long want, int first_unit, bool hist0_ready, int32_t* d_out_alloc);
int launch_allocate_free(slaq_handle* h, double epoch_seconds, long long want, int first_unit, int32_t* d_out_alloc);
int launch_normalise_export(slaq_handle* h, int32_t n, const int64_t* d_offsets, double* d_changes,
                            double* d_levels, double* d_largest);
int launch_time_model(slaq_handle* h, double* d_s, double* d_w);
int launch_shard_pick(slaq_handle* h, int pass, long long want);
int launch_shard_pass(slaq_handle* h, int pass, int first_unit);
int launch_shard_count(slaq_handle* h, int first_unit, const long long** d_total);
int launch_shard_finalise(slaq_handle* h, int first_unit, long long ties_before, const long long* d_ties_before,
                          int32_t* d_out_alloc);

}  // namespace slaq
