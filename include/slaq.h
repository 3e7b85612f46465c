/*
 * slaq.h - C ABI of the per-epoch scheduling path of a quality-driven scheduler for
 * ML training jobs (Zhang et al., "SLAQ: Quality-Driven Scheduling for Distributed
 * Machine Learning", Design section), as CUDA kernels for one sm_100a GPU.
 *
 * The problem (Design, "Scheduling Based on Quality Improvements"): J jobs run
 * concurrently, each reports one loss value per iteration; every epoch of T seconds
 * the scheduler chooses a_j cores for each job, sum_j a_j <= C, to maximise the total
 * normalised loss reduction  sum_j [Loss_j(a_j, t) - Loss_j(a_j, t+T)].
 * One call of slaq_schedule() runs the paper's three duties for every active job:
 *   - normalise  ("Normalizing Quality Metrics"): change in loss between iterations
 *     over the largest change seen so far;
 *   - predict    ("Predicting Quality Improvement"): exponentially weighted least
 *     squares of f(k) = 1/(a k^2 + b k + c) + d and f(k) = mu^(k-b) + c, the lower
 *     weighted residual wins, then the loss reduction over one epoch for each core
 *     count n = 1..max_cores_per_job, an iteration on n cores taking s + w/n seconds;
 *   - allocate   (the greedy loop of "Scheduling Based on Quality Improvements"): one
 *     core each, then one core at a time to the largest predicted marginal gain, equal
 *     gains to the lowest job id.
 *
 * Conventions
 *   - Every function returns an int status: 0 = SLAQ_OK, < 0 error, > 0 warning.
 *     Nothing throws or aborts.  slaq_last_error() gives a message for the last
 *     non-zero status of a handle.
 *   - "host" pointers are ordinary host memory, "device" pointers are memory of the
 *     GPU that was current when the handle was created.  The caller owns every pointer
 *     it passes and may release it when the call returns, unless stated otherwise.
 *   - The handle owns all scheduler state on the device.  Calls on one handle must not
 *     overlap; work is ordered on the handle's stream (slaq_set_stream).  Functions
 *     that take or fill host buffers return after the stream has finished that work.
 *   - Calls on a handle must be made with the handle's device current (SLAQ_E_ARG otherwise).
 *   - Job ids are 0 .. max_jobs-1.  A job is active from its first loss until removed.
 *   - The library needs a CUDA device: there is no CPU path.
 */
#ifndef SLAQ_H
#define SLAQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct slaq_handle slaq_t;

enum {
    SLAQ_OK = 0,
    SLAQ_E_ARG = -1,        /* null pointer, negative count, duplicate job id, bad key or value */
    SLAQ_E_RANGE = -2,      /* job id outside 0 .. max_jobs-1, or a size beyond what the handle was created for */
    SLAQ_E_NONFINITE = -3,  /* a loss or time that is NaN or infinite */
    SLAQ_E_NOMEM = -4,      /* device or host allocation failed, or the given workspace is too small */
    SLAQ_E_CUDA = -5,       /* a CUDA call failed; the message holds its error string */
    SLAQ_E_TIMEOUT = -6,    /* reserved: no kernel of this library waits on another, so nothing returns it */
    SLAQ_W_OVERSUBSCRIBED = 1, /* fewer cores than active jobs: no one-core floor, cores go to the best first units */
    SLAQ_W_UNDERFILLED = 2     /* more cores than active jobs x max_cores_per_job: every job is at its cap */
};

/* keys of slaq_set_param / slaq_get_param */
enum {
    SLAQ_P_GAMMA = 1,             /* weight base of the fit, point i of H weighs gamma^(H-1-i); default 0.9; (0, 1] */
    SLAQ_P_LM_TRIALS = 2,         /* Levenberg-Marquardt trials per family; default 20; 0 .. 1000 */
    SLAQ_P_MAX_CORES_PER_JOB = 3, /* cap on a_j; default 64; 1 .. what the handle was created for */
    SLAQ_P_MIN_FIT_POINTS = 4,    /* fewer stored points than this use linear extrapolation; default 4; >= 4 */
    SLAQ_P_FIT_SLICE_BYTES = 5,   /* tuning: shared memory one warp of the fit kernel may use (8 KB..200 KB,
                                     default 13,824: sixteen warps per SM); decides how many lanes share a
                                     job; results stay within rounding */
    SLAQ_P_WARM_START = 6,        /* 0 (default) or 1.  The scheduler refits every job at short intervals
                                     (Evaluation, "Scalability and efficiency"); with 1, a family starts from the
                                     parameters the job's last epoch ended with, carried into this epoch's window
                                     coordinates, instead of from its linearised first guess (which it still uses
                                     where there is no earlier fit or the carried point has no finite residual).
                                     The starting point of a job changes only when its history changes, so
                                     slaq_schedule stays repeatable.  Together with a smaller SLAQ_P_LM_TRIALS
                                     this spreads a fit's iterations over the epochs.  The paper does not say how
                                     its fits are started. */
    SLAQ_P_FIT_CLUSTER_JOBS = 7,  /* tuning: with few active jobs the fit gives every job more lanes (up to a whole
                                     warp), so that a small cluster still fills the GPU; the number of lanes is
                                     chosen from the handle's active jobs.  A handle that holds one shard of a
                                     larger cluster is told the cluster's number of active jobs here, so that
                                     every shard makes the choice the undivided cluster would make and the
                                     results agree bit for bit; 0 (default): the handle's own active jobs */
    SLAQ_P_EPOCH_GRAPH = 8,       /* 1: slaq_schedule / slaq_schedule_device replay the epoch's launches as one
                                     CUDA graph once two calls in a row had the same arguments, parameters and
                                     number of active jobs (an epoch of a small cluster is bound by its sixteen
                                     launches); 0: always plain launches; -1 (default): graph for handles
                                     created for at most 20,000 jobs.  Results are the same either way.  Not
                                     used while the handle's stream is itself being captured. */
    SLAQ_P_GAIN_ENVELOPE = 9,     /* 0 (default) or 1.  The greedy loop is exact when every job's predicted reduction
                                     R(n) is concave in its cores n, which a convex fitted curve gives.  Where a fit is
                                     not convex ahead of the newest point (the paper assumes convex losses: footnotes of
                                     "Predicting Quality Improvement"), the marginal gains may rise with n.  0: they
                                     are made non-increasing by a running minimum (never predicts more than the curve).
                                     1: they are replaced by the slopes of the upper concave envelope of the points
                                     (n, R(n)), the smallest concave function nowhere below R, which keeps the curve's
                                     whole drop at max_cores_per_job.  Rows of convex fits are the same either way. */
    SLAQ_P_SELECTION = 10         /* How the greedy loop's threshold is found.  0: every job's gains for n = 1..max
                                     are written to a table first and the selection reads the table.  1: no table -
                                     a job's gains fall with n, so the selection finds what it needs of a row by
                                     binary search over n with the gain in closed form, and evaluates only the gains
                                     that share the threshold's leading digits (the effective gain of the n-th core is
                                     then min(g(1), g(n)), which differs from the table's running minimum by rounding
                                     at most).  Used for the plain prediction only: with SLAQ_P_GAIN_ENVELOPE, with
                                     target-loss hints, and in the sharded steps the table is written.  The gain
                                     rows that slaq_get_predictions returns are then written on request. */
};

/* per-job status written by slaq_schedule (slaq_get_predictions, out_status) */
enum {
    SLAQ_JOB_INACTIVE = -1,  /* no loss reported */
    SLAQ_JOB_FITTED = 0,     /* a curve family was fitted */
    SLAQ_JOB_SHORT = 1,      /* two or three points: linear extrapolation of the normalised reduction */
    SLAQ_JOB_NEW = 2,        /* one point: normalised loss 1, one unit per iteration */
    SLAQ_JOB_FIT_FAILED = 3, /* both families failed numerically: linear extrapolation */
    SLAQ_JOB_FLAT = 4,       /* the loss never fell: no predicted gain */
    SLAQ_JOB_NONFINITE = 5,  /* a stored value is not finite: no predicted gain */
    SLAQ_JOB_NO_TIME = 6     /* no iteration-time model yet: no predicted gain */
};

/* Timings and counts of the last slaq_schedule / slaq_schedule_device call. */
typedef struct slaq_stats {
    float ms_total;        /* device time of the whole epoch */
    float ms_fit;          /* normalise + fit kernel (the three stage times are 0 for an epoch replayed as a CUDA graph) */
    float ms_gain;         /* marginal-gain kernel (with the first selection histogram) */
    float ms_alloc;        /* threshold selection, per-job counts, allocation */
    int32_t launches;      /* kernels launched by the call */
    int32_t active_jobs;
    int64_t cores_handed_out;
    int64_t points;        /* loss values read by the fit kernel */
    int64_t model_sweeps;  /* sum over fitted jobs and families of (history length x sweeps over it) */
    int64_t tie_units;     /* units taken at exactly the threshold gain */
    double threshold;      /* smallest gain that received a core beyond the floor (0 if none) */
    int32_t fitted_jobs;
    int32_t sublinear_wins;
    int32_t exponential_wins;
    int32_t fallback_jobs;
    int32_t nonconvex_fits;  /* fitted jobs whose winning curve is not convex ahead of the newest point (family I with
                                b^2 < a c): their marginal gains rise before they fall, see SLAQ_P_GAIN_ENVELOPE */
} slaq_stats;

/*
 * Create a scheduler for job ids 0..max_jobs-1, each keeping a window of its newest
 * max_hist losses (4 <= max_hist <= 6000) - the loss history that the weighted fit of
 * Design, "Predicting Quality Improvement" works on.
 * Allocates all device state with cudaMalloc on the current device:
 * slaq_workspace_bytes(max_jobs, max_hist, 64) bytes; up to 64 cores per job.
 * *out receives the handle.  The three calls slaq_create, slaq_append_losses and
 * slaq_schedule are the inputs and the output of the problem statement (Design,
 * "Scheduling Based on Quality Improvements": J jobs with their loss histories, the epoch
 * T, the capacity C; a_j out).  Errors: SLAQ_E_ARG, SLAQ_E_NOMEM, SLAQ_E_CUDA.
 */
int slaq_create(int32_t max_jobs, int32_t max_hist, slaq_t** out);

/*
 * Same with an explicit cap on cores per job (1..1024; the paper has no cap).  dev_ws == NULL: the library
 * allocates.  Otherwise the state lives inside device memory the caller owns (for
 * instance a torch tensor): dev_ws must be 256-byte aligned, hold at least
 * slaq_workspace_bytes(max_jobs, max_hist, max_cores_per_job) bytes and outlive the
 * handle.  The library never frees it.
 */
int slaq_create_in(void* dev_ws, size_t bytes, int32_t max_jobs, int32_t max_hist, int32_t max_cores_per_job,
                   slaq_t** out);
/* Bytes slaq_create_in needs for these sizes (0 for sizes outside the limits).  Host arithmetic only. */
size_t slaq_workspace_bytes(int32_t max_jobs, int32_t max_hist, int32_t max_cores_per_job);

/*
 * Release the handle and the device memory it allocated itself (workspace, packed pool, call
 * buffer).  NULL is accepted.  Housekeeping: the paper has no counterpart.
 */
int slaq_destroy(slaq_t* h);

/*
 * Message for the last non-zero status of h (handle-owned storage; valid until the next call
 * on h).  Housekeeping: the paper has no counterpart.
 */
const char* slaq_last_error(const slaq_t* h);

/*
 * cuda_stream is a cudaStream_t (NULL = default stream).  The call waits for the work already
 * queued on the old stream; all later work of h runs on the new one.  Housekeeping: the paper
 * has no counterpart.
 */
int slaq_set_stream(slaq_t* h, void* cuda_stream);

/*
 * Set / read one of the SLAQ_P_* parameters above.  The paper fixes none of them: it asks for
 * an exponentially weighted fit (Design, "Predicting Quality Improvement") without naming the
 * weight base, the solver or its trial count, and it has no cap on cores per job; the defaults
 * are this library's readings.  Errors: SLAQ_E_ARG (unknown key, value outside the range given
 * with the key), SLAQ_E_RANGE (more cores per job than the handle was created for).
 */
int slaq_set_param(slaq_t* h, int key, double value);
int slaq_get_param(const slaq_t* h, int key, double* out_value);

/*
 * One new iteration for each listed job: losses[i] is the loss job_ids[i] reports,
 * iter_times[i] the wall seconds that iteration took.  A job id may appear at most once
 * per call.  The first loss activates the job (iteration index 0).  The call updates the
 * job's window (the oldest point is dropped once max_hist are stored), its iteration
 * index, the largest reduction l_{k-1} - l_k it has shown so far (the denominator of the
 * normalised change in Design, "Normalizing Quality Metrics"), and the sums of its iteration-time
 * law t(n) = s + w/n, the iteration being booked at the job's current core count: its
 * allocation from the last slaq_schedule, 1 before any.  iter_times may be NULL (no time
 * sample).  All pointers are host pointers, n entries each.
 * Errors: SLAQ_E_ARG (n < 0, null, duplicate id), SLAQ_E_RANGE, SLAQ_E_NONFINITE
 * (nothing is applied when an error is returned).
 */
int slaq_append_losses(slaq_t* h, int32_t n, const int32_t* job_ids, const double* losses,
                       const double* iter_times);
/* Same with the core count of each sample given explicitly (cores_used[i] >= 1). */
int slaq_append_losses_ex(slaq_t* h, int32_t n, const int32_t* job_ids, const double* losses,
                          const double* iter_times, const int32_t* cores_used);

/*
 * The same update with all four arrays in device memory (d_iter_times and d_cores_used may be NULL),
 * asynchronous on the handle's stream and without any wait of the host: for trainers that reduce
 * their losses on this GPU.  The host never sees the values, so what slaq_append_losses checks
 * before it applies anything is checked per entry on the device instead: an id outside
 * 0 .. max_jobs-1, a job that has no loss yet (a job's FIRST loss must come through
 * slaq_append_losses or a bulk load, which also count it as active), a loss or time that is not
 * finite, a core count below 1 - such an entry is skipped and the next slaq_schedule returns
 * SLAQ_E_CUDA with a message that says so.  A job id listed twice in one call gives an unspecified
 * order of its two updates.  The arrays must stay valid until the stream has passed the call.
 * Errors: SLAQ_E_ARG (null, n < 0, n > max_jobs, cores without times).  The paper has no counterpart.
 */
int slaq_append_losses_device(slaq_t* h, int32_t n, const int32_t* d_job_ids, const double* d_losses,
                              const double* d_iter_times, const int32_t* d_cores_used);

/*
 * Bulk load: replace the stored window of n_jobs jobs.  Histories are ragged, in CSR
 * form: job job_ids[i] owns losses[offsets[i] .. offsets[i+1]), oldest first; k_last[i]
 * is the iteration index of its newest loss; m_seen[i] (array may be NULL) the largest
 * one-step reduction of its earlier life, joined at scheduling time with the window's
 * own.  If a history is longer than max_hist only its newest max_hist points are kept.
 * Time sums, time models and current core counts of the listed jobs are left as they
 * are.  Host pointers.
 * slaq_load_histories stores each job in its own max_hist-long ring, so later appends
 * extend the window up to max_hist.  slaq_load_histories_packed keeps the rows packed
 * back to back on the device exactly as given (one cudaMalloc of the total size, which
 * replaces any earlier packed load - jobs of an earlier packed load that are not listed
 * again lose their storage with it: they become inactive and forget everything, as after
 * slaq_remove_jobs): a job loaded this way keeps a window of the length it was loaded
 * with, later appends overwrite its oldest point.
 * Errors: SLAQ_E_ARG, SLAQ_E_RANGE, SLAQ_E_NONFINITE, SLAQ_E_NOMEM (the handle is as it
 * was before the call), SLAQ_E_CUDA.
 */
int slaq_load_histories(slaq_t* h, int32_t n_jobs, const int32_t* job_ids, const int64_t* offsets,
                        const double* losses, const int64_t* k_last, const double* m_seen);
int slaq_load_histories_packed(slaq_t* h, int32_t n_jobs, const int32_t* job_ids, const int64_t* offsets,
                               const double* losses, const int64_t* k_last, const double* m_seen);

/*
 * Fix the iteration-time law t(n) = s[i] + w[i]/n of the listed jobs (s >= 0 seconds,
 * w > 0 core-seconds), overriding the estimate from iter_times.  The paper asks for a
 * prediction of a job's progress under a given amount of resources (Design, second duty of
 * the scheduler) without giving the map from cores to iterations; this law is the library's.
 * Host pointers.  Errors: SLAQ_E_ARG (null, duplicate id, s < 0, w <= 0, not finite), SLAQ_E_RANGE.
 */
int slaq_set_time_model(slaq_t* h, int32_t n, const int32_t* job_ids, const double* s, const double* w);

/*
 * Hints of the loss the listed jobs are expected to end at (Conclusion, "Non-convex optimization":
 * users may tell the scheduler their target loss, from earlier trials or published results, so that
 * it does not over-estimate what a job can still gain).  The paper gives no rule; the library's: a
 * job is never predicted to fall below its target, i.e. its predicted reduction over the epoch is
 * capped at max(newest loss - target, 0) in units of its largest reduction seen, for every core
 * count.  targets[i] = NaN removes the hint; infinities are refused (SLAQ_E_NONFINITE).  Hints stay
 * until replaced or the job is removed.  Host pointers.  Errors: SLAQ_E_ARG, SLAQ_E_RANGE.
 */
int slaq_set_target_loss(slaq_t* h, int32_t n, const int32_t* job_ids, const double* targets);

/*
 * Deactivate the listed jobs (finished or cancelled: they leave the set J of running jobs of
 * Design, "Scheduling Based on Quality Improvements") and forget their histories, largest
 * reduction, time sums, time law and fitted curves; a later append starts them anew at
 * iteration 0.  Ids may repeat.  Host pointer.  Errors: SLAQ_E_ARG, SLAQ_E_RANGE.
 */
int slaq_remove_jobs(slaq_t* h, int32_t n, const int32_t* job_ids);

/*
 * One scheduling epoch (Design: normalise, predict, allocate): epoch_seconds = T,
 * total_cores = C.  out_alloc (host, max_jobs entries) receives a_j: 0 for inactive
 * ids, otherwise 1..max_cores_per_job with sum = min(C, active x max_cores_per_job)
 * (0..max when C < active jobs).  Stored histories are not modified: the call can be
 * repeated.  The allocation is remembered as each job's current core count.
 * Returns SLAQ_OK, SLAQ_W_OVERSUBSCRIBED, SLAQ_W_UNDERFILLED, or an error
 * (SLAQ_E_ARG for T <= 0, C < 0 or null; SLAQ_E_CUDA).
 */
int slaq_schedule(slaq_t* h, double epoch_seconds, int64_t total_cores, int32_t* out_alloc);
/*
 * Same, asynchronous on the handle's stream; d_out_alloc is a device pointer (max_jobs entries) or
 * NULL (the result stays in the handle: slaq_get_predictions, the next append's core counts).
 */
int slaq_schedule_device(slaq_t* h, double epoch_seconds, int64_t total_cores, int32_t* d_out_alloc);

/*
 * Results of the last epoch, host pointers, any may be NULL; sizes in entries:
 * out_reduction [max_jobs]: predicted normalised loss reduction at the allocation,
 * Loss_j(a_j, t) - Loss_j(a_j, t+T) in units of the largest reduction seen;
 * out_gain [max_jobs x max_cores_per_job], row-major, gain of the n-th core at [j][n-1];
 * out_family [max_jobs]: 0 = 1/(a x^2 + b x + c) + d, 1 = exp(alpha - beta x) + c, -1 none;
 * out_params [max_jobs x 4]: (a, b, c, d) or (alpha, beta, c, 0) in window coordinates
 * (x = 0 at the newest point, -1 at the oldest, y = loss / out_largest);
 * out_residual [max_jobs x 2]: final weighted residual of each family;
 * out_status [max_jobs]: SLAQ_JOB_*; out_sweeps [max_jobs x 2]: sweeps over the history
 * spent on each family; out_largest [max_jobs]: largest reduction seen.
 */
int slaq_get_predictions(slaq_t* h, double* out_reduction, double* out_gain, int8_t* out_family,
                         double* out_params, double* out_residual, int32_t* out_status, int32_t* out_sweeps,
                         double* out_largest);

/*
 * Normalisation alone, for inspection: for each listed job, oldest first and packed
 * back to back in the order given, the normalised changes (l_{i-1} - l_i) / M (0 for a
 * job's first stored point) and the normalised levels l_i / M; out_offsets [n+1] receives
 * where each job's values start, out_largest [n] the M used.  capacity = entries available
 * in out_changes / out_levels (SLAQ_E_RANGE if too small).  Host pointers; any output may be NULL.
 */
int slaq_get_normalised(slaq_t* h, int32_t n, const int32_t* job_ids, int64_t capacity, int64_t* out_offsets,
                        double* out_changes, double* out_levels, double* out_largest);

/*
 * Iteration-time law in use for every job: the fixed one where slaq_set_time_model gave one,
 * else the least-squares estimate from the appended iteration times (NaN where a job has
 * neither).  Host pointers [max_jobs].  The law itself is the library's (see
 * slaq_set_time_model); the paper has no counterpart.
 */
int slaq_get_time_model(slaq_t* h, double* out_s, double* out_w);

/*
 * The fitted curves as scheduler state (for SLAQ_P_WARM_START: to carry them over a restart,
 * or to inspect them).  Per job: both families' parameters in window coordinates
 * (out_params [max_jobs][8]: family I a, b, c, d, then family II alpha, beta, c, and one unused
 * slot), which of them ended with a finite residual (out_mask [max_jobs], bit 0 family I,
 * bit 1 family II, 0 = no fit), and what the coordinates refer to: the index of the newest
 * iteration at that fit (out_k [max_jobs]), the window span max(H-1, 1) (out_span) and the
 * largest reduction the window was scaled by (out_scale).  slaq_get_fit_state reports the last
 * epoch's end points.  slaq_set_fit_state makes the given entries both the last epoch's record
 * and the starting points of each job's next fit; entries with mask 0 clear a job's.  It
 * returns SLAQ_E_ARG for a mask above 3, a masked entry of a job without losses, or a masked
 * entry whose span or scale is not positive and finite; parameters are not checked (a family
 * whose carried-over point has no finite residual starts from its first guess).  Host pointers.
 * The paper has no counterpart.
 */
int slaq_get_fit_state(slaq_t* h, double* out_params, uint8_t* out_mask, int64_t* out_k, double* out_span,
                       double* out_scale);
int slaq_set_fit_state(slaq_t* h, const double* params, const uint8_t* mask, const int64_t* k, const double* span,
                       const double* scale);

/*
 * Test hook for the allocation step alone (the greedy loop of Design, "Scheduling Based on
 * Quality Improvements", on gains the caller supplies): overwrite the gain rows (host,
 * max_jobs x max_cores_per_job, rows non-increasing, values >= +0) and allocate from
 * them with slaq_allocate_only, which runs only the greedy-equivalent selection and fills
 * out_alloc (host, max_jobs) like slaq_schedule.
 */
int slaq_set_gains(slaq_t* h, const double* gain);
int slaq_allocate_only(slaq_t* h, int64_t total_cores, int32_t* out_alloc);

/*
 * Timings and counts of the last epoch (the struct above).  Diagnostic: the paper reports only
 * the total time of a scheduling decision (Evaluation, "Scalability and efficiency").
 * Errors: SLAQ_E_ARG (null, or no epoch has run yet), SLAQ_E_CUDA.
 */
int slaq_get_stats(slaq_t* h, slaq_stats* out);

/*
 * Checkpoint and resume (the paper has no counterpart: its scheduler lives inside a long-running
 * driver).  slaq_export_state writes everything the handle knows about its jobs into one host
 * blob: per job the stored window (oldest first), the index of its newest iteration, the largest
 * reduction seen, the sums and the fixed value of its iteration-time law, its target-loss hint, its current core count,
 * and both records of its fitted curves (what the last epoch ended with, what the next fit
 * starts from).  Parameters (slaq_set_param) and the stream are not part of it.
 * slaq_export_state_bytes gives the size the blob needs now; capacity below it: SLAQ_E_RANGE.
 * slaq_import_state replaces the whole state of h by a blob's: h must have been created for the
 * same max_jobs and for a max_hist of at least the blob's longest window (SLAQ_E_RANGE
 * otherwise); windows are stored as rings of max_hist slots, also those that the exporting handle
 * held packed (such a job kept the window length it was loaded with; after the import its window
 * grows with later appends up to max_hist).  Apart from that, a handle that imported a blob
 * schedules, appends and warm-starts bit for bit like the handle that exported it, given the same
 * max_hist and parameters.  The blob is plain host memory in this machine's byte order, valid
 * for this library version (SLAQ_E_ARG for anything else, or for sizes that disagree; the losses
 * are checked as in slaq_load_histories).  On an error found while reading the blob's tables the
 * handle is unchanged; after that point a failing import leaves it empty.
 */
int slaq_export_state_bytes(slaq_t* h, size_t* out_bytes);
int slaq_export_state(slaq_t* h, void* out_blob, size_t capacity);
int slaq_import_state(slaq_t* h, const void* blob, size_t bytes);

/*
 * Diagnostic (the paper has no counterpart).  In a library built with -DSLAQ_PHASE_CLOCKS
 * (paper_1802_04819_b200.build.build_variant("clocks")) the fit kernel adds up, over all its
 * warps, the SM cycles a warp spent in each phase of the last epoch's fit; out_cycles (host,
 * 6 entries) receives them: 0 staging and normalisation, 1 first guesses and the sweep at
 * the starting points, 2 solver steps of the trials, 3 sweeps at the trial points with
 * their reductions and accept/reject, 4 winner and record, 5 work queue and statistics.
 * The ordinary library carries no clocks and reports zeros.
 */
int slaq_get_fit_phase_cycles(slaq_t* h, int64_t* out_cycles);

/*
 * One cluster sharded over several GPUs.  The jobs of ONE cluster are split into contiguous
 * blocks of job ids, block r on GPU r (shard r: its own handle, local ids 0..max_jobs-1 in global
 * order), and all shards share the cluster's cores.  Normalise, fit and gains need no exchange.  The
 * greedy loop of "Scheduling Based on Quality Improvements" picks the globally largest gain at every
 * step, so the threshold search needs the SUM over shards of each digit histogram (2048 x uint64 per
 * pass, six passes) and the tie rule (lowest job id first) needs the number of threshold-equal gains in
 * lower shards.  These calls are the steps between which the caller performs that exchange with its
 * collective library (an all-reduce per pass, one all-gather of one integer per shard); every shard
 * must make the same calls in the same order:
 *   slaq_get_active_count                      -> sum over shards = J; floor iff C >= J;
 *                                                 want = min(C, J x max_cores_per_job) - (floor ? J : 0)
 *   slaq_shard_predict(T, floor)               normalise + fit + gains + local histogram of digit 0
 *   for pass = 0..5:
 *       if pass > 0: slaq_shard_pass(pass)     narrow by the bin of digit pass-1, local histogram of digit pass
 *       slaq_shard_histogram(pass, buf, 0)     export; all-reduce(sum) buf over shards;
 *       slaq_shard_histogram(pass, buf, 1)     import the summed histogram
 *       slaq_shard_pick(pass, want)            same bin on every shard
 *   slaq_shard_count(&ties)                    all-gather ties; ties_before = sum over lower shards
 *   slaq_shard_finalise(ties_before, out_alloc)
 * d_hist is device memory of 2048 uint64 owned by the caller; out_alloc is a host array of max_jobs
 * entries.  The result equals slaq_schedule on one handle holding all jobs.  All calls are ordered on
 * the handle's stream; slaq_shard_count and slaq_shard_finalise return after the stream has finished.
 * slaq_shard_count_device / slaq_shard_finalise_device are the same two steps without the host in
 * between: the first leaves the shard's tie count in device memory of the caller (one int64,
 * stream-ordered, no wait), the second reads ties_before from device memory (one int64 that the
 * caller's collective left there, ordered on the handle's stream) - a whole sharded epoch then
 * waits for the device once, when the allocation is copied out.
 */
int slaq_get_active_count(slaq_t* h, int32_t* out_active);
int slaq_shard_predict(slaq_t* h, double epoch_seconds, int32_t with_floor);
int slaq_shard_histogram(slaq_t* h, int32_t pass, uint64_t* d_hist, int32_t import_it);
int slaq_shard_pick(slaq_t* h, int32_t pass, int64_t want);
int slaq_shard_pass(slaq_t* h, int32_t pass);
int slaq_shard_count(slaq_t* h, int64_t* out_local_ties);
int slaq_shard_finalise(slaq_t* h, int64_t ties_before, int32_t* out_alloc);
int slaq_shard_count_device(slaq_t* h, int64_t* d_out_local_ties);
int slaq_shard_finalise_device(slaq_t* h, const int64_t* d_ties_before, int32_t* out_alloc);

/*
 * The allocation step for callers that must not allocate device memory.  (The paper has
 * no counterpart: it is the selection of slaq_allocate_only, packaged so that it touches
 * the allocator nowhere.)
 *
 * Who needs it: a scheduler loop that runs beside other GPU work and cannot afford the
 * device-wide synchronisation that cudaMalloc and cudaFree imply; a plug-in that was
 * handed a fixed memory budget and a stream by its host and is not allowed to grow it;
 * code that runs after start-up in a process whose policy is "no allocation after
 * initialisation".  Such a caller has no handle (creating one allocates), so there is no
 * handle here: inputs and outputs are the caller's device buffers, and the scratch the
 * kernels need (histograms of the threshold search, per-job counts) lives in an array
 * that is part of the library image, about 0.6 MB on every GPU that loads the library,
 * until the process ends.
 *
 * d_gain [n_jobs x max_cores_per_job], row-major device memory: gain of the n-th core of
 * row j at [j][n-1], every row non-increasing, values >= +0; every row is an active job.
 * d_out_alloc [n_jobs] receives a_j (1..max_cores_per_job, sum = min(total_cores,
 * n_jobs x max_cores_per_job); 0..max when total_cores < n_jobs), d_out_reduction
 * [n_jobs] the sum of the row's first a_j gains.  cuda_stream: cudaStream_t or NULL.
 * The call is asynchronous on that stream.  Limits: n_jobs <= 32768,
 * max_cores_per_job <= 1024; beyond them SLAQ_E_RANGE and nothing is launched.
 * Other errors: SLAQ_E_ARG (null pointer, n_jobs < 1, total_cores < 0), SLAQ_E_CUDA.
 * Warnings as slaq_schedule.  No cudaMalloc, cudaFree or other allocating call is made.
 *
 * The first call on each device looks up the device address of the static array (the
 * device that is current at the call); make that first call outside any stream capture.
 * All calls on one device share the array: it still holds the previous call's values,
 * the call clears the parts that must start at zero, and two calls whose kernels overlap
 * on the GPU (different streams, or different host threads without ordering) race on it -
 * run them one after the other.
 */
int slaq_allocate_static(const double* d_gain, int32_t n_jobs, int32_t max_cores_per_job, int64_t total_cores,
                         int32_t* d_out_alloc, double* d_out_reduction, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SLAQ_H */
