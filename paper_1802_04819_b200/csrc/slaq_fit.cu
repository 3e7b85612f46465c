// Normalisation and curve fit.
//
// For every active job: stage the window of stored losses in shared memory, find the largest
// one-step reduction seen so far and scale the window by it ("Normalizing Quality Metrics"),
// then fit both convergence families of "Predicting Quality Improvement",
//     I : f(x) = 1 / (a x^2 + b x + c) + d          II : f(x) = exp(alpha - beta x) + c,
// by exponentially weighted least squares with Levenberg-Marquardt, in window coordinates
// (newest point x = 0, oldest x = -1); the family with the lower weighted residual wins.
//
// Work split.  Jobs are sorted by window length (counting sort, longest first) and cut into
// length classes.  In class c a group of L lanes (L = 2, 4, .. 32: the fewest lanes at which
// the window fits the rows of a warp's shared-memory slice) owns one job (so a warp carries
// 32/L jobs; with few active jobs L is raised so that every warp of the GPU has work).  One
// persistent launch (one block of 16 warps per SM) serves all classes from one work queue,
// longest windows first.  A lane walks its job's points m = l, l + L, l + 2L, ... counted
// from the newest one; both families
// are evaluated in the same sweep over the window; the partial sums of the normal equations
// are reduced over the L lanes with shuffles; the even lanes of a group then run family I's
// solver step for the job and the odd lanes family II's.  All per-job control flow is per
// lane, so the jobs of a warp may be in different phases of the solver.
#include <math_constants.h>

#include <algorithm>

#include "slaq_internal.cuh"
#include "slaq_fit_sweep.cuh"

namespace slaq {

namespace {

// Phase clocks (only in a library built with -DSLAQ_PHASE_CLOCKS): lane 0 of every warp adds up the
// SM cycles it spends in each phase of the fit; the totals go to counters[8..13].
#ifdef SLAQ_PHASE_CLOCKS
#define SLAQ_PHASE_DECL long long ph_[6] = {0, 0, 0, 0, 0, 0}, ph_t_ = clock64()
#define SLAQ_PHASE(i)                      \
    do {                                   \
        const long long now_ = clock64();  \
        ph_[i] += now_ - ph_t_;            \
        ph_t_ = now_;                      \
    } while (0)
#else
#define SLAQ_PHASE_DECL
#define SLAQ_PHASE(i)
#endif

constexpr int kMaxWarpsPerBlock = 16;          // one block per SM: its warps share one copy of the weight table
constexpr size_t kSmemLimit = 226 * 1024;   // shared memory one block may use on sm_100, less the static part
constexpr double kLambda0 = 1e-3, kLambdaMin = 1e-5, kLambdaMax = 1e12;

// Reductions over the L lanes of a group (L a power of two); every lane of the warp takes part.
__device__ __forceinline__ double group_sum(double v, int L) {
    for (int o = L >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double group_max(double v, int L) {
    for (int o = L >> 1; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ double group_min(double v, int L) {
    for (int o = L >> 1; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ int group_and(int v, int L) {
    for (int o = L >> 1; o > 0; o >>= 1) v &= __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ int warp_max_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// One asynchronous copy of a double from global to shared memory (both 8-byte aligned).
__device__ __forceinline__ void copy_async_8(double* dst_shared, const double* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_shared);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(src) : "memory");
}

// Copy the job's window into the lane columns (ring storage: the newest loss sits just before
// `head`).  Returns H, or 0 after flagging storage that cannot be right.
__device__ int stage_window(const JobArrays& job, int j, int h_cap, const Lanes& S, int32_t* err_word) {
    if (j < 0) return 0;
    const double* row = job.row[j];
    const int cap = job.cap[j];
    const int H = job.count[j];
    if (H <= 0) return 0;
    if (H > cap || H > h_cap || row == nullptr) {   // never expected: record and skip the job
        if (S.l == 0) atomicOr(err_word, kErrWindow);
        return 0;
    }
#ifdef SLAQ_DEBUG_BOUNDS
    {   // the ring lies inside one of the pools, and the write position inside the ring
        const bool in_ring = row >= job.ring_lo && row + cap <= job.ring_hi;
        const bool in_packed = job.packed_lo && row >= job.packed_lo && row + cap <= job.packed_hi;
        const int head = job.head[j];
        if (!(in_ring || in_packed) || head < 0 || head >= cap) {
            if (S.l == 0) atomicOr(err_word, kErrStorage);
            return 0;
        }
    }
#endif
    int newest = job.head[j] - 1;
    if (newest < 0) newest += cap;
    // asynchronous 8-byte copies straight into the lane's column: all of a lane's points are in
    // flight at once, and nothing passes through registers
    double* dst = S.y + S.lane;
    for (int m = S.l; m < H; m += S.L, dst += 32) {
        int pos = newest - m;
        pos += pos < 0 ? cap : 0;
        if (index_ok(pos, cap, kErrStorage, err_word) && S.holds(dst)) copy_async_8(dst, row + pos);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    return H;
}

struct Normalised {
    double M;        // largest reduction seen so far
    int status;      // SLAQ_JOB_FITTED here means "usable": M > 0 and everything finite
    double rho;      // weighted mean normalised reduction per iteration (linear extrapolation)
    double ymin, ymax;
};

// Largest reduction over the window joined with what was seen before it; weighted mean
// normalised change; then the window is scaled in place to levels y = l / M.  k_all: uniform
// trip count of the warp.  changes_out (optional, global, indexed oldest first) receives the
// normalised changes.
__device__ Normalised normalise_window(const Lanes& S, int H, int k_all, double m_seen, int min_fit_points,
                                       double* changes_out) {
    Normalised out;
    out.M = CUDART_NAN;
    out.rho = 0.0;
    // Rows of the lane with a point (m < H), and with a point that has an older neighbour (m + 1 < H).  The rows
    // that every lane of the warp has are walked without a test per row (a branch in these loops costs issue
    // slots on every row), the ragged rest with one.
    const int shift = __ffs(S.L) - 1;
    const int rows = H - 1 - S.l >= 0 ? ((H - 1 - S.l) >> shift) + 1 : 0;
    const int rows_nb = H - 2 - S.l >= 0 ? ((H - 2 - S.l) >> shift) + 1 : 0;
    const int full_nb = __reduce_min_sync(kFull, rows_nb);
    const int nb_off = S.l + 1 < S.L ? 1 : 32 - (S.L - 1);   // from a point to its older neighbour
    int fin = 1;
    double dmax = -CUDART_INF;
    {
        const double* yp = S.y + S.lane;
        int k = 0;
#pragma unroll 2
        for (; k < full_nb; ++k, yp += 32) {
            const double v = S.holds(yp) ? *yp : 0.0;
            const double older = S.holds(yp + nb_off) ? yp[nb_off] : 0.0;
            fin &= finite_d(v) ? 1 : 0;
            dmax = fmax(dmax, older - v);
        }
        for (; k < k_all; ++k, yp += 32) {
            if (k < rows) {
                const double v = S.holds(yp) ? *yp : 0.0;
                fin &= finite_d(v) ? 1 : 0;
                if (k < rows_nb) dmax = fmax(dmax, (S.holds(yp + nb_off) ? yp[nb_off] : 0.0) - v);
            }
        }
    }
    fin = group_and(fin, S.L);
    dmax = group_max(dmax, S.L);
    if (H <= 0) {
        out.status = SLAQ_JOB_INACTIVE;
    } else if (!fin || m_seen != m_seen || m_seen == CUDART_INF) {
        out.status = SLAQ_JOB_NONFINITE;
    } else if (H == 1) {
        out.status = SLAQ_JOB_NEW;
    } else {
        out.M = fmax(m_seen, dmax);
        out.status = (out.M > 0.0 && finite_d(out.M)) ? SLAQ_JOB_FITTED : SLAQ_JOB_FLAT;
    }
    const bool usable = out.status == SLAQ_JOB_FITTED;
    const double M = out.M;
    // the normalised changes feed only the linear extrapolation of short windows (and the export)
    const bool want_changes = usable && (H < min_fit_points || changes_out != nullptr);
    double num = 0.0, den = 0.0;
    if (__any_sync(kFull, want_changes)) {
        for (int k = 0; k < k_all; ++k) {
            const int m = S.l + S.L * k;
            if (want_changes && m + 1 < H) {
                const double change = __ddiv_rn(older_neighbour(S, k) - S.level(k), M);
                const double w = S.weight(m);
                num = fma(w, change, num);
                den += w;
                if (changes_out) changes_out[H - 1 - m] = change;
            }
        }
        if (changes_out && usable && S.l == 0) changes_out[0] = 0.0;
        num = group_sum(num, S.L);
        den = group_sum(den, S.L);
        out.rho = fmax(num / den, 0.0);
    }
    __syncwarp();   // all neighbour reads are done before the window is overwritten
    double lo = CUDART_INF, hi = -CUDART_INF;
    {
        // unusable jobs keep their window as it is: they count as lanes without rows
        const int own = usable ? rows : 0;
        const int full = __reduce_min_sync(kFull, own);
        double* yp = S.y + S.lane;
        int k = 0;
#pragma unroll 2
        for (; k < full; ++k, yp += 32) {
            const double y = __ddiv_rn(S.holds(yp) ? *yp : 0.0, M);
            if (S.holds(yp)) *yp = y;
            lo = fmin(lo, y);
            hi = fmax(hi, y);
        }
        for (; k < k_all; ++k, yp += 32) {
            if (k < own) {
                const double y = __ddiv_rn(S.holds(yp) ? *yp : 0.0, M);
                if (S.holds(yp)) *yp = y;
                lo = fmin(lo, y);
                hi = fmax(hi, y);
            }
        }
    }
    out.ymin = group_min(lo, S.L);
    out.ymax = group_max(hi, S.L);
    __syncwarp();
    return out;
}

// Weighted mean normalised change per iteration from the scaled window (used when a window long
// enough for a fit ends without one): sum w (y_{i-1} - y_i) / sum w.
__device__ double mean_change_of_levels(const Lanes& S, int H, int k_all) {
    double num = 0.0, den = 0.0;
    for (int k = 0; k < k_all; ++k) {
        const int m = S.l + S.L * k;
        if (m + 1 < H) {
            const double w = S.weight(m);
            num = fma(w, older_neighbour(S, k) - S.level(k), num);
            den += w;
        }
    }
    num = group_sum(num, S.L);
    den = group_sum(den, S.L);
    return fmax(num / den, 0.0);
}

// ---- small dense algebra: every lane solves its own job's system ----

struct Sym4 {   // symmetric 4x4, upper triangle
    double a00, a01, a02, a03, a11, a12, a13, a22, a23, a33;
};

// Solve B x = r for symmetric positive definite B by the root-free Cholesky factorisation
// B = L D L^T.  False if a pivot is not positive and finite or the solution is not finite.
__device__ bool ldl_solve(const Sym4& B, const double (&r)[4], double (&x)[4]) {
    const double d0 = B.a00;
    const double i0 = fast_rcp(d0);
    const double l10 = B.a01 * i0, l20 = B.a02 * i0, l30 = B.a03 * i0;
    const double d1 = fma(-l10, B.a01, B.a11);
    const double i1 = fast_rcp(d1);
    const double t21 = fma(-l20, B.a01, B.a12), t31 = fma(-l30, B.a01, B.a13);
    const double l21 = t21 * i1, l31 = t31 * i1;
    const double d2 = fma(-l21, t21, fma(-l20, B.a02, B.a22));
    const double i2 = fast_rcp(d2);
    const double t32 = fma(-l31, t21, fma(-l30, B.a02, B.a23));
    const double l32 = t32 * i2;
    const double d3 = fma(-l32, t32, fma(-l31, t31, fma(-l30, B.a03, B.a33)));
    const double i3 = fast_rcp(d3);
    bool ok = d0 > 0.0 && d1 > 0.0 && d2 > 0.0 && d3 > 0.0 && finite_d(d0) && finite_d(d1) && finite_d(d2) &&
              finite_d(d3);
    const double z0 = r[0];
    const double z1 = fma(-l10, z0, r[1]);
    const double z2 = fma(-l21, z1, fma(-l20, z0, r[2]));
    const double z3 = fma(-l32, z2, fma(-l31, z1, fma(-l30, z0, r[3])));
    x[3] = z3 * i3;
    x[2] = fma(-l32, x[3], z2 * i2);
    x[1] = fma(-l31, x[3], fma(-l21, x[2], z1 * i1));
    x[0] = fma(-l30, x[3], fma(-l20, x[2], fma(-l10, x[1], z0 * i0)));
    ok = ok && finite_d(x[0]) && finite_d(x[1]) && finite_d(x[2]) && finite_d(x[3]);
    return ok;
}

// Solver state of ONE family for one job.  The lanes of a group alternate: even lanes carry
// family I, odd lanes family II, so one instruction stream advances both solvers at once.
struct Family {
    double p[4];       // current parameters
    double S;          // weighted residual at p
    double lambda, nu;
    double predicted;  // reduction the quadratic model promises for the trial step
    unsigned was_frozen;
    int sweeps;
    bool ok;           // the starting point was usable
    bool done;         // no further trials
    bool has_trial;    // the running sweep evaluates the trial point
};

// Lower bounds.  Family I (fam 0): a >= 0, b >= 0, c >= 1e-12 keep the curve non-increasing ahead
// of the newest point and its denominator positive there.  Family II (fam 1): beta >= 0.
__device__ __forceinline__ double lower_bound_of(int fam, int a) {
    if (fam == 0) return a == 3 ? -CUDART_INF : (a == 2 ? 1e-12 : 0.0);
    return a == 1 ? 0.0 : -CUDART_INF;
}

// One Levenberg-Marquardt trial up to the point where the model must be evaluated: freeze
// parameters that sit on their bound while the descent direction or the solved step points
// outside (and keep them frozen from then on), solve (A + lambda diag A) step = g over the
// rest, clip the trial point to the bounds, and record the reduction the quadratic model
// promises.  `busy` = this lane has a trial to prepare; the re-solve loop runs while any
// lane of the warp needs another round.  Family II has three parameters: its fourth row is
// a fixed identity row.
__device__ void prepare_trial(Family& F, int fam, const Sym4& A, const double (&g)[4], bool busy, double sum_wy2,
                              double (&trial)[4]) {
    F.has_trial = false;
    if (busy && F.S <= 1e-28 * sum_wy2) {   // residual is zero to rounding
        F.done = true;
        busy = false;
    }
    const int P = fam == 0 ? 4 : 3;
    double lo[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) lo[a] = lower_bound_of(fam, a);
    unsigned frozen = fam == 0 ? 0u : 8u;
#pragma unroll
    for (int a = 0; a < 4; ++a)
        if (a < P && F.p[a] <= lo[a] && (g[a] < 0.0 || ((F.was_frozen >> a) & 1u))) frozen |= 1u << a;
    double step[4] = {0.0, 0.0, 0.0, 0.0};
    bool solved = false, again = busy;
    for (int round = 0; round <= 4; ++round) {
        if (!__any_sync(kFull, again)) break;
        if (again && round <= P) {
            const bool f0 = frozen & 1u, f1 = frozen & 2u, f2 = frozen & 4u, f3 = frozen & 8u;
            Sym4 B;
            B.a00 = f0 ? 1.0 : fma(F.lambda, fmax(A.a00, 1e-300), A.a00);
            B.a11 = f1 ? 1.0 : fma(F.lambda, fmax(A.a11, 1e-300), A.a11);
            B.a22 = f2 ? 1.0 : fma(F.lambda, fmax(A.a22, 1e-300), A.a22);
            B.a33 = f3 ? 1.0 : fma(F.lambda, fmax(A.a33, 1e-300), A.a33);
            B.a01 = (f0 || f1) ? 0.0 : A.a01;
            B.a02 = (f0 || f2) ? 0.0 : A.a02;
            B.a03 = (f0 || f3) ? 0.0 : A.a03;
            B.a12 = (f1 || f2) ? 0.0 : A.a12;
            B.a13 = (f1 || f3) ? 0.0 : A.a13;
            B.a23 = (f2 || f3) ? 0.0 : A.a23;
            const double rhs[4] = {f0 ? 0.0 : g[0], f1 ? 0.0 : g[1], f2 ? 0.0 : g[2], f3 ? 0.0 : g[3]};
            solved = ldl_solve(B, rhs, step);
            unsigned grow = 0;
            if (solved) {
#pragma unroll
                for (int a = 0; a < 4; ++a)
                    if (a < P && !((frozen >> a) & 1u) && F.p[a] <= lo[a] && step[a] < 0.0) grow |= 1u << a;
            }
            frozen |= grow;
            again = solved && grow != 0;
        } else {
            again = false;
        }
    }
    if (!busy) return;
    F.was_frozen |= frozen;
    if (!solved) {   // no step: counts as a rejected trial
        F.lambda = fmin(F.lambda * F.nu, kLambdaMax);
        F.nu *= 2.0;
        return;
    }
    double d[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        trial[a] = a < P ? fmax(F.p[a] + step[a], lo[a]) : 0.0;
        d[a] = trial[a] - F.p[a];
    }
    const double dg = fma(d[0], g[0], fma(d[1], g[1], fma(d[2], g[2], d[3] * g[3])));
    const double Ad0 = fma(A.a00, d[0], fma(A.a01, d[1], fma(A.a02, d[2], A.a03 * d[3])));
    const double Ad1 = fma(A.a01, d[0], fma(A.a11, d[1], fma(A.a12, d[2], A.a13 * d[3])));
    const double Ad2 = fma(A.a02, d[0], fma(A.a12, d[1], fma(A.a22, d[2], A.a23 * d[3])));
    const double Ad3 = fma(A.a03, d[0], fma(A.a13, d[1], fma(A.a23, d[2], A.a33 * d[3])));
    const double dAd = fma(d[0], Ad0, fma(d[1], Ad1, fma(d[2], Ad2, d[3] * Ad3)));
    F.predicted = 2.0 * dg - dAd;
    F.has_trial = true;
    F.sweeps += 1;   // every solved trial costs one sweep over the window
}

// After the sweep at the trial point: accept it only if the residual strictly fell, and move
// the damping by the gain ratio (Madsen, Nielsen, Tingleff 2004).  Returns whether accepted.
__device__ __forceinline__ bool finish_trial(Family& F, const double (&trial)[4], bool ok_trial, double S_trial) {
    if (!F.has_trial) return false;
    F.has_trial = false;
    if (ok_trial && S_trial < F.S) {
        const double S_before = F.S;
#pragma unroll
        for (int a = 0; a < 4; ++a) F.p[a] = trial[a];
        F.S = S_trial;
        const double rho = F.predicted > 0.0 ? (S_before - S_trial) * fast_rcp(F.predicted) : 0.0;
        const double c = 2.0 * rho - 1.0;
        F.lambda *= fmax(1.0 / 3.0, 1.0 - c * c * c);
        F.nu = 2.0;
        F.lambda = fmin(fmax(F.lambda, kLambdaMin), kLambdaMax);
        if (S_before - S_trial <= 1e-14 * S_before) F.done = true;
        return true;
    }
    F.lambda = fmin(F.lambda * F.nu, kLambdaMax);
    F.nu *= 2.0;
    return false;
}

// The sums of the last accepted point live in shared memory between sweeps, one column per job
// and family: after the reduction every lane of a group's parity holds the same sums, so the
// group's first two lanes write them for all.  Every lane of the warp calls this; `keep` says
// whether the lane's family has new sums to park.
__device__ __forceinline__ void park(const Lanes& S, const SweepSums& s, bool keep) {
    if (keep && S.l < 2) {
        const int n = S.park_stride();
#pragma unroll
        for (int k = 0; k < kParked; ++k)
            if (S.holds(S.park + k * n)) S.park[k * n] = s.v[k];
    }
    __syncwarp();
}

// Normal equations A = sum w J J^T, g = sum w J r of the lane's family from the parked sums.
__device__ __forceinline__ void normal_equations(const Lanes& S, int fam, double sw, Sym4& A, double (&g)[4]) {
    const double* c = S.park;
    const int n = S.park_stride();
    if (!S.holds(c) || !S.holds(c + (kParked - 1) * n)) {   // bounds build only: leave the system empty
        A = Sym4{0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
        g[0] = g[1] = g[2] = g[3] = 0.0;
        return;
    }
    if (fam == 0) {
        A.a00 = c[4 * n]; A.a01 = c[3 * n]; A.a02 = c[2 * n]; A.a11 = c[2 * n]; A.a12 = c[1 * n];
        A.a22 = c[0];
        A.a03 = -c[7 * n]; A.a13 = -c[6 * n]; A.a23 = -c[5 * n]; A.a33 = sw;
        g[0] = -c[10 * n]; g[1] = -c[9 * n]; g[2] = -c[8 * n]; g[3] = c[11 * n];
    } else {
        A.a00 = c[0]; A.a01 = -c[1 * n]; A.a11 = c[2 * n]; A.a02 = c[3 * n]; A.a12 = -c[4 * n]; A.a22 = sw;
        A.a03 = 0.0; A.a13 = 0.0; A.a23 = 0.0; A.a33 = 1.0;
        g[0] = c[5 * n]; g[1] = -c[6 * n]; g[2] = c[7 * n]; g[3] = 0.0;
    }
}

struct Moments {
    double sw, swy2;
};

// First guesses.  d0 lies below every level; with the offset fixed at d0, 1/(y - d0) is a
// quadratic in x (family I: weighted linear least squares, or the line through the oldest and
// newest transformed points if that fit is not a decreasing curve with a positive denominator)
// and log(y - d0) is a line in x (family II: weighted linear regression).  needI / needII: the
// job wants that family's guess (a family that starts from last epoch's parameters does not);
// the weight sums in `mom` are always produced.
struct GuessSums {
    double sw, swx, swx2, swx3, swx4, swy2, r0, r1, r2, su, sxu;
};

// One point of the first-guess pass.  kI / kII: the transformed values of family I (1 / (y - d0)) and of
// family II (log(y - d0)) are wanted by some lane of the warp.
template <bool kI, bool kII>
__device__ __forceinline__ void guess_point(const Lanes& S, const double* wp, const double* yp, double md, double inv_span,
                                            double d0, GuessSums& g) {
    const double x = -md * inv_span;
    const double w = S.weight(wp);
    const double y = S.holds(yp) ? *yp : 0.0;
    g.sw += w;
    g.swy2 = fma(w * y, y, g.swy2);
    if (kI || kII) {
        const double wx = w * x, wx2 = wx * x;
        g.swx += wx;
        g.swx2 += wx2;
        g.swx3 = fma(wx2, x, g.swx3);
        g.swx4 = fma(wx2 * x, x, g.swx4);
    }
    if (kI) {
        const double wz = w * fast_rcp(y - d0);
        g.r2 += wz;
        g.r1 = fma(wz, x, g.r1);
        g.r0 = fma(wz * x, x, g.r0);
    }
    if (kII) {
        const double wu = w * log(y - d0);
        g.su += wu;
        g.sxu = fma(wu, x, g.sxu);
    }
}

// The rows every lane of the warp has without a test per row, the ragged rest with one.
template <bool kI, bool kII>
__device__ __forceinline__ void guess_rows(const Lanes& S, int own, int k_all, double inv_span, double d0, GuessSums& g) {
    const int full = __reduce_min_sync(kFull, own);
    const double* yp = S.y + S.lane;
    const double* wp = S.wtab + S.l;
    double md = (double)S.l;
    const double dL = (double)S.L;
    int k = 0;
#pragma unroll 1
    for (; k < full; ++k, md += dL, yp += 32, wp += S.L) guess_point<kI, kII>(S, wp, yp, md, inv_span, d0, g);
#pragma unroll 1
    for (; k < k_all; ++k, md += dL, yp += 32, wp += S.L)
        if (k < own) guess_point<kI, kII>(S, wp, yp, md, inv_span, d0, g);
}

__device__ void first_guesses(const Lanes& S, int H, int k_all, double inv_span, double ymin, double ymax, bool busy,
                              bool needI, bool needII, Moments& mom, double (&pI)[4], double (&pII)[4]) {
    const double d0 = ymax > ymin ? ymin - 0.1 * (ymax - ymin) : ymin - 1e-3 * fmax(fabs(ymin), 1.0);
    GuessSums g = {};
    const int shift = __ffs(S.L) - 1;
    const int own = busy && H - 1 - S.l >= 0 ? ((H - 1 - S.l) >> shift) + 1 : 0;   // the lane's rows
    // a family that no lane of the warp wants a guess for is left out of the pass; a lane that does not want
    // what the warp computes gets sums it does not use
    const bool anyI = __any_sync(kFull, needI), anyII = __any_sync(kFull, needII);
    if (anyI && anyII) {
        guess_rows<true, true>(S, own, k_all, inv_span, d0, g);
    } else {
        if (anyI) guess_rows<true, false>(S, own, k_all, inv_span, d0, g);
        else if (anyII) guess_rows<false, true>(S, own, k_all, inv_span, d0, g);
        else guess_rows<false, false>(S, own, k_all, inv_span, d0, g);
    }
    double sw = g.sw, swx = g.swx, swx2 = g.swx2, swx3 = g.swx3, swx4 = g.swx4, swy2 = g.swy2;
    double r0 = g.r0, r1 = g.r1, r2 = g.r2, su = g.su, sxu = g.sxu;
    for (int o = S.L >> 1; o > 0; o >>= 1) {
        sw += __shfl_xor_sync(kFull, sw, o); swx += __shfl_xor_sync(kFull, swx, o);
        swx2 += __shfl_xor_sync(kFull, swx2, o); swx3 += __shfl_xor_sync(kFull, swx3, o);
        swx4 += __shfl_xor_sync(kFull, swx4, o); swy2 += __shfl_xor_sync(kFull, swy2, o);
        r0 += __shfl_xor_sync(kFull, r0, o); r1 += __shfl_xor_sync(kFull, r1, o);
        r2 += __shfl_xor_sync(kFull, r2, o); su += __shfl_xor_sync(kFull, su, o);
        sxu += __shfl_xor_sync(kFull, sxu, o);
    }
    mom.sw = sw;
    mom.swy2 = swy2;
    // family I
    if (__any_sync(kFull, needI)) {
        Sym4 B;
        B.a00 = swx4; B.a01 = swx3; B.a02 = swx2; B.a11 = swx2; B.a12 = swx; B.a22 = sw;
        B.a03 = B.a13 = B.a23 = 0.0; B.a33 = 1.0;
        const double rhs[4] = {r0, r1, r2, 0.0};
        double sol[4] = {0.0, 0.0, 0.0, 0.0};
        bool good = needI && ldl_solve(B, rhs, sol) && sol[0] >= 0.0 && sol[1] >= 0.0;
        int pos = 1;
        {
            const int mine = needI ? own : 0;
            const int full = __reduce_min_sync(kFull, mine);
            const double dL = (double)S.L;
            double md = (double)S.l;
            int k = 0;
            for (; k < full; ++k, md += dL) {
                const double x = -md * inv_span;
                pos &= fma(fma(sol[0], x, sol[1]), x, sol[2]) > 0.0 ? 1 : 0;
            }
            for (; k < k_all; ++k, md += dL) {
                if (k < mine) {
                    const double x = -md * inv_span;
                    pos &= fma(fma(sol[0], x, sol[1]), x, sol[2]) > 0.0 ? 1 : 0;
                }
            }
        }
        pos = group_and(pos, S.L);
        good = good && pos;
        // the oldest point (m = H - 1) and the newest (m = 0), read from the lanes that own them
        const int m_old = max(H - 1, 0);
        const double* at_old = S.y + (m_old / S.L) * 32 + (S.lane - S.l) + (m_old & (S.L - 1));
        const double y_old = S.holds(at_old) ? *at_old : 0.0;
        const double y_new = S.holds(S.y + S.lane - S.l) ? S.y[S.lane - S.l] : 0.0;
        if (good) {
            pI[0] = sol[0]; pI[1] = sol[1]; pI[2] = sol[2];
        } else {
            const double z_old = 1.0 / (y_old - d0), z_new = 1.0 / (y_new - d0);
            pI[0] = 0.0;
            pI[1] = fmax(z_new - z_old, 0.0);
            pI[2] = z_new;
        }
        pI[3] = d0;
    }
    // family II
    const double den = sw * swx2 - swx * swx;
    const double slope = (sw * sxu - swx * su) / den;
    pII[0] = (su - slope * swx) / sw;
    pII[1] = fmax(-slope, 1e-8);
    pII[2] = d0;
    pII[3] = 0.0;
}

// Last epoch's end points of both families in this epoch's window coordinates.  The curves
// are functions of the iteration index and the raw loss; with x0 = (k - K0)/span0, y0 = l/M0
// then and x = (k - K)/span, y = l/M now, x0 = t + r x and y = sigma y0, where
// t = (K - K0)/span0, r = span/span0, sigma = M0/M, and both families keep their form under
// that substitution.  Clears `wmask` if the stored coordinates cannot be used.
__device__ void carry_over(const FitArrays& fit, const JobArrays& job, int j, double span, double M, unsigned& wmask,
                           double (&pI)[4], double (&pII)[4]) {
    const double span0 = fit.warm_span[j], M0 = fit.warm_scale[j];
    if (!(span0 > 0.0) || !(M0 > 0.0) || !finite_d(M0)) {
        wmask = 0;
        return;
    }
    const double* q = fit.warm_p + 8 * (size_t)j;
    const double t = (double)(job.k_last[j] - fit.warm_k[j]) / span0;
    const double r = span / span0, sigma = M0 / M;
    if (wmask & 1u) {
        const double a = q[0], b = q[1], c = q[2], d = q[3];
        pI[0] = a * r * r / sigma;
        pI[1] = (2.0 * a * t + b) * r / sigma;
        pI[2] = ((a * t + b) * t + c) / sigma;
        pI[3] = sigma * d;
    }
    if (wmask & 2u) {
        pII[0] = q[4] - q[5] * t + log(sigma);
        pII[1] = q[5] * r;
        pII[2] = sigma * q[6];
        pII[3] = 0.0;
    }
}

// The second round of a warm start: the families whose carried-over point had no finite
// residual (`redo`, per lane for its own family) take their first guesses and are swept again.
__device__ __noinline__ void restart_from_first_guesses(const Lanes& S, int fam, int H, int k_all, double inv_span,
                                                        double ymin, double ymax, bool fits, bool redo, double* pI,
                                                        double* pII, SweepSums* sums) {
    const int lane = S.lane;
    const bool redoI = __shfl_sync(kFull, (int)redo, lane & ~1) != 0;
    const bool redoII = __shfl_sync(kFull, (int)redo, lane | 1) != 0;
    Moments mom;
    double gI[4], gII[4], qI[4], qII[4];
    first_guesses(S, H, k_all, inv_span, ymin, ymax, fits, redoI, redoII, mom, gI, gII);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        qI[a] = redoI ? gI[a] : pI[a];
        qII[a] = redoII ? gII[a] : pII[a];
        pI[a] = qI[a];
        pII[a] = qII[a];
    }
    SweepSums again;
    sweep(S, fam, H, k_all, inv_span, qI, redoI, qII, redoII, again);
    if (redo) *sums = again;
}

// Window-length classes, longest first: class c holds the jobs with h_lo[c] < H <= h_hi[c] and
// gives each of them L[c] lanes.  All classes are served by one launch from one work queue
// whose slots are numbered class by class, so the longest windows start first.
struct FitClasses {
    int n;
    int h_lo[kMaxFitClasses], h_hi[kMaxFitClasses], L[kMaxFitClasses];
    int rows;        // sweeps a lane makes at most, over all classes
    int h_max;       // longest window
    int slice;       // doubles of shared memory per warp: parked sums, window rows, one spare row
};

// kWarm: families may start from last epoch's parameters (a separate instantiation, so that the
// plain one carries none of that code).
template <bool kWarm>
__global__ void __launch_bounds__(kMaxWarpsPerBlock * 32, 1)
fit_kernel(JobArrays job, FitArrays fit, const double* __restrict__ g_wtab, const int32_t* __restrict__ order,
           const int32_t* __restrict__ start, FitClasses cls, int lm_trials, int min_fit_points,
           unsigned int* queue, long long* counters, int32_t* err_word) {
    extern __shared__ double smem[];
    __shared__ int slot_base[kMaxFitClasses + 1];
    double* wtab = smem;                                   // [h_max]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double* const slice = smem + cls.h_max + (size_t)warp * cls.slice;   // this warp's: parked sums, then the window rows
    Lanes S;
    S.wtab = wtab;
    S.lane = lane;
    S.slice = slice;
    S.slice_len = cls.slice;
    S.wtab_len = cls.h_max;
    S.err_word = err_word;
    for (int i = threadIdx.x; i < cls.h_max; i += blockDim.x) wtab[i] = g_wtab[i];
    if (threadIdx.x == 0) {   // queue slots of each class: one slot = one warp's worth of jobs
        int run = 0;
        for (int c = 0; c < cls.n; ++c) {
            slot_base[c] = run;
            const int jobs = start[cls.h_lo[c]] - start[cls.h_hi[c]], per_slot = 32 / cls.L[c];
            run += (jobs + per_slot - 1) / per_slot;
        }
        for (int c = cls.n; c <= kMaxFitClasses; ++c) slot_base[c] = run;
    }
    __syncthreads();
    const int fam = lane & 1;             // even lanes solve family I, odd lanes family II
    const int even = lane & ~1, oddl = lane | 1;

    long long n_points = 0, n_sweep_points = 0;
    int n_fit = 0, n_sub = 0, n_exp = 0, n_fallback = 0, n_nonconvex = 0;
    SLAQ_PHASE_DECL;
    for (;;) {
        int slot = 0;
        if (lane == 0) slot = (int)atomicAdd(queue, 1u);
        slot = __shfl_sync(kFull, slot, 0);
        SLAQ_PHASE(5);   // between jobs: statistics, record tail, queue
        if (slot >= slot_base[cls.n]) break;
        int c = 0;
        while (slot >= slot_base[c + 1]) ++c;
        const int L = cls.L[c], h_hi = cls.h_hi[c];
        S.L = L;
        S.l = lane & (L - 1);
        const int G = 32 / L, g = lane / L;
        S.park = slice + 2 * g + (lane & 1);
        S.y = slice + kParked * 2 * G;
        const int last = start[cls.h_lo[c]];
        const int base = start[h_hi] + (slot - slot_base[c]) * G;
        const int idx = base + g;
        int j = idx < last && index_ok(idx, job.max_jobs, kErrJob, err_word) ? order[idx] : -1;
        if (j >= 0 && !index_ok(j, job.max_jobs, kErrJob, err_word)) j = -1;
        __syncwarp();
        const int H = stage_window(job, j, h_hi, S, err_word);
        const int k_all = warp_max_int((H + L - 1) / L);
        __syncwarp();
        const double m_seen = j >= 0 ? job.m_seen[j] : -CUDART_INF;
        const Normalised nz = normalise_window(S, H, k_all, m_seen, min_fit_points, nullptr);
        SLAQ_PHASE(0);   // staging and normalisation

        int status = nz.status, family = -1;
        double p_out[4] = {CUDART_NAN, CUDART_NAN, CUDART_NAN, CUDART_NAN};
        double S_out[2] = {CUDART_INF, CUDART_INF};
        int sweeps_out[2] = {0, 0};
        int ended = 0;   // bit 0 / 1: family I / II ended with a finite residual
        bool any_ended = false;
        double both_out[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};   // both families' end points
        const double span = (double)max(H - 1, 1);
        const bool fits = status == SLAQ_JOB_FITTED && H >= min_fit_points;   // this lane's job gets curves fitted

        if (__any_sync(kFull, fits)) {
            const double inv_span = 1.0 / span;
            Moments mom = {0.0, 0.0};
            Family F = {};
            double pI[4] = {0.0, 0.0, 0.0, 0.0}, pII[4] = {0.0, 0.0, 0.0, 0.0};   // the points the next sweep evaluates
            // Starting points: the first guesses, or (kWarm) last epoch's parameters where the job
            // has some; a carried-over point without a finite residual is dropped for the
            // family's first guess in a second round.
            int spent = 0;
            SweepSums sums = {};
            if (!kWarm) {
                first_guesses(S, H, k_all, inv_span, nz.ymin, nz.ymax, fits, fits, fits, mom, pI, pII);
                sweep(S, fam, H, k_all, inv_span, pI, fits, pII, fits, sums);
            } else {
                unsigned wmask = fits ? fit.warm_mask[j] : 0u;
                if (wmask) carry_over(fit, job, j, span, nz.M, wmask, pI, pII);
                {
                    double gI[4], gII[4];
                    const bool needI = fits && !(wmask & 1u), needII = fits && !(wmask & 2u);
                    first_guesses(S, H, k_all, inv_span, nz.ymin, nz.ymax, fits, needI, needII, mom, gI, gII);
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        if (needI) pI[a] = gI[a];
                        if (needII) pII[a] = gII[a];
                    }
                }
                sweep(S, fam, H, k_all, inv_span, pI, fits, pII, fits, sums);
                const bool redo = fits && ((wmask >> fam) & 1u) && !sums.usable;
                if (__any_sync(kFull, redo)) {   // rare: kept out of line, with its own copies of what it changes
                    double tI[4], tII[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) tI[a] = pI[a], tII[a] = pII[a];
                    SweepSums again = sums;
                    restart_from_first_guesses(S, fam, H, k_all, inv_span, nz.ymin, nz.ymax, fits, redo, tI, tII, &again);
#pragma unroll
                    for (int a = 0; a < 4; ++a) pI[a] = tI[a], pII[a] = tII[a];
                    sums = again;
                    spent = redo ? 1 : 0;
                }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) F.p[a] = fam ? pII[a] : pI[a];
            F.ok = fits && sums.usable;
            F.S = sums.v[fam ? 8 : 12];
            F.lambda = kLambda0;
            F.nu = 2.0;
            F.was_frozen = 0;
            F.sweeps = fits ? 1 + spent : 0;
            F.done = !F.ok;
            F.has_trial = false;
            F.predicted = 0.0;
            park(S, sums, true);
            SLAQ_PHASE(1);   // first guesses and the sweep at the starting points
            for (int t = 0; t < lm_trials; ++t) {
                if (!__any_sync(kFull, !F.done)) break;
                double trial[4] = {0.0, 0.0, 0.0, 0.0};
                {
                    Sym4 A;
                    double gr[4];
                    normal_equations(S, fam, mom.sw, A, gr);
                    prepare_trial(F, fam, A, gr, !F.done, mom.swy2, trial);
                }
                const unsigned trying = __ballot_sync(kFull, F.has_trial);
                SLAQ_PHASE(2);   // solver step of a trial
                if (!trying) continue;
#pragma unroll
                for (int a = 0; a < 4; ++a) {   // each lane of a pair fetches the other family's trial point
                    pI[a] = __shfl_sync(kFull, trial[a], even);
                    pII[a] = __shfl_sync(kFull, trial[a], oddl);
                }
                sweep(S, fam, H, k_all, inv_span, pI, (trying >> even) & 1u, pII, (trying >> oddl) & 1u, sums);
                park(S, sums, finish_trial(F, trial, sums.usable, sums.v[fam ? 8 : 12]));
                SLAQ_PHASE(3);   // sweep at the trial points, reduction, accept or reject
            }
            // both results of the job, in every lane
            const double S_I = __shfl_sync(kFull, F.S, even), S_II = __shfl_sync(kFull, F.S, oddl);
            const bool ok_I = __shfl_sync(kFull, (int)F.ok, even), ok_II = __shfl_sync(kFull, (int)F.ok, oddl);
            sweeps_out[0] = __shfl_sync(kFull, F.sweeps, even);
            sweeps_out[1] = __shfl_sync(kFull, F.sweeps, oddl);
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                pI[a] = __shfl_sync(kFull, F.p[a], even);
                pII[a] = __shfl_sync(kFull, F.p[a], oddl);
            }
            if (fits) {
                if (ok_I) S_out[0] = S_I;
                if (ok_II) S_out[1] = S_II;
                const bool okI = ok_I && finite_d(S_I), okII = ok_II && finite_d(S_II);
                ended = (okI ? 1 : 0) | (okII ? 2 : 0);
                // Kept as a flag of its own: a branch on `ended` placed here was compiled as never taken (nvcc 12.9,
                // also with ptxas -O1) although the same value, stored below, is non-zero; a branch on okI || okII is taken.
                any_ended = okI || okII;
#pragma unroll
                for (int a = 0; a < 4; ++a) both_out[a] = pI[a], both_out[4 + a] = pII[a];
                if (okI && (!okII || S_I <= S_II)) {   // a tie goes to family I
                    family = 0;
#pragma unroll
                    for (int a = 0; a < 4; ++a) p_out[a] = pI[a];
                } else if (okII) {
                    family = 1;
#pragma unroll
                    for (int a = 0; a < 4; ++a) p_out[a] = pII[a];
                }
            } else {
                sweeps_out[0] = sweeps_out[1] = 0;
            }
        }
        const bool fit_failed = fits && family < 0;
        double rho = nz.rho;
        if (__any_sync(kFull, fit_failed)) {   // rare: the whole warp walks its windows once more
            const double from_levels = mean_change_of_levels(S, H, k_all);
            if (fit_failed) rho = from_levels;
        }
        if (status == SLAQ_JOB_NEW) {
            p_out[0] = 1.0;   // one normalised unit per iteration
            p_out[1] = 1.0;   // at most the whole normalised loss
        } else if (status == SLAQ_JOB_FITTED && family < 0) {
            status = H >= min_fit_points ? SLAQ_JOB_FIT_FAILED : SLAQ_JOB_SHORT;
            const double y_new = S.holds(S.y + lane - S.l) ? S.y[lane - S.l] : 0.0;
            p_out[0] = rho;
            p_out[1] = y_new > 0.0 ? y_new : CUDART_INF;
            p_out[2] = p_out[3] = CUDART_NAN;
        }
        if (S.l == 0 && H > 0) {
            n_points += H;
            n_sweep_points += (long long)H * (sweeps_out[0] + sweeps_out[1]);
            if (status == SLAQ_JOB_FITTED) {
                n_fit += 1;
                n_sub += family == 0;
                n_exp += family == 1;
                // 1/(a x^2 + b x + c) is convex for all x >= 0 exactly when b^2 >= a c
                n_nonconvex += family == 0 && p_out[1] * p_out[1] < p_out[0] * p_out[2];
            } else if (status == SLAQ_JOB_SHORT || status == SLAQ_JOB_NEW || status == SLAQ_JOB_FIT_FAILED) {
                n_fallback += 1;
            }
            fit.status[j] = status;
            fit.mask[j] = (uint8_t)ended;
            if (any_ended) {   // what the next epoch may start from
                fit.k_fit[j] = job.k_last[j];
#pragma unroll
                for (int a = 0; a < 8; ++a) fit.both[8 * (size_t)j + a] = both_out[a];
            }
            fit.family[j] = (int8_t)family;
#pragma unroll
            for (int a = 0; a < 4; ++a) fit.params[4 * (size_t)j + a] = p_out[a];
            fit.residual[2 * (size_t)j] = S_out[0];
            fit.residual[2 * (size_t)j + 1] = S_out[1];
            fit.sweeps[2 * (size_t)j] = sweeps_out[0];
            fit.sweeps[2 * (size_t)j + 1] = sweeps_out[1];
            fit.largest[j] = nz.M;
            fit.span[j] = span;
        }
        __syncwarp();
        SLAQ_PHASE(4);   // winner, fallback, the job's record
    }
    // per-warp totals of the statistics
    for (int o = 16; o > 0; o >>= 1) {
        n_points += __shfl_xor_sync(kFull, n_points, o);
        n_sweep_points += __shfl_xor_sync(kFull, n_sweep_points, o);
        n_fit += __shfl_xor_sync(kFull, n_fit, o);
        n_sub += __shfl_xor_sync(kFull, n_sub, o);
        n_exp += __shfl_xor_sync(kFull, n_exp, o);
        n_fallback += __shfl_xor_sync(kFull, n_fallback, o);
        n_nonconvex += __shfl_xor_sync(kFull, n_nonconvex, o);
    }
    if (lane == 0 && n_points > 0) {
        atomicAdd((unsigned long long*)&counters[0], (unsigned long long)n_points);
        atomicAdd((unsigned long long*)&counters[1], (unsigned long long)n_sweep_points);
        atomicAdd((unsigned long long*)&counters[2], (unsigned long long)n_fit);
        atomicAdd((unsigned long long*)&counters[3], (unsigned long long)n_sub);
        atomicAdd((unsigned long long*)&counters[4], (unsigned long long)n_exp);
        atomicAdd((unsigned long long*)&counters[5], (unsigned long long)n_fallback);
        atomicAdd((unsigned long long*)&counters[14], (unsigned long long)n_nonconvex);
    }
#ifdef SLAQ_PHASE_CLOCKS
    if (lane == 0)
        for (int i = 0; i < 6; ++i) atomicAdd((unsigned long long*)&counters[8 + i], (unsigned long long)ph_[i]);
#endif
}

// Normalisation only, written out for inspection: same staging and scaling code as the fit,
// one warp per listed job.
__global__ void __launch_bounds__(kMaxWarpsPerBlock * 32)
normalise_export_kernel(JobArrays job, const int32_t* __restrict__ ids, const int64_t* __restrict__ offsets, int n,
                        const double* __restrict__ g_wtab, int max_hist, double* changes, double* levels,
                        double* largest, int32_t* err_word) {
    extern __shared__ double smem[];
    double* wtab = smem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_cap = (max_hist + 31) / 32;
    Lanes S;
    S.y = smem + max_hist + (size_t)warp * (k_cap + 1) * 32;
    S.slice = S.y;
    S.slice_len = (k_cap + 1) * 32;
    S.wtab_len = max_hist;
    S.err_word = err_word;
    S.park = nullptr;
    S.wtab = wtab;
    S.lane = lane;
    S.L = 32;
    S.l = lane;
    for (int i = threadIdx.x; i < max_hist; i += blockDim.x) wtab[i] = g_wtab[i];
    __syncthreads();
    const int slot = blockIdx.x * (blockDim.x >> 5) + warp;
    if (slot >= n) return;
    int j = ids[slot];
    if (!index_ok(j, job.max_jobs, kErrJob, err_word)) j = -1;
    const int H = stage_window(job, j, max_hist, S, err_word);
    __syncwarp();
    if (H <= 0) {
        if (lane == 0 && largest) largest[slot] = CUDART_NAN;
        return;
    }
    const int64_t base = offsets[slot];
    const int k_all = (H + 31) / 32;
    const Normalised nz = normalise_window(S, H, k_all, job.m_seen[j], 0, changes ? changes + base : nullptr);
    if (lane == 0 && largest) largest[slot] = nz.M;
    for (int k = 0; k < k_all; ++k) {
        const int m = lane + 32 * k;
        if (m < H) {
            if (nz.status != SLAQ_JOB_FITTED) {   // nothing was scaled: report NaN levels and changes
                if (levels) levels[base + H - 1 - m] = CUDART_NAN;
                if (changes) changes[base + H - 1 - m] = CUDART_NAN;
            } else if (levels) {
                levels[base + H - 1 - m] = S.level(k);
            }
        }
    }
}

// ---- work list: job ids sorted by window length, longest first (counting sort) ----

// Jobs per window length.  Many jobs share a length (a full ring), so lengths are first counted
// in shared memory, lanes with equal lengths adding once, and each block then adds its non-zero
// bins to the global table.
constexpr int kSortThreads = 256;
constexpr int kSortJobsPerBlock = 2048;

__device__ __forceinline__ int clamped_length(const int32_t* __restrict__ count, int j, int max_hist) {
    const int H = count[j];
    return H < 0 ? 0 : (H > max_hist ? max_hist : H);
}

__global__ void __launch_bounds__(kSortThreads)
length_count_kernel(const int32_t* __restrict__ count, int max_jobs, int max_hist, int32_t* bucket) {
    extern __shared__ int sh_count[];   // [max_hist + 1]
    for (int i = threadIdx.x; i <= max_hist; i += blockDim.x) sh_count[i] = 0;
    __syncthreads();
    const int lo = blockIdx.x * kSortJobsPerBlock, hi = min(lo + kSortJobsPerBlock, max_jobs);
    for (int base = lo; base < hi; base += blockDim.x) {
        const int j = base + threadIdx.x;
        const bool in = j < hi;
        const int H = in ? clamped_length(count, j, max_hist) : 0;
        const unsigned live = __ballot_sync(kFull, in);
        if (in) {
            const unsigned peers = __match_any_sync(live, H);
            if ((int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&sh_count[H], __popc(peers));
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= max_hist; i += blockDim.x) {
        const int v = sh_count[i];
        if (v) atomicAdd(&bucket[i], v);
    }
}

// start[h] = number of jobs with a window longer than h (h = 0..max_hist); cursor = copy for the scatter.
__global__ void __launch_bounds__(1024) length_scan_kernel(const int32_t* __restrict__ bucket, int max_hist,
                                                           int32_t* start, int32_t* cursor) {
    __shared__ int sh[1024];
    const int t = threadIdx.x, n = max_hist + 1;
    const int per = (n + 1023) / 1024;
    // thread t owns lengths h = max_hist - (t * per + i): it walks from the longest down
    int sum = 0;
    for (int i = 0; i < per; ++i) {
        const int h = max_hist - (t * per + i);
        if (h >= 0) sum += bucket[h];
    }
    sh[t] = sum;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
        const int v = t >= o ? sh[t - o] : 0;
        __syncthreads();
        sh[t] += v;
        __syncthreads();
    }
    int run = sh[t] - sum;   // jobs longer than this thread's first length
    for (int i = 0; i < per; ++i) {
        const int h = max_hist - (t * per + i);
        if (h < 0) break;
        start[h] = run;
        cursor[h] = run;
        run += bucket[h];
    }
}

// Scatter: a block counts its jobs per length again, reserves one contiguous range per non-zero
// length with a single global atomic, and places its jobs inside those ranges.
__global__ void __launch_bounds__(kSortThreads)
length_scatter_kernel(const int32_t* __restrict__ count, int max_jobs, int max_hist, int32_t* cursor,
                      int32_t* order, int32_t* err_word) {
    extern __shared__ int sh_sort[];    // [max_hist + 1] counts, then [max_hist + 1] next free position
    int* sh_count = sh_sort;
    int* sh_next = sh_sort + (max_hist + 1);
    for (int i = threadIdx.x; i <= max_hist; i += blockDim.x) sh_count[i] = 0;
    __syncthreads();
    const int lo = blockIdx.x * kSortJobsPerBlock, hi = min(lo + kSortJobsPerBlock, max_jobs);
    const int lane = threadIdx.x & 31;
    for (int base = lo; base < hi; base += blockDim.x) {
        const int j = base + threadIdx.x;
        const bool in = j < hi;
        const int H = in ? clamped_length(count, j, max_hist) : 0;
        const unsigned live = __ballot_sync(kFull, in);
        if (in) {
            const unsigned peers = __match_any_sync(live, H);
            if ((int)(__ffs(peers) - 1) == lane) atomicAdd(&sh_count[H], __popc(peers));
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= max_hist; i += blockDim.x) {
        const int v = sh_count[i];
        sh_next[i] = v ? atomicAdd(&cursor[i], v) : 0;
    }
    __syncthreads();
    for (int base = lo; base < hi; base += blockDim.x) {
        const int j = base + threadIdx.x;
        const bool in = j < hi;
        const int H = in ? clamped_length(count, j, max_hist) : 0;
        const unsigned live = __ballot_sync(kFull, in);
        if (in) {
            const unsigned peers = __match_any_sync(live, H);
            const int leader = __ffs(peers) - 1;
            int first = 0;
            if (lane == leader) first = atomicAdd(&sh_next[H], __popc(peers));
            first = __shfl_sync(peers, first, leader);
            const int at = first + __popc(peers & ((1u << lane) - 1u));
            if (index_ok(at, max_jobs, kErrJob, err_word)) order[at] = j;
        }
    }
}

size_t fit_smem_bytes(const FitClasses& c, int warps) {
    return sizeof(double) * ((size_t)c.h_max + (size_t)warps * (size_t)c.slice);
}

}  // namespace

int launch_fit(slaq_handle* h) {
    cudaStream_t st = h->stream;
    const int J = h->max_jobs, Hmax = h->max_hist;
    int launches = 0;
    // work list
    {
        const int blocks = (J + kSortJobsPerBlock - 1) / kSortJobsPerBlock;
        const size_t one = sizeof(int) * ((size_t)Hmax + 1);
        cudaFuncSetAttribute(length_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * one));
        length_count_kernel<<<blocks, kSortThreads, one, st>>>(h->job.count, J, Hmax, h->scratch.bucket);
        length_scan_kernel<<<1, 1024, 0, st>>>(h->scratch.bucket, Hmax, h->scratch.start, h->scratch.cursor);
        length_scatter_kernel<<<blocks, kSortThreads, 2 * one, st>>>(h->job.count, J, Hmax, h->scratch.cursor,
                                                                     h->scratch.order, h->err_word);
        launches += 3;
    }
    // Length classes, longest first.  A warp's slice holds the parked sums of its jobs (kParked
    // doubles per job and family), the window rows of 32 points and one spare row; with L lanes
    // per job that leaves rows_at(L) rows.  The class with L = 32, 16, .. 2 lanes per job takes
    // the windows that do not fit at L/2 lanes.  The slice grows if the longest window does not
    // fit at 32 lanes.
    FitClasses cls;
    cls.n = 0;
    cls.rows = 1;
    cls.h_max = Hmax;
    cls.slice = (int)(h->fit_slice_bytes / sizeof(double));
    cls.slice = std::max(cls.slice, kParked * 2 + ((Hmax + 31) / 32 + 1) * 32);
    auto rows_at = [&](int L) { return (cls.slice - kParked * (64 / L)) / 32 - 1; };
    // With few active jobs every job gets more lanes, so that the warps of the GPU all have work:
    // the fewest lanes at which the jobs fill about two slots per warp.
    const long long jobs_for_lanes = h->fit_cluster_jobs > 0 ? (long long)h->fit_cluster_jobs : (long long)h->n_active;
    const long long lanes_wanted = 64LL * h->sm_count * kMaxWarpsPerBlock;
    int L_min = 2;
    while (L_min < 32 && jobs_for_lanes * L_min < lanes_wanted) L_min <<= 1;
    int h_hi = Hmax;
    for (int L = 32; L >= L_min && h_hi > 0; L >>= 1) {
        const int h_lo = L > L_min ? std::max(rows_at(L / 2), 0) * (L / 2) : 0;
        if (h_lo >= h_hi) continue;
        cls.h_lo[cls.n] = h_lo;
        cls.h_hi[cls.n] = h_hi;
        cls.L[cls.n] = L;
        cls.rows = std::max(cls.rows, (h_hi + L - 1) / L);
        ++cls.n;
        h_hi = h_lo;
    }
    for (int c = cls.n; c < kMaxFitClasses; ++c) cls.h_lo[c] = cls.h_hi[c] = 0, cls.L[c] = 32;
    int warps = kMaxWarpsPerBlock;
    while (warps > 1 && fit_smem_bytes(cls, warps) > kSmemLimit) --warps;
    const size_t smem = fit_smem_bytes(cls, warps);
    if (smem > kSmemLimit) {
        h->err = "fit kernel: a window does not fit in shared memory";
        return -1;
    }
    const auto kernel = h->warm_start ? fit_kernel<true> : fit_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        h->err = std::string("fit kernel shared memory: ") + cudaGetErrorString(e);
        return -1;
    }
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, warps * 32, smem);
    if (per_sm < 1) per_sm = 1;
    int blocks = h->sm_count * per_sm;
    const int needed = (J + warps - 1) / warps;   // at least one job per slot
    if (blocks > needed) blocks = needed;
    if (blocks < 1) blocks = 1;
    kernel<<<blocks, warps * 32, smem, st>>>(h->job, h->fit, h->wtab, h->scratch.order, h->scratch.start, cls,
                                            h->lm_trials, h->min_fit_points, h->scratch.ticket + kFitQueueBase,
                                            h->scratch.counters, h->err_word);
    ++launches;
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("fit kernel launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return launches;
}

int launch_normalise_export(slaq_handle* h, int32_t n, const int64_t* d_offsets, double* d_changes,
                            double* d_levels, double* d_largest) {
    if (n <= 0) return 0;
    const int k_cap = (h->max_hist + 31) / 32;
    int warps = kMaxWarpsPerBlock;
    auto bytes = [&](int w) { return sizeof(double) * ((size_t)h->max_hist + (size_t)w * (k_cap + 1) * 32); };
    while (warps > 1 && bytes(warps) > kSmemLimit) --warps;
    const size_t smem = bytes(warps);
    cudaError_t e =
        cudaFuncSetAttribute(normalise_export_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        h->err = std::string("normalise kernel shared memory: ") + cudaGetErrorString(e);
        return -1;
    }
    const int blocks = (n + warps - 1) / warps;
    normalise_export_kernel<<<blocks, warps * 32, smem, h->stream>>>(
        h->job, h->stage.ids, d_offsets, n, h->wtab, h->max_hist, d_changes, d_levels, d_largest, h->err_word);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("normalise kernel launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return 1;
}

}  // namespace slaq
