// A job's predicted reduction as a function of its cores, shared by the kernel that writes the gain
// table and by the selection that works without one: the iteration-time law, the fitted curve in the
// form the gain formulas need, and the gain of the n-th core.
#pragma once

#include <math_constants.h>

#include "slaq_internal.cuh"

namespace slaq {

namespace gaincurve {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ bool finite_d(double v) { return fabs(v) <= 1.7976931348623157e308; }

// Iteration-time law of job j: the fixed one if set, else ordinary least squares of the
// sampled seconds on u = 1/cores from the running sums.  s and w are left untouched if the
// job has neither; returns whether the law can be used (s >= 0, w > 0, finite).
__device__ inline bool time_law(const JobArrays& job, int j, int max_jobs, double& s, double& w) {
    const double s_fix = job.s_set[j], w_fix = job.w_set[j];
    if (finite_d(s_fix) && finite_d(w_fix)) {
        s = s_fix;
        w = w_fix;
    } else {
        const double* tm = job.tm + j;
        const size_t J = (size_t)max_jobs;
        const double cnt = tm[0], su = tm[J], suu = tm[2 * J], st = tm[3 * J], sut = tm[4 * J], stn = tm[5 * J];
        const double umin = tm[6 * J], umax = tm[7 * J];
        if (!(cnt > 0.0)) return false;
        bool fitted = false;
        if (umax > umin) {
            const double den = __dsub_rn(__dmul_rn(cnt, suu), __dmul_rn(su, su));
            const double ww = __ddiv_rn(__dsub_rn(__dmul_rn(cnt, sut), __dmul_rn(su, st)), den);
            const double ss = __ddiv_rn(__dsub_rn(st, __dmul_rn(ww, su)), cnt);
            if (den > 0.0 && finite_d(ww) && finite_d(ss) && ss >= 0.0 && ww > 0.0) {
                s = ss;
                w = ww;
                fitted = true;
            }
        }
        if (!fitted) {   // one core count only, or an unphysical fit: all time is parallel work
            s = 0.0;
            w = __ddiv_rn(stn, cnt);
        }
    }
    return finite_d(s) && finite_d(w) && w > 0.0 && s >= 0.0;
}

// Reciprocal to about one ulp: hardware seed and two Newton steps.
__device__ __forceinline__ double fast_rcp(double q) {
    double x;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(x) : "d"(q));
    double e = fma(-q, x, 1.0);
    x = fma(x, e, x);
    e = fma(-q, x, 1.0);
    return fma(x, e, x);
}

struct Curve {
    int kind;        // 0 family I, 1 family II, 2 linear extrapolation, 3 no gain
    double p0, p1, p2;
    double inv_span, s, w, T;
    double step_scale;   // T w / span: X_n - X_{n-1} = step_scale / ((s n + w)(s (n-1) + w))
};

// Gain of the n-th core.  After an epoch on n cores the job has run m(n) = T n / (s n + w) iterations,
// X_n = m(n) / span in window coordinates.
__device__ inline double raw_gain(const Curve& c, int n) {
    const double den = fma(c.s, (double)n, c.w), denp = fma(c.s, (double)(n - 1), c.w);
    const double inv_den = fast_rcp(den), inv_denp = fast_rcp(denp);
    const double m = c.T * (double)n * inv_den, mp = c.T * (double)(n - 1) * inv_denp;
    const double X = m * c.inv_span, Xp = mp * c.inv_span;
    double gain;
    if (c.kind == 0) {
        // 1/q(Xp) - 1/q(X) = (q(X) - q(Xp)) / (q(X) q(Xp)), q(X) - q(Xp) = (X - Xp)(a (X + Xp) + b)
        const double dX = c.step_scale * inv_den * inv_denp;
        const double q_now = fma(fma(c.p0, X, c.p1), X, c.p2);
        const double q_prev = fma(fma(c.p0, Xp, c.p1), Xp, c.p2);
        const double dq = dX * fma(c.p0, X + Xp, c.p1);
        gain = dq * fast_rcp(q_now * q_prev);
    } else if (c.kind == 1) {
        // e^(alpha - beta Xp) - e^(alpha - beta X) = e^(alpha - beta Xp) (1 - e^(-beta (X - Xp)))
        const double dX = c.step_scale * inv_den * inv_denp;
        gain = exp(fma(-c.p1, Xp, c.p0)) * (-expm1(-c.p1 * dX));
    } else {
        gain = fmin(c.p0 * m, c.p1) - fmin(c.p0 * mp, c.p1);
    }
    return (finite_d(gain) && gain > 0.0) ? gain : 0.0;
}

// The curve of job j for this epoch.  Sets kind 3 (no gain) for jobs that predict nothing; a job
// that could predict but has no usable time law gets status SLAQ_JOB_NO_TIME, which the caller
// records (*no_time).
__device__ inline Curve load_curve(const JobArrays& job, const FitArrays& fit, int j, int max_jobs, double T,
                                   bool* no_time) {
    const int status = fit.status[j];
    const bool active = job.count[j] > 0;
    Curve c;
    c.kind = 3;
    c.T = T;
    c.inv_span = 1.0 / fit.span[j];
    c.s = c.w = c.p0 = c.p1 = c.p2 = c.step_scale = 0.0;
    *no_time = false;
    const bool predicts = status == SLAQ_JOB_FITTED || status == SLAQ_JOB_SHORT || status == SLAQ_JOB_NEW ||
                          status == SLAQ_JOB_FIT_FAILED;
    if (active && status != SLAQ_JOB_NONFINITE && status != SLAQ_JOB_FLAT) {
        if (!time_law(job, j, max_jobs, c.s, c.w)) {
            *no_time = true;
        } else if (predicts) {
            c.p0 = fit.params[4 * (size_t)j];
            c.p1 = fit.params[4 * (size_t)j + 1];
            c.p2 = fit.params[4 * (size_t)j + 2];
            c.kind = status == SLAQ_JOB_FITTED ? (int)fit.family[j] : 2;
            c.step_scale = T * c.w * c.inv_span;
        }
    }
    return c;
}

}  // namespace gaincurve

}  // namespace slaq
