// CPU oracle for the per-epoch scheduling path of a quality-driven ML-job scheduler.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, sequential, plain restatement of
// what the path computes, written from the paper (Zhang et al., "SLAQ: Quality-Driven
// Scheduling for Distributed Machine Learning", Design section).  It shares no code
// with the CUDA library and must never be called from the product path: only tests,
// the smoke check and the benchmark's CPU-baseline leg load it.
//
// The four steps, in the paper's order:
//   1. normalise   (Design, "Normalizing Quality Metrics"): the change in loss between
//      iterations divided by the largest change seen so far;
//   2. fit         (Design, "Predicting Quality Improvement"): exponentially weighted
//      least squares of f(k) = 1/(a k^2 + b k + c) + d and f(k) = mu^(k-b) + c;
//   3. predict     (Design, "Scheduling Based on Quality Improvements", the objective
//      Loss_j(a_j, t) - Loss_j(a_j, t+T)): loss reduction over one epoch per core count;
//   4. allocate    (same paragraph, the greedy loop): one core each, then one core at a
//      time to the job whose next core buys the largest predicted reduction.
//
// The paper names neither the solver, the weight base, the initial guess nor the
// iteration-time law; the choices below are stated where they are made.
//
// Pins (tests/test_oracle_*.py): normalisation invariants and a hand-worked example;
// the solver on a linear model against closed-form weighted regression; analytic
// Jacobians against central differences; exact recovery of noise-free curves; the
// optimum against an independent library solver; gain telescoping and monotonicity;
// the greedy loop against brute-force enumeration.
// Parity unpinned: the damping schedule (initial value, update factors, bounds), the
// constants of the initial guess, the stopping thresholds and the fallback for jobs
// with fewer than four points have no external reference; their text here is their
// definition.
//
// Arithmetic: IEEE double; sums over history points accumulate in long double.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <queue>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr double kInf = std::numeric_limits<double>::infinity();
constexpr double kNaN = std::numeric_limits<double>::quiet_NaN();

// Per-job status codes reported beside the fit.
enum JobStatus : int32_t {
    ST_INACTIVE = -1,   // no loss reported yet
    ST_FITTED = 0,      // a curve family was fitted
    ST_SHORT = 1,       // two or three points: linear extrapolation
    ST_NEW = 2,         // one point: a new job's normalised loss is 1
    ST_FIT_FAILED = 3,  // both families failed: linear extrapolation
    ST_FLAT = 4,        // the loss never fell: no predicted gain
    ST_NONFINITE = 5,   // a stored loss is not finite: no predicted gain
    ST_NO_TIME = 6      // no iteration-time model: no predicted gain
};

struct Settings {
    double gamma = 0.9;      // weight base: newest point weighs 1, each older point gamma times less
    int lm_trials = 20;      // damped Gauss-Newton trials per family
    int min_fit_points = 4;  // fewer points than this take the linear extrapolation
};

// ---------------------------------------------------------------------------------
// Step 1.  Normalisation (Design, "Normalizing Quality Metrics").
// delta_i = l_{i-1} - l_i is the reduction of iteration i; M is the largest reduction
// the job has shown so far (its whole life: m_seen carries what the stored window no
// longer holds); the normalised change is delta_i / M and the normalised level l_i / M.
// ---------------------------------------------------------------------------------
double largest_reduction(const double* loss, int64_t H, double m_seen) {
    double M = m_seen;  // -inf when nothing was seen before the window
    for (int64_t i = 1; i < H; ++i) {
        const double delta = loss[i - 1] - loss[i];
        if (delta > M) M = delta;
    }
    return M;
}

bool all_finite(const double* v, int64_t n) {
    for (int64_t i = 0; i < n; ++i)
        if (!std::isfinite(v[i])) return false;
    return true;
}

// ---------------------------------------------------------------------------------
// Step 2.  Weighted least-squares fit (Design, "Predicting Quality Improvement").
// Coordinates: the newest stored point sits at x = 0, the oldest at x = -1, the future
// at x > 0: x_i = (i - (H-1)) / (H-1).  Both families are closed under affine maps of k
// and under scaling of the loss, so fitting y(x) is the same model class as fitting
// l(k).  Weights w_i = gamma^(H-1-i): recent iterations count more.
// ---------------------------------------------------------------------------------
struct FitData {
    int64_t H = 0;
    double span = 1.0;
    std::vector<double> x, y, w;
    double sum_wy2 = 0.0;
};

// Family I: f(x) = 1 / (a x^2 + b x + c) + d, parameters (a, b, c, d).
struct Sublinear {
    static constexpr int P = 4;
    // value and partial derivatives at x; false when the denominator is not positive
    static bool eval(const double* p, double x, double* f, double* J) {
        const double q = p[0] * x * x + p[1] * x + p[2];
        if (!(q > 0.0)) return false;
        const double inv = 1.0 / q;
        *f = inv + p[3];
        if (J) {
            const double dq = -inv * inv;  // d(1/q)/dq
            J[0] = dq * x * x;
            J[1] = dq * x;
            J[2] = dq;
            J[3] = 1.0;
        }
        return true;
    }
    // lower bounds: keep the curve decreasing ahead of the newest point and its denominator positive there
    static double lower(int a) {
        const double lo[4] = {0.0, 0.0, 1e-12, -kInf};
        return lo[a];
    }
};

// Family II: f(x) = exp(alpha - beta x) + c, parameters (alpha, beta, c);
// mu^(k - b) + c with mu = exp(-beta / (H-1)).
struct Exponential {
    static constexpr int P = 3;
    static bool eval(const double* p, double x, double* f, double* J) {
        const double e = std::exp(p[0] - p[1] * x);
        *f = e + p[2];
        if (J) {
            J[0] = e;
            J[1] = -x * e;
            J[2] = 1.0;
        }
        return true;
    }
    static double lower(int a) { return a == 1 ? 0.0 : -kInf; }  // beta >= 0: never an increasing curve
};

// Test-only straight line f = p0 + p1 x: with it the solver below must reproduce
// closed-form weighted linear regression.
struct Line {
    static constexpr int P = 2;
    static bool eval(const double* p, double x, double* f, double* J) {
        *f = p[0] + p[1] * x;
        if (J) {
            J[0] = 1.0;
            J[1] = x;
        }
        return true;
    }
    static double lower(int) { return -kInf; }
};

// S = sum w r^2, A = sum w J J^T, g = sum w J r with r = y - f.  Returns false (and
// S = +inf) when the model is undefined at a point or a sum is not finite.
template <class M>
bool normal_equations(const double* p, const FitData& D, double A[4][4], double g[4], double* S) {
    constexpr int P = M::P;
    long double accA[4][4] = {}, accg[4] = {}, accS = 0.0L;
    for (int64_t i = 0; i < D.H; ++i) {
        double f, J[4];
        if (!M::eval(p, D.x[i], &f, J)) {
            *S = kInf;
            return false;
        }
        const double r = D.y[i] - f;
        const long double w = D.w[i];
        accS += w * (long double)r * r;
        for (int a = 0; a < P; ++a) {
            accg[a] += w * (long double)J[a] * r;
            for (int b = 0; b <= a; ++b) accA[a][b] += w * (long double)J[a] * J[b];
        }
    }
    *S = (double)accS;
    bool ok = std::isfinite(*S);
    for (int a = 0; a < P; ++a) {
        g[a] = (double)accg[a];
        ok = ok && std::isfinite(g[a]);
        for (int b = 0; b <= a; ++b) {
            A[a][b] = A[b][a] = (double)accA[a][b];
            ok = ok && std::isfinite(A[a][b]);
        }
    }
    if (!ok) *S = kInf;
    return ok;
}

template <class M>
double cost(const double* p, const FitData& D) {
    for (int a = 0; a < M::P; ++a)
        if (!std::isfinite(p[a])) return kInf;
    long double accS = 0.0L;
    for (int64_t i = 0; i < D.H; ++i) {
        double f;
        if (!M::eval(p, D.x[i], &f, nullptr)) return kInf;
        const double r = D.y[i] - f;
        accS += (long double)D.w[i] * r * r;
    }
    const double S = (double)accS;
    return std::isfinite(S) ? S : kInf;
}

// Solve B d = g for symmetric positive definite B (n <= 4) by Cholesky B = L L^T.
bool cholesky_solve(int n, const double B[4][4], const double* g, double* d) {
    double L[4][4] = {};
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j <= i; ++j) {
            double sum = B[i][j];
            for (int k = 0; k < j; ++k) sum -= L[i][k] * L[j][k];
            if (i == j) {
                if (!(sum > 0.0) || !std::isfinite(sum)) return false;
                L[i][i] = std::sqrt(sum);
            } else {
                L[i][j] = sum / L[j][j];
            }
        }
    }
    double z[4];
    for (int i = 0; i < n; ++i) {
        double sum = g[i];
        for (int k = 0; k < i; ++k) sum -= L[i][k] * z[k];
        z[i] = sum / L[i][i];
    }
    for (int i = n - 1; i >= 0; --i) {
        double sum = z[i];
        for (int k = i + 1; k < n; ++k) sum -= L[k][i] * d[k];
        d[i] = sum / L[i][i];
    }
    for (int i = 0; i < n; ++i)
        if (!std::isfinite(d[i])) return false;
    return true;
}

struct LmOutcome {
    bool ok = false;   // the starting point was feasible and finite
    double S = kInf;   // final weighted residual sum
    int evals = 0;     // model sweeps over the history (start + one per solved trial)
    int accepted = 0;
};

// Levenberg-Marquardt with Marquardt's diagonal scaling and the gain-ratio damping update
// of Madsen, Nielsen and Tingleff ("Methods for non-linear least squares problems", 2004).
// A fixed number of trials.  Each trial
//   - freezes every parameter that sits on its lower bound while the descent direction
//     (g_a < 0) or the solved step points outside, solves (A + lambda diag(A)) step = g
//     over the rest (again after each freeze) and clips the trial point to the bounds;
//     a parameter once frozen is released only by leaving its bound, which a frozen
//     parameter never does: a tiny gradient at a constrained stationary point is all
//     rounding noise, and releasing on its sign would make the result depend on it;
//   - accepts the trial point only if the weighted residual strictly falls;
//   - accepted: lambda *= max(1/3, 1 - (2 rho - 1)^3), rho = actual / predicted reduction,
//     and the rejection factor returns to 2; rejected: lambda *= nu, nu *= 2;
//     lambda stays within [lambda_min, lambda_max].
// Stops early once the residual is zero to rounding or an accepted step no longer
// reduces it beyond 1e-14 of its value.
constexpr double kLambdaMin = 1e-5;
constexpr double kLambdaMax = 1e12;

template <class M>
LmOutcome levenberg_marquardt(double* p, const FitData& D, int trials, double lambda0) {
    constexpr int P = M::P;
    LmOutcome out;
    double A[4][4], g[4], S;
    out.evals = 1;
    if (!normal_equations<M>(p, D, A, g, &S)) return out;
    out.ok = true;
    double lambda = lambda0, nu = 2.0;
    bool was_frozen[4] = {false, false, false, false};
    for (int t = 0; t < trials; ++t) {
        if (S <= 1e-28 * D.sum_wy2) break;
        double B[4][4], rhs[4], step[4], trial[4];
        bool frozen[4];
        for (int a = 0; a < P; ++a) frozen[a] = p[a] <= M::lower(a) && (g[a] < 0.0 || was_frozen[a]);
        bool solved = false;
        for (int round = 0; round <= P; ++round) {
            for (int a = 0; a < P; ++a) {
                for (int b = 0; b < P; ++b) B[a][b] = (frozen[a] || frozen[b]) ? 0.0 : A[a][b];
                B[a][a] = frozen[a] ? 1.0 : A[a][a] + lambda * std::max(A[a][a], 1e-300);
                rhs[a] = frozen[a] ? 0.0 : g[a];
            }
            solved = cholesky_solve(P, B, rhs, step);
            if (!solved) break;
            // a parameter on its bound that the step would push outside joins the frozen set
            bool grew = false;
            for (int a = 0; a < P; ++a)
                if (!frozen[a] && p[a] <= M::lower(a) && step[a] < 0.0) {
                    frozen[a] = true;
                    grew = true;
                }
            if (!grew) break;
        }
        for (int a = 0; a < P; ++a) was_frozen[a] = was_frozen[a] || frozen[a];
        double S_trial = kInf, predicted = 0.0;
        if (solved) {
            for (int a = 0; a < P; ++a) trial[a] = std::max(p[a] + step[a], M::lower(a));
            S_trial = cost<M>(trial, D);
            out.evals += 1;
            // reduction the local quadratic model promises for the step actually taken
            double d[4], dg = 0.0, dAd = 0.0;
            for (int a = 0; a < P; ++a) d[a] = trial[a] - p[a];
            for (int a = 0; a < P; ++a) {
                dg += d[a] * g[a];
                for (int b = 0; b < P; ++b) dAd += d[a] * A[a][b] * d[b];
            }
            predicted = 2.0 * dg - dAd;
        }
        bool accepted = false;
        if (S_trial < S) {
            const double S_before = S;
            double A2[4][4], g2[4], S2;
            if (normal_equations<M>(trial, D, A2, g2, &S2)) {
                accepted = true;
                for (int a = 0; a < P; ++a) {
                    p[a] = trial[a];
                    g[a] = g2[a];
                    for (int b = 0; b < P; ++b) A[a][b] = A2[a][b];
                }
                S = S2;
                out.accepted += 1;
                const double rho = predicted > 0.0 ? (S_before - S) / predicted : 0.0;
                const double c = 2.0 * rho - 1.0;
                lambda *= std::max(1.0 / 3.0, 1.0 - c * c * c);
                nu = 2.0;
                lambda = std::min(std::max(lambda, kLambdaMin), kLambdaMax);
                if (S_before - S <= 1e-14 * S_before) break;
            }
        }
        if (!accepted) {
            lambda = std::min(lambda * nu, kLambdaMax);
            nu *= 2.0;
        }
    }
    out.S = S;
    return out;
}

// Offset below every level, used to linearise both families for their first guess.
double floor_guess(const FitData& D) {
    double lo = D.y[0], hi = D.y[0];
    for (int64_t i = 1; i < D.H; ++i) {
        lo = std::min(lo, D.y[i]);
        hi = std::max(hi, D.y[i]);
    }
    if (hi > lo) return lo - 0.1 * (hi - lo);
    return lo - 1e-3 * std::max(std::fabs(lo), 1.0);
}

// Family I start: with d fixed at the floor guess, 1/(y - d) is a quadratic in x;
// fit it by weighted linear least squares.
void init_sublinear(const FitData& D, double* p) {
    const double d0 = floor_guess(D);
    const int64_t H = D.H;
    std::vector<double> z(H);
    for (int64_t i = 0; i < H; ++i) z[i] = 1.0 / (D.y[i] - d0);
    long double N[3][3] = {}, rhs[3] = {};
    for (int64_t i = 0; i < H; ++i) {
        const double phi[3] = {D.x[i] * D.x[i], D.x[i], 1.0};
        for (int a = 0; a < 3; ++a) {
            rhs[a] += (long double)D.w[i] * phi[a] * z[i];
            for (int b = 0; b < 3; ++b) N[a][b] += (long double)D.w[i] * phi[a] * phi[b];
        }
    }
    double B[4][4] = {}, r[4] = {}, sol[4] = {};
    for (int a = 0; a < 3; ++a) {
        r[a] = (double)rhs[a];
        for (int b = 0; b < 3; ++b) B[a][b] = (double)N[a][b];
    }
    bool good = cholesky_solve(3, B, r, sol) && sol[0] >= 0.0 && sol[1] >= 0.0;
    if (good) {
        for (int64_t i = 0; i < H && good; ++i) {
            const double q = sol[0] * D.x[i] * D.x[i] + sol[1] * D.x[i] + sol[2];
            good = q > 0.0;
        }
    }
    if (good) {
        p[0] = sol[0];
        p[1] = sol[1];
        p[2] = sol[2];
    } else {  // straight line through the oldest and newest transformed points
        p[0] = 0.0;
        p[1] = std::max(z[H - 1] - z[0], 0.0);
        p[2] = z[H - 1];
    }
    p[3] = d0;
}

// Family II start: with c fixed at the floor guess, ln(y - c) is a line in x.
void init_exponential(const FitData& D, double* p) {
    const double d0 = floor_guess(D);
    long double sw = 0, swx = 0, swxx = 0, swu = 0, swxu = 0;
    for (int64_t i = 0; i < D.H; ++i) {
        const double u = std::log(D.y[i] - d0);
        const long double w = D.w[i], x = D.x[i];
        sw += w;
        swx += w * x;
        swxx += w * x * x;
        swu += w * u;
        swxu += w * x * u;
    }
    const double den = (double)(sw * swxx - swx * swx);
    const double slope = (double)(sw * swxu - swx * swu) / den;
    const double intercept = (double)((swu - (long double)slope * swx) / sw);
    p[0] = intercept;
    p[1] = std::max(-slope, 1e-8);
    p[2] = d0;
    p[3] = 0.0;
}

FitData make_fit_data(const double* loss, int64_t H, double M, double gamma) {
    FitData D;
    D.H = H;
    D.span = (double)std::max<int64_t>(H - 1, 1);
    D.x.resize(H);
    D.y.resize(H);
    D.w.resize(H);
    long double swy2 = 0;
    for (int64_t i = 0; i < H; ++i) {
        D.x[i] = (double)(i - (H - 1)) / D.span;
        D.y[i] = loss[i] / M;
        D.w[i] = std::pow(gamma, (double)(H - 1 - i));
        swy2 += (long double)D.w[i] * D.y[i] * D.y[i];
    }
    D.sum_wy2 = (double)swy2;
    return D;
}

// ---------------------------------------------------------------------------------
// Warm start (Evaluation, "Scalability and efficiency": the scheduler reruns every few
// seconds and keeps rebalancing): a scheduler that refits that often may start
// each family from the parameters it found last epoch instead of from the linearised
// first guess.  The paper does not say how its fits are started; this is this
// implementation's rule.  The fitted curve is a function of the iteration index k and
// the raw loss, but its parameters are kept in window coordinates, and those move from
// epoch to epoch: with x0 = (k - K0)/span0 and y0 = l/M0 last epoch, x = (k - K)/span and
// y = l/M now,
//     x0 = t + r x,  t = (K - K0)/span0,  r = span/span0,      y = sigma y0,  sigma = M0/M.
// Substituting into either family gives the same curve in the new coordinates.
// ---------------------------------------------------------------------------------
struct WarmStart {
    uint8_t valid = 0;   // bit 0: family I parameters present, bit 1: family II
    double pI[4] = {kNaN, kNaN, kNaN, kNaN};
    double pII[4] = {kNaN, kNaN, kNaN, kNaN};
    int64_t K = 0;       // index of the newest iteration when the parameters were fitted
    double span = 1.0;   // their window span
    double M = kNaN;     // their scale
};

// 1/(a x0^2 + b x0 + c) + d with x0 = t + r x, times sigma.
void carry_sublinear(const double* p, double t, double r, double sigma, double* out) {
    const double a = p[0], b = p[1], c = p[2], d = p[3];
    out[0] = a * r * r / sigma;
    out[1] = (2.0 * a * t + b) * r / sigma;
    out[2] = ((a * t + b) * t + c) / sigma;
    out[3] = sigma * d;
}

// (exp(alpha - beta x0) + c) sigma with x0 = t + r x.
void carry_exponential(const double* p, double t, double r, double sigma, double* out) {
    out[0] = p[0] - p[1] * t + std::log(sigma);
    out[1] = p[1] * r;
    out[2] = sigma * p[2];
    out[3] = 0.0;
}

struct JobFit {
    uint8_t fitted_mask = 0;       // bit 0 / 1: family I / II ended with a finite residual
    double both[8] = {kNaN, kNaN, kNaN, kNaN, kNaN, kNaN, kNaN, kNaN};   // final parameters of I then II
    int32_t status = ST_INACTIVE;
    int8_t family = -1;            // 0 = sublinear, 1 = exponential, -1 = none
    double params[4] = {kNaN, kNaN, kNaN, kNaN};
    double S[2] = {kInf, kInf};    // final weighted residual of each family
    int32_t evals[2] = {0, 0};     // history sweeps spent on each family
    double M = kNaN;               // largest reduction seen
    double rho = 0.0;              // linear extrapolation: normalised reduction per iteration
    double r_cap = kInf;           // linear extrapolation: cannot reduce more than what is left
    double span = 1.0;
};

// Steps 1 and 2 for one job.  With `warm` (and K, the index of the newest iteration), a
// family whose carried-over parameters give a finite residual starts from them; otherwise,
// and always without `warm`, it starts from its first guess.
JobFit fit_job(const double* loss, int64_t H, double m_seen, const Settings& cfg, const WarmStart* warm = nullptr,
               int64_t K = 0) {
    JobFit out;
    if (H <= 0) return out;
    if (!all_finite(loss, H) || std::isnan(m_seen) || m_seen == kInf) {
        out.status = ST_NONFINITE;
        return out;
    }
    out.span = (double)std::max<int64_t>(H - 1, 1);
    if (H == 1) {
        // A job that has reported one loss: its normalised loss is 1 and its first
        // change is by definition the largest seen, i.e. one unit per iteration.
        out.status = ST_NEW;
        out.rho = 1.0;
        out.r_cap = 1.0;
        return out;
    }
    const double M = largest_reduction(loss, H, m_seen);
    out.M = M;
    if (!(M > 0.0) || !std::isfinite(M)) {
        out.status = ST_FLAT;
        return out;
    }
    const FitData D = make_fit_data(loss, H, M, cfg.gamma);

    bool fitted = false;
    if (H >= cfg.min_fit_points) {
        double pI[4], pII[4];
        LmOutcome rI, rII;
        int spentI = 0, spentII = 0;   // the sweep of a carried-over start that was not usable
        bool startedI = false, startedII = false;
        if (warm && warm->valid && warm->span > 0.0 && warm->M > 0.0 && std::isfinite(warm->M)) {
            const double t = (double)(K - warm->K) / warm->span;
            const double r = D.span / warm->span;
            const double sigma = warm->M / M;
            if (warm->valid & 1) {
                carry_sublinear(warm->pI, t, r, sigma, pI);
                rI = levenberg_marquardt<Sublinear>(pI, D, cfg.lm_trials, 1e-3);
                startedI = rI.ok;
                spentI = startedI ? 0 : 1;
            }
            if (warm->valid & 2) {
                carry_exponential(warm->pII, t, r, sigma, pII);
                rII = levenberg_marquardt<Exponential>(pII, D, cfg.lm_trials, 1e-3);
                startedII = rII.ok;
                spentII = startedII ? 0 : 1;
            }
        }
        if (!startedI) {
            init_sublinear(D, pI);
            rI = levenberg_marquardt<Sublinear>(pI, D, cfg.lm_trials, 1e-3);
        }
        if (!startedII) {
            init_exponential(D, pII);
            rII = levenberg_marquardt<Exponential>(pII, D, cfg.lm_trials, 1e-3);
        }
        out.evals[0] = rI.evals + spentI;
        out.evals[1] = rII.evals + spentII;
        if (rI.ok && std::isfinite(rI.S)) {
            out.fitted_mask |= 1;
            std::memcpy(out.both, pI, sizeof pI);
        }
        if (rII.ok && std::isfinite(rII.S)) {
            out.fitted_mask |= 2;
            std::memcpy(out.both + 4, pII, sizeof pII);
        }
        if (rI.ok) out.S[0] = rI.S;
        if (rII.ok) out.S[1] = rII.S;
        const bool okI = rI.ok && std::isfinite(rI.S);
        const bool okII = rII.ok && std::isfinite(rII.S);
        if (okI && (!okII || rI.S <= rII.S)) {  // lower weighted residual wins; a tie goes to family I
            out.family = 0;
            std::memcpy(out.params, pI, sizeof pI);
            fitted = true;
        } else if (okII) {
            out.family = 1;
            std::memcpy(out.params, pII, sizeof pII);
            fitted = true;
        }
    }
    if (fitted) {
        out.status = ST_FITTED;
        return out;
    }
    // Linear extrapolation: weighted mean of the normalised reductions per iteration,
    // never negative, and never more than the whole remaining normalised loss.
    long double num = 0, den = 0;
    for (int64_t i = 1; i < H; ++i) {
        const double dnorm = (loss[i - 1] - loss[i]) / M;
        num += (long double)D.w[i] * dnorm;
        den += (long double)D.w[i];
    }
    out.rho = std::max((double)(num / den), 0.0);
    out.r_cap = D.y[H - 1] > 0.0 ? D.y[H - 1] : kInf;
    out.status = (H >= cfg.min_fit_points) ? ST_FIT_FAILED : ST_SHORT;
    return out;
}

// ---------------------------------------------------------------------------------
// Step 3.  Predicted loss reduction over one epoch as a function of the core count
// (the objective's Loss_j(a_j, t) - Loss_j(a_j, t+T)).  The paper leaves the map from
// cores to iterations open; here an iteration on n cores takes t(n) = s + w/n seconds,
// so an epoch of T seconds runs m(n) = T n / (s n + w) iterations (real-valued).
// R(n) = f(0) - f(m(n)/span) with f the fitted curve, so R(0) = 0.  The marginal gain
// of the n-th core is g(n) = R(n) - R(n-1), evaluated in a form without cancellation,
// clamped to +0 where it is not a positive finite number and forced non-increasing in n.
// ---------------------------------------------------------------------------------
//
// Two options, both off unless asked for:
// envelope - where the fitted curve is not convex ahead of the newest point, R(n) is not concave
//   and its differences may rise with n.  The default makes the row non-increasing with a running
//   minimum.  With `envelope` the row becomes the slopes of the upper concave envelope of the
//   points (n, R(n)), n = 0..cap, R(n) = sum of the clamped differences: the smallest concave
//   function that is nowhere below R (the function a greedy, one-core-at-a-time allocation is
//   exact for).
// reduction_cap - a user's hint of the loss the job is expected to end at (Conclusion,
//   "Non-convex optimization": hints of the target loss against over-estimated reductions).  The
//   job cannot be predicted to fall below its target: with newest loss l and target tau the
//   reduction is capped at max(l - tau, 0) / M, i.e. g(n) <- min(g(n), cap left after n-1 cores).
void upper_concave_envelope(int cap, const double* R /* cap + 1 */, double* slopes /* cap */) {
    std::vector<int> hull;   // indices of the envelope's vertices, left to right
    for (int n = 0; n <= cap; ++n) {
        while (hull.size() >= 2) {
            const int a = hull[hull.size() - 2], b = hull.back();
            // b lies on or below the chord a -> n: it is no vertex
            if ((R[b] - R[a]) * (double)(n - b) <= (R[n] - R[b]) * (double)(b - a)) hull.pop_back();
            else break;
        }
        hull.push_back(n);
    }
    for (size_t v = 1; v < hull.size(); ++v) {
        const int a = hull[v - 1], b = hull[v];
        const double slope = (R[b] - R[a]) / (double)(b - a);
        for (int n = a + 1; n <= b; ++n) slopes[n - 1] = slope;
    }
}

void job_gains(const JobFit& fit, double s, double w, double T, int cap, double* g, bool envelope = false,
               double reduction_cap = kInf) {
    for (int n = 0; n < cap; ++n) g[n] = 0.0;
    const bool predicts = fit.status == ST_FITTED || fit.status == ST_SHORT || fit.status == ST_NEW ||
                          fit.status == ST_FIT_FAILED;
    if (!predicts) return;
    if (!(w > 0.0) || !(s >= 0.0) || !std::isfinite(s) || !std::isfinite(w)) return;

    double X_prev = 0.0, den_prev = w, R_prev = 0.0;
    for (int n = 1; n <= cap; ++n) {
        const double den = s * (double)n + w;
        const double m = T * (double)n / den;          // iterations completed in the epoch
        const double X = m / fit.span;                 // same, in fit coordinates
        double gain;
        if (fit.status == ST_FITTED && fit.family == 0) {
            const double a = fit.params[0], b = fit.params[1], c = fit.params[2];
            const double dX = T * w / (fit.span * den * den_prev);
            const double q_now = a * X * X + b * X + c;
            const double q_prev = a * X_prev * X_prev + b * X_prev + c;
            const double dq = dX * (a * (X + X_prev) + b);
            gain = dq / (q_now * q_prev);
        } else if (fit.status == ST_FITTED && fit.family == 1) {
            const double alpha = fit.params[0], beta = fit.params[1];
            const double dX = T * w / (fit.span * den * den_prev);
            gain = std::exp(alpha - beta * X_prev) * (-std::expm1(-beta * dX));
        } else {
            const double R = std::min(fit.rho * m, fit.r_cap);
            gain = R - R_prev;
            R_prev = R;
        }
        if (!(std::isfinite(gain) && gain > 0.0)) gain = 0.0;
        if (!envelope && n >= 2 && gain > g[n - 2]) gain = g[n - 2];
        g[n - 1] = gain;
        X_prev = X;
        den_prev = den;
    }
    if (envelope) {
        bool rises = false;
        for (int n = 1; n < cap; ++n) rises = rises || g[n] > g[n - 1];
        if (rises) {   // a non-increasing row is its own envelope
            std::vector<double> R(cap + 1, 0.0);
            for (int n = 1; n <= cap; ++n) R[n] = R[n - 1] + g[n - 1];
            upper_concave_envelope(cap, R.data(), g);
        }
    }
    if (reduction_cap < kInf) {
        double before = 0.0;   // uncapped reduction of the first n - 1 cores
        for (int n = 1; n <= cap; ++n) {
            const double left = reduction_cap - before;
            before += g[n - 1];
            g[n - 1] = left > 0.0 ? std::min(g[n - 1], left) : 0.0;
        }
    }
}

// Iteration-time law t(n) = s + w/n from samples: ordinary least squares of t on
// u = 1/n using the sums a scheduler keeps per job.  With fewer than two distinct
// core counts, or a fit that is not physical, all time is taken as parallel work.
void time_model_from_sums(double cnt, double su, double suu, double st, double sut, double stn,
                          double umin, double umax, double* s, double* w) {
    if (!(cnt > 0.0)) {
        *s = kNaN;
        *w = kNaN;
        return;
    }
    if (umax > umin) {
        const double den = cnt * suu - su * su;
        const double ww = (cnt * sut - su * st) / den;
        const double ss = (st - ww * su) / cnt;
        if (den > 0.0 && std::isfinite(ww) && std::isfinite(ss) && ss >= 0.0 && ww > 0.0) {
            *s = ss;
            *w = ww;
            return;
        }
    }
    *s = 0.0;
    *w = stn / cnt;
}

// ---------------------------------------------------------------------------------
// Step 4.  Greedy allocation (Design, "Scheduling Based on Quality Improvements").
// Every active job starts with one core; then, one core at a time, the job whose next
// core has the largest predicted gain receives it, until the cores run out.  Equal
// gains go to the lowest job id.  With fewer cores than jobs there is no floor and the
// same loop hands out all cores from zero.  Returns the number of cores handed out.
// ---------------------------------------------------------------------------------
int64_t greedy_allocate(int64_t n_jobs, int cap, const double* gain, const uint8_t* active,
                        int64_t total_cores, int32_t* alloc) {
    int64_t n_active = 0;
    for (int64_t j = 0; j < n_jobs; ++j) {
        alloc[j] = 0;
        if (active[j]) ++n_active;
    }
    if (total_cores < 0) total_cores = 0;
    const int64_t usable = std::min<int64_t>(total_cores, n_active * (int64_t)cap);
    int64_t handed = 0;
    if (total_cores >= n_active) {
        for (int64_t j = 0; j < n_jobs; ++j)
            if (active[j]) {
                alloc[j] = 1;
                ++handed;
            }
    }
    struct Offer {
        double gain;
        int64_t job;
    };
    auto worse = [](const Offer& l, const Offer& r) {
        if (l.gain != r.gain) return l.gain < r.gain;
        return l.job > r.job;
    };
    std::priority_queue<Offer, std::vector<Offer>, decltype(worse)> heap(worse);
    for (int64_t j = 0; j < n_jobs; ++j)
        if (active[j] && alloc[j] < cap) heap.push({gain[j * cap + alloc[j]], j});
    while (handed < usable && !heap.empty()) {
        const Offer top = heap.top();
        heap.pop();
        const int64_t j = top.job;
        alloc[j] += 1;
        ++handed;
        if (alloc[j] < cap) heap.push({gain[j * cap + alloc[j]], j});
    }
    return handed;
}

void set_threads(int threads) {
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
}

}  // namespace

extern "C" {

// Threads the last parallel call could use.
int oracle_max_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Step 1 over CSR histories.  out_M[j]: largest reduction (NaN for jobs with < 2 points and
// nothing seen); out_dnorm / out_y: per point, dnorm of a job's first point is 0.
int oracle_normalise(int64_t n_jobs, const int64_t* offsets, const double* losses, const double* m_seen,
                     double* out_M, double* out_dnorm, double* out_y) {
    for (int64_t j = 0; j < n_jobs; ++j) {
        const int64_t lo = offsets[j], H = offsets[j + 1] - lo;
        const double seen = m_seen ? m_seen[j] : -kInf;
        const double M = H >= 1 ? largest_reduction(losses + lo, H, seen) : kNaN;
        out_M[j] = M;
        for (int64_t i = 0; i < H; ++i) {
            if (out_y) out_y[lo + i] = losses[lo + i] / M;
            if (out_dnorm) out_dnorm[lo + i] = i == 0 ? 0.0 : (losses[lo + i - 1] - losses[lo + i]) / M;
        }
    }
    return 0;
}

// Steps 1-3 over CSR histories: fit record and gain rows gain[j*cap + (n-1)], n = 1..cap.
// With warm_valid: the warm-started variant; warm_p holds [n_jobs][8] (family I then II),
// warm_K / warm_span / warm_M the coordinates those parameters refer to, k_last the index of
// each job's newest iteration now.  out_both [n_jobs][8] and out_mask receive both families'
// final parameters and which of them ended with a finite residual.
int oracle_predict_warm(int64_t n_jobs, const int64_t* offsets, const double* losses, const double* m_seen,
                        const double* s, const double* w, double epoch_seconds, int32_t cap, double gamma,
                        int32_t lm_trials, int32_t threads, int8_t* out_family, double* out_params,
                        double* out_S, int32_t* out_status, int32_t* out_evals, double* out_M, double* out_gain,
                        const int64_t* k_last, const uint8_t* warm_valid, const double* warm_p,
                        const int64_t* warm_K, const double* warm_span, const double* warm_M, double* out_both,
                        uint8_t* out_mask, int32_t envelope, const double* target_loss) {
    Settings cfg;
    cfg.gamma = gamma;
    cfg.lm_trials = lm_trials;
    set_threads(threads);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t j = 0; j < n_jobs; ++j) {
        const int64_t lo = offsets[j], H = offsets[j + 1] - lo;
        WarmStart warm;
        if (warm_valid && warm_valid[j]) {
            warm.valid = warm_valid[j];
            std::memcpy(warm.pI, warm_p + 8 * j, sizeof warm.pI);
            std::memcpy(warm.pII, warm_p + 8 * j + 4, sizeof warm.pII);
            warm.K = warm_K[j];
            warm.span = warm_span[j];
            warm.M = warm_M[j];
        }
        JobFit fit = fit_job(losses + lo, H, m_seen ? m_seen[j] : -kInf, cfg, warm.valid ? &warm : nullptr,
                             k_last ? k_last[j] : 0);
        if (out_both) std::memcpy(out_both + 8 * j, fit.both, sizeof fit.both);
        if (out_mask) out_mask[j] = fit.fitted_mask;
        const bool has_time = std::isfinite(s[j]) && std::isfinite(w[j]) && w[j] > 0.0 && s[j] >= 0.0;
        if (fit.status != ST_INACTIVE && fit.status != ST_NONFINITE && fit.status != ST_FLAT && !has_time)
            fit.status = ST_NO_TIME;
        if (out_family) out_family[j] = fit.family;
        if (out_params) std::memcpy(out_params + 4 * j, fit.params, sizeof fit.params);
        if (out_S) {
            out_S[2 * j] = fit.S[0];
            out_S[2 * j + 1] = fit.S[1];
        }
        if (out_status) out_status[j] = fit.status;
        if (out_evals) {
            out_evals[2 * j] = fit.evals[0];
            out_evals[2 * j + 1] = fit.evals[1];
        }
        if (out_M) out_M[j] = fit.M;
        if (out_gain) {
            double reduction_cap = kInf;   // a target-loss hint: nothing is gained below the target
            if (target_loss && std::isfinite(target_loss[j]) && H >= 1 && fit.M > 0.0)
                reduction_cap = std::max(losses[lo + H - 1] - target_loss[j], 0.0) / fit.M;
            job_gains(fit, s[j], w[j], epoch_seconds, cap, out_gain + (int64_t)j * cap, envelope != 0, reduction_cap);
        }
    }
    return 0;
}

int oracle_predict(int64_t n_jobs, const int64_t* offsets, const double* losses, const double* m_seen,
                   const double* s, const double* w, double epoch_seconds, int32_t cap, double gamma,
                   int32_t lm_trials, int32_t threads, int8_t* out_family, double* out_params,
                   double* out_S, int32_t* out_status, int32_t* out_evals, double* out_M, double* out_gain) {
    return oracle_predict_warm(n_jobs, offsets, losses, m_seen, s, w, epoch_seconds, cap, gamma, lm_trials, threads,
                               out_family, out_params, out_S, out_status, out_evals, out_M, out_gain, nullptr,
                               nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr);
}

// Step 4 alone on given gain rows.  Returns cores handed out.
int64_t oracle_allocate(int64_t n_jobs, int32_t cap, const double* gain, const uint8_t* active,
                        int64_t total_cores, int32_t* out_alloc) {
    return greedy_allocate(n_jobs, cap, gain, active, total_cores, out_alloc);
}

// Predicted reduction at the allocation: R_j(a_j) = sum of the job's first a_j gains.
void oracle_reduction_at(int64_t n_jobs, int32_t cap, const double* gain, const int32_t* alloc, double* out_R) {
    for (int64_t j = 0; j < n_jobs; ++j) {
        double R = 0.0;
        for (int n = 0; n < alloc[j]; ++n) R += gain[j * cap + n];
        out_R[j] = R;
    }
}

void oracle_time_model(int64_t n_jobs, const double* cnt, const double* su, const double* suu, const double* st,
                       const double* sut, const double* stn, const double* umin, const double* umax,
                       double* out_s, double* out_w) {
    for (int64_t j = 0; j < n_jobs; ++j)
        time_model_from_sums(cnt[j], su[j], suu[j], st[j], sut[j], stn[j], umin[j], umax[j], out_s + j, out_w + j);
}

// ---- hooks that exist only so tests can pin the pieces above ----

// Slopes of the upper concave envelope of (n, R[n]), n = 0..cap.
void oracle_envelope(int32_t cap, const double* R, double* out_slopes) { upper_concave_envelope(cap, R, out_slopes); }

// Value and Jacobian of a family (0 sublinear, 1 exponential) at x.  Returns 0 if undefined there.
int oracle_family_eval(int32_t family, const double* p, double x, double* f, double* jac) {
    return family == 0 ? Sublinear::eval(p, x, f, jac) : Exponential::eval(p, x, f, jac);
}

// The solver on the straight-line model; p holds the start and receives the result.
int oracle_lm_line(int64_t H, const double* x, const double* y, const double* w, int32_t trials, double lambda0,
                   double* p, double* out_S) {
    FitData D;
    D.H = H;
    D.x.assign(x, x + H);
    D.y.assign(y, y + H);
    D.w.assign(w, w + H);
    for (int64_t i = 0; i < H; ++i) D.sum_wy2 += w[i] * y[i] * y[i];
    const LmOutcome r = levenberg_marquardt<Line>(p, D, trials, lambda0);
    *out_S = r.S;
    return r.ok ? r.evals : -1;
}

// A family's parameters carried into new window coordinates (x_old = t + r x_new, y_new = sigma y_old).
void oracle_carry(int32_t family, const double* p, double t, double r, double sigma, double* out) {
    if (family == 0) carry_sublinear(p, t, r, sigma, out);
    else carry_exponential(p, t, r, sigma, out);
}

// Fit one family only, from its own initial guess, on one history; returns sweeps used or -1.
// out_grad receives sum w J r at the end point (zero at a stationary point).
int oracle_fit_family(int32_t family, int64_t H, const double* loss, double m_seen, double gamma, int32_t trials,
                      double* out_p, double* out_S, double* out_grad, double* out_p0) {
    const double M = largest_reduction(loss, H, m_seen);
    const FitData D = make_fit_data(loss, H, M, gamma);
    double p[4] = {0, 0, 0, 0};
    LmOutcome r;
    double A[4][4], g[4] = {0, 0, 0, 0}, S;
    if (family == 0) {
        init_sublinear(D, p);
        if (out_p0) std::memcpy(out_p0, p, sizeof p);
        r = levenberg_marquardt<Sublinear>(p, D, trials, 1e-3);
        normal_equations<Sublinear>(p, D, A, g, &S);
    } else {
        init_exponential(D, p);
        if (out_p0) std::memcpy(out_p0, p, sizeof p);
        r = levenberg_marquardt<Exponential>(p, D, trials, 1e-3);
        normal_equations<Exponential>(p, D, A, g, &S);
    }
    std::memcpy(out_p, p, sizeof p);
    *out_S = r.S;
    if (out_grad) std::memcpy(out_grad, g, sizeof g);
    return r.ok ? r.evals : -1;
}

}  // extern "C"
