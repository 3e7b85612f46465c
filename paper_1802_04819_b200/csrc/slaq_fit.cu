// Normalisation and curve fit: one warp per job.
//
// The warp stages the job's window of stored losses in shared memory, finds the largest
// one-step reduction seen so far, scales the window by it ("Normalizing Quality Metrics"),
// then fits both convergence families of "Predicting Quality Improvement",
//     I : f(x) = 1 / (a x^2 + b x + c) + d          II : f(x) = exp(alpha - beta x) + c,
// by exponentially weighted least squares with Levenberg-Marquardt, in window coordinates
// (newest point x = 0, oldest x = -1).  Lanes stride over the points, the normal equations
// are reduced with warp shuffles, every lane then solves the same 4x4 system.  The family
// with the lower weighted residual wins.
#include <math_constants.h>

#include "slaq_internal.cuh"

namespace slaq {

namespace {

constexpr int kMaxWarpsPerBlock = 8;
constexpr size_t kSmemLimit = 227 * 1024;   // shared memory one block may use on sm_100
constexpr unsigned kFull = 0xffffffffu;
constexpr double kLambda0 = 1e-3, kLambdaMin = 1e-5, kLambdaMax = 1e12;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ double warp_min(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ bool finite_d(double v) { return fabs(v) <= 1.7976931348623157e308; }

// Copy the job's window, oldest first, into sm[0..H).  Ring storage: the newest loss sits
// just before `head`.  Returns H, or 0 after flagging storage that cannot be right.
__device__ int stage_window(const JobArrays& job, int j, int max_hist, double* sm, int lane, int32_t* err_word) {
    const double* row = job.row[j];
    const int cap = job.cap[j];
    const int H = job.count[j];
    if (H == 0) return 0;
    if (H > cap || cap > max_hist || H < 0 || row == nullptr) {   // never expected: record and skip the job
        if (lane == 0) atomicOr(err_word, 1);
        return 0;
    }
    int start = job.head[j] - H;
    if (start < 0) start += cap;
    for (int i = lane; i < H; i += 32) {
        int s = start + i;
        if (s >= cap) s -= cap;
        sm[i] = row[s];
    }
    __syncwarp();
    return H;
}

struct Normalised {
    double M;        // largest reduction seen so far
    int status;      // SLAQ_JOB_FITTED here means "usable": M > 0 and everything finite
    double rho;      // weighted mean normalised reduction per iteration (linear extrapolation)
};

// Largest reduction over the window joined with what was seen before it; weighted mean
// normalised change; then the window is scaled in place to levels y = l / M.
// d_changes (optional, global) receives the normalised changes of the window.
__device__ Normalised normalise_window(double* sm, int H, double m_seen, const double* wtab, int lane,
                                       double* d_changes) {
    Normalised out;
    out.M = CUDART_NAN;
    out.rho = 0.0;
    bool fin = true;
    double dmax = -CUDART_INF;
    for (int i = lane; i < H; i += 32) {
        const double v = sm[i];
        fin = fin && finite_d(v);
        if (i > 0) dmax = fmax(dmax, sm[i - 1] - v);
    }
    fin = __all_sync(kFull, fin) && !(m_seen != m_seen) && !(m_seen == CUDART_INF);
    if (!fin) {
        out.status = SLAQ_JOB_NONFINITE;
        return out;
    }
    if (H == 1) {
        out.status = SLAQ_JOB_NEW;
        return out;
    }
    dmax = warp_max(dmax);
    const double M = fmax(m_seen, dmax);
    out.M = M;
    if (!(M > 0.0) || !finite_d(M)) {
        out.status = SLAQ_JOB_FLAT;
        return out;
    }
    double num = 0.0, den = 0.0;
    for (int i = lane; i < H; i += 32) {
        if (i > 0) {
            const double change = __ddiv_rn(sm[i - 1] - sm[i], M);
            const double w = wtab[H - 1 - i];
            num = fma(w, change, num);
            den += w;
            if (d_changes) d_changes[i] = change;
        } else if (d_changes) {
            d_changes[0] = 0.0;
        }
    }
    num = warp_sum(num);
    den = warp_sum(den);
    out.rho = fmax(num / den, 0.0);
    __syncwarp();
    for (int i = lane; i < H; i += 32) sm[i] = __ddiv_rn(sm[i], M);
    __syncwarp();
    out.status = SLAQ_JOB_FITTED;
    return out;
}

// ---- small dense algebra, every lane does the same work on the same numbers ----

// Solve B d = r for a symmetric positive definite N x N system (N = 3 or 4) by Cholesky.
template <int N>
__device__ bool chol_solve(const double (&B)[4][4], const double (&r)[4], double (&d)[4]) {
    double L[4][4];
#pragma unroll
    for (int i = 0; i < N; ++i) {
#pragma unroll
        for (int j = 0; j <= i; ++j) {
            double sum = B[i][j];
#pragma unroll
            for (int k = 0; k < j; ++k) sum = fma(-L[i][k], L[j][k], sum);
            if (i == j) {
                if (!(sum > 0.0) || !finite_d(sum)) return false;
                L[i][i] = sqrt(sum);
            } else {
                L[i][j] = sum / L[j][j];
            }
        }
    }
    double z[4];
#pragma unroll
    for (int i = 0; i < N; ++i) {
        double sum = r[i];
#pragma unroll
        for (int k = 0; k < i; ++k) sum = fma(-L[i][k], z[k], sum);
        z[i] = sum / L[i][i];
    }
    bool ok = true;
#pragma unroll
    for (int i = N - 1; i >= 0; --i) {
        double sum = z[i];
#pragma unroll
        for (int k = i + 1; k < N; ++k) sum = fma(-L[k][i], d[k], sum);
        d[i] = sum / L[i][i];
        ok = ok && finite_d(d[i]);
    }
    return ok;
}

struct Window {
    const double* y;      // normalised levels in shared memory
    const double* wtab;   // gamma^m in shared memory
    int H;
    int lane;
    double inv_span;      // 1 / (H - 1)
    double sw;            // sum of weights
};

// Normal equations of one family at parameters p: S = sum w r^2, A = sum w J J^T,
// g = sum w J r, r = y - f.  False when the model is undefined at a stored point or a
// sum is not finite.
struct Sublinear {
    static constexpr int P = 4;
    __device__ static double lower(int a) { return a == 3 ? -CUDART_INF : (a == 2 ? 1e-12 : 0.0); }
    __device__ static bool normal_eq(const Window& W, const double (&p)[4], double (&A)[4][4], double (&g)[4],
                                     double& S) {
        // with u = 1/q^2: J = (-u x^2, -u x, -u, 1); A needs the moments of w u^2 and w u
        double m0 = 0, m1 = 0, m2 = 0, m3 = 0, m4 = 0, n0 = 0, n1 = 0, n2 = 0;
        double h0 = 0, h1 = 0, h2 = 0, gd = 0, acc = 0;
        bool ok = true;
        for (int i = W.lane; i < W.H; i += 32) {
            const double x = (double)(i - (W.H - 1)) * W.inv_span;
            const double w = W.wtab[W.H - 1 - i];
            const double q = fma(fma(p[0], x, p[1]), x, p[2]);
            ok = ok && (q > 0.0);
            const double inv = 1.0 / q;
            const double r = W.y[i] - (inv + p[3]);
            const double u = inv * inv;
            const double x2 = x * x;
            const double wu = w * u, wuu = wu * u, wur = wu * r, wr = w * r;
            const double t = wuu * x2;
            m0 += wuu;
            m1 = fma(wuu, x, m1);
            m2 += t;
            m3 = fma(t, x, m3);
            m4 = fma(t, x2, m4);
            n0 += wu;
            n1 = fma(wu, x, n1);
            n2 = fma(wu, x2, n2);
            h0 += wur;
            h1 = fma(wur, x, h1);
            h2 = fma(wur, x2, h2);
            gd += wr;
            acc = fma(wr, r, acc);
        }
        ok = __all_sync(kFull, ok);
        if (!ok) return false;
        m0 = warp_sum(m0); m1 = warp_sum(m1); m2 = warp_sum(m2); m3 = warp_sum(m3); m4 = warp_sum(m4);
        n0 = warp_sum(n0); n1 = warp_sum(n1); n2 = warp_sum(n2);
        h0 = warp_sum(h0); h1 = warp_sum(h1); h2 = warp_sum(h2);
        gd = warp_sum(gd);
        S = warp_sum(acc);
        A[0][0] = m4; A[0][1] = A[1][0] = m3; A[0][2] = A[2][0] = m2; A[1][1] = m2;
        A[1][2] = A[2][1] = m1; A[2][2] = m0;
        A[0][3] = A[3][0] = -n2; A[1][3] = A[3][1] = -n1; A[2][3] = A[3][2] = -n0; A[3][3] = W.sw;
        g[0] = -h2; g[1] = -h1; g[2] = -h0; g[3] = gd;
        const double chk = m0 + m1 + m2 + m3 + m4 + n0 + n1 + n2 + h0 + h1 + h2 + gd + S;
        return finite_d(chk);
    }
};

struct Exponential {
    static constexpr int P = 3;
    __device__ static double lower(int a) { return a == 1 ? 0.0 : -CUDART_INF; }
    __device__ static bool normal_eq(const Window& W, const double (&p)[4], double (&A)[4][4], double (&g)[4],
                                     double& S) {
        // J = (e, -x e, 1) with e = exp(alpha - beta x)
        double e0 = 0, e1 = 0, e2 = 0, f0 = 0, f1 = 0, h0 = 0, h1 = 0, gc = 0, acc = 0;
        for (int i = W.lane; i < W.H; i += 32) {
            const double x = (double)(i - (W.H - 1)) * W.inv_span;
            const double w = W.wtab[W.H - 1 - i];
            const double e = exp(fma(-p[1], x, p[0]));
            const double r = W.y[i] - (e + p[2]);
            const double we = w * e, wee = we * e, wer = we * r, wr = w * r;
            const double t = wee * x;
            e0 += wee;
            e1 += t;
            e2 = fma(t, x, e2);
            f0 += we;
            f1 = fma(we, x, f1);
            h0 += wer;
            h1 = fma(wer, x, h1);
            gc += wr;
            acc = fma(wr, r, acc);
        }
        e0 = warp_sum(e0); e1 = warp_sum(e1); e2 = warp_sum(e2);
        f0 = warp_sum(f0); f1 = warp_sum(f1);
        h0 = warp_sum(h0); h1 = warp_sum(h1);
        gc = warp_sum(gc);
        S = warp_sum(acc);
        A[0][0] = e0; A[0][1] = A[1][0] = -e1; A[1][1] = e2;
        A[0][2] = A[2][0] = f0; A[1][2] = A[2][1] = -f1; A[2][2] = W.sw;
        A[0][3] = A[3][0] = A[1][3] = A[3][1] = A[2][3] = A[3][2] = 0.0; A[3][3] = 1.0;
        g[0] = h0; g[1] = -h1; g[2] = gc; g[3] = 0.0;
        const double chk = e0 + e1 + e2 + f0 + f1 + h0 + h1 + gc + S;
        return finite_d(chk);
    }
};

struct LmResult {
    bool ok;      // the starting point was usable
    double S;     // final weighted residual
    int sweeps;   // passes over the window: the start plus one per solved trial
};

// Levenberg-Marquardt with Marquardt's diagonal scaling and the gain-ratio damping update
// (Madsen, Nielsen, Tingleff 2004).  Parameters on their lower bound are frozen while the
// descent direction or the solved step points outside, and stay frozen from then on; the
// trial point is clipped to the bounds; a trial is accepted only if the residual strictly falls.
template <class F>
__device__ LmResult levenberg_marquardt(const Window& W, double (&p)[4], int trials, double sum_wy2) {
    constexpr int P = F::P;
    LmResult out;
    out.sweeps = 1;
    out.S = CUDART_INF;
    double A[4][4], g[4], S;
    out.ok = F::normal_eq(W, p, A, g, S);
    if (!out.ok) return out;
    double lambda = kLambda0, nu = 2.0;
    unsigned was_frozen = 0;
    for (int t = 0; t < trials; ++t) {
        if (S <= 1e-28 * sum_wy2) break;
        unsigned frozen = 0;
#pragma unroll
        for (int a = 0; a < P; ++a)
            if (p[a] <= F::lower(a) && (g[a] < 0.0 || ((was_frozen >> a) & 1u))) frozen |= 1u << a;
        double step[4] = {0.0, 0.0, 0.0, 0.0};
        bool solved = false;
        for (int round = 0; round <= P; ++round) {
            double B[4][4], rhs[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const bool fa = a >= P || ((frozen >> a) & 1u);
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const bool fb = b >= P || ((frozen >> b) & 1u);
                    B[a][b] = (fa || fb) ? 0.0 : A[a][b];
                }
                B[a][a] = fa ? 1.0 : fma(lambda, fmax(A[a][a], 1e-300), A[a][a]);
                rhs[a] = fa ? 0.0 : g[a];
            }
            solved = chol_solve<P>(B, rhs, step);
            if (!solved) break;
            unsigned grow = 0;
#pragma unroll
            for (int a = 0; a < P; ++a)
                if (!((frozen >> a) & 1u) && p[a] <= F::lower(a) && step[a] < 0.0) grow |= 1u << a;
            if (!grow) break;
            frozen |= grow;
        }
        was_frozen |= frozen;
        bool accepted = false;
        if (solved) {
            double trial[4] = {0.0, 0.0, 0.0, 0.0}, d[4] = {0.0, 0.0, 0.0, 0.0};
            bool fin = true;
#pragma unroll
            for (int a = 0; a < P; ++a) {
                trial[a] = fmax(p[a] + step[a], F::lower(a));
                d[a] = trial[a] - p[a];
                fin = fin && finite_d(trial[a]);
            }
            double dg = 0.0, dAd = 0.0;
#pragma unroll
            for (int a = 0; a < P; ++a) {
                dg = fma(d[a], g[a], dg);
#pragma unroll
                for (int b = 0; b < P; ++b) dAd = fma(d[a] * A[a][b], d[b], dAd);
            }
            const double predicted = 2.0 * dg - dAd;
            double A2[4][4], g2[4], S2 = CUDART_INF;
            bool ok2 = false;
            out.sweeps += 1;   // every solved trial counts as one sweep over the window
            if (fin) ok2 = F::normal_eq(W, trial, A2, g2, S2);
            if (ok2 && S2 < S) {
                accepted = true;
                const double S_before = S;
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    p[a] = trial[a];
                    g[a] = g2[a];
#pragma unroll
                    for (int b = 0; b < 4; ++b) A[a][b] = A2[a][b];
                }
                S = S2;
                const double rho = predicted > 0.0 ? (S_before - S) / predicted : 0.0;
                const double c = 2.0 * rho - 1.0;
                lambda *= fmax(1.0 / 3.0, 1.0 - c * c * c);
                nu = 2.0;
                lambda = fmin(fmax(lambda, kLambdaMin), kLambdaMax);
                if (S_before - S <= 1e-14 * S_before) break;
            }
        }
        if (!accepted) {
            lambda = fmin(lambda * nu, kLambdaMax);
            nu *= 2.0;
        }
    }
    out.S = S;
    return out;
}

struct Moments {
    double sw, swx, swx2, swx3, swx4, swy2, ymin, ymax;
};

__device__ Moments window_moments(const Window& W) {
    Moments m = {0, 0, 0, 0, 0, 0, CUDART_INF, -CUDART_INF};
    for (int i = W.lane; i < W.H; i += 32) {
        const double x = (double)(i - (W.H - 1)) * W.inv_span;
        const double w = W.wtab[W.H - 1 - i];
        const double y = W.y[i];
        const double wx = w * x, wx2 = wx * x;
        m.sw += w;
        m.swx += wx;
        m.swx2 += wx2;
        m.swx3 = fma(wx2, x, m.swx3);
        m.swx4 = fma(wx2 * x, x, m.swx4);
        m.swy2 = fma(w * y, y, m.swy2);
        m.ymin = fmin(m.ymin, y);
        m.ymax = fmax(m.ymax, y);
    }
    m.sw = warp_sum(m.sw); m.swx = warp_sum(m.swx); m.swx2 = warp_sum(m.swx2);
    m.swx3 = warp_sum(m.swx3); m.swx4 = warp_sum(m.swx4); m.swy2 = warp_sum(m.swy2);
    m.ymin = warp_min(m.ymin); m.ymax = warp_max(m.ymax);
    return m;
}

// Offset below every level; both families are linearised around it for their first guess.
__device__ double floor_guess(const Moments& m) {
    if (m.ymax > m.ymin) return m.ymin - 0.1 * (m.ymax - m.ymin);
    return m.ymin - 1e-3 * fmax(fabs(m.ymin), 1.0);
}

// Family I: with d fixed, 1/(y - d) is a quadratic in x: weighted linear least squares.
__device__ void init_sublinear(const Window& W, const Moments& m, double (&p)[4]) {
    const double d0 = floor_guess(m);
    double r0 = 0, r1 = 0, r2 = 0;
    for (int i = W.lane; i < W.H; i += 32) {
        const double x = (double)(i - (W.H - 1)) * W.inv_span;
        const double w = W.wtab[W.H - 1 - i];
        const double wz = w / (W.y[i] - d0);
        r2 += wz;
        r1 = fma(wz, x, r1);
        r0 = fma(wz * x, x, r0);
    }
    r0 = warp_sum(r0); r1 = warp_sum(r1); r2 = warp_sum(r2);
    double B[4][4] = {{m.swx4, m.swx3, m.swx2, 0}, {m.swx3, m.swx2, m.swx, 0}, {m.swx2, m.swx, m.sw, 0}, {0, 0, 0, 1}};
    double rhs[4] = {r0, r1, r2, 0}, sol[4] = {0, 0, 0, 0};
    bool good = chol_solve<3>(B, rhs, sol) && sol[0] >= 0.0 && sol[1] >= 0.0;
    if (good) {
        bool pos = true;
        for (int i = W.lane; i < W.H; i += 32) {
            const double x = (double)(i - (W.H - 1)) * W.inv_span;
            pos = pos && (fma(fma(sol[0], x, sol[1]), x, sol[2]) > 0.0);
        }
        good = __all_sync(kFull, pos);
    }
    if (good) {
        p[0] = sol[0]; p[1] = sol[1]; p[2] = sol[2];
    } else {   // straight line through the oldest and newest transformed points
        const double z_old = 1.0 / (W.y[0] - d0), z_new = 1.0 / (W.y[W.H - 1] - d0);
        p[0] = 0.0;
        p[1] = fmax(z_new - z_old, 0.0);
        p[2] = z_new;
    }
    p[3] = d0;
}

// Family II: with c fixed, log(y - c) is a line in x.
__device__ void init_exponential(const Window& W, const Moments& m, double (&p)[4]) {
    const double d0 = floor_guess(m);
    double su = 0, sxu = 0;
    for (int i = W.lane; i < W.H; i += 32) {
        const double x = (double)(i - (W.H - 1)) * W.inv_span;
        const double w = W.wtab[W.H - 1 - i];
        const double wu = w * log(W.y[i] - d0);
        su += wu;
        sxu = fma(wu, x, sxu);
    }
    su = warp_sum(su); sxu = warp_sum(sxu);
    const double den = m.sw * m.swx2 - m.swx * m.swx;
    const double slope = (m.sw * sxu - m.swx * su) / den;
    p[0] = (su - slope * m.swx) / m.sw;
    p[1] = fmax(-slope, 1e-8);
    p[2] = d0;
    p[3] = 0.0;
}

__global__ void __launch_bounds__(kMaxWarpsPerBlock * 32)
fit_kernel(JobArrays job, FitArrays fit, const double* __restrict__ g_wtab, const int32_t* __restrict__ order,
           int n_work, int max_hist, int lm_trials, int min_fit_points, unsigned int* queue, long long* counters,
           int32_t* err_word) {
    extern __shared__ double smem[];
    double* wtab = smem;                                   // [max_hist]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double* win = smem + max_hist + (size_t)warp * max_hist;   // this warp's window
    for (int i = threadIdx.x; i < max_hist; i += blockDim.x) wtab[i] = g_wtab[i];
    __syncthreads();

    long long n_points = 0, n_sweep_points = 0;
    int n_fit = 0, n_sub = 0, n_exp = 0, n_fallback = 0;
    for (;;) {
        int slot = 0;
        if (lane == 0) slot = (int)atomicAdd(queue, 1u);
        slot = __shfl_sync(kFull, slot, 0);
        if (slot >= n_work) break;
        const int j = order ? order[slot] : slot;
        const int H = stage_window(job, j, max_hist, win, lane, err_word);

        int status = SLAQ_JOB_INACTIVE, family = -1;
        double p_out[4] = {CUDART_NAN, CUDART_NAN, CUDART_NAN, CUDART_NAN};
        double S_out[2] = {CUDART_INF, CUDART_INF};
        int sweeps[2] = {0, 0};
        double M = CUDART_NAN;
        const double span = (double)max(H - 1, 1);
        if (H > 0) {
            const Normalised nz = normalise_window(win, H, job.m_seen[j], wtab, lane, nullptr);
            status = nz.status;
            M = nz.M;
            n_points += H;
            if (status == SLAQ_JOB_NEW) {
                p_out[0] = 1.0;   // one normalised unit per iteration
                p_out[1] = 1.0;   // at most the whole normalised loss
            } else if (status == SLAQ_JOB_FITTED) {
                bool fitted = false;
                if (H >= min_fit_points) {
                    Window W = {win, wtab, H, lane, 1.0 / span, 0.0};
                    const Moments mom = window_moments(W);
                    W.sw = mom.sw;
                    double pI[4], pII[4];
                    init_sublinear(W, mom, pI);
                    const LmResult rI = levenberg_marquardt<Sublinear>(W, pI, lm_trials, mom.swy2);
                    init_exponential(W, mom, pII);
                    const LmResult rII = levenberg_marquardt<Exponential>(W, pII, lm_trials, mom.swy2);
                    sweeps[0] = rI.sweeps;
                    sweeps[1] = rII.sweeps;
                    if (rI.ok) S_out[0] = rI.S;
                    if (rII.ok) S_out[1] = rII.S;
                    const bool okI = rI.ok && finite_d(rI.S), okII = rII.ok && finite_d(rII.S);
                    if (okI && (!okII || rI.S <= rII.S)) {   // a tie goes to family I
                        family = 0;
#pragma unroll
                        for (int a = 0; a < 4; ++a) p_out[a] = pI[a];
                        fitted = true;
                    } else if (okII) {
                        family = 1;
#pragma unroll
                        for (int a = 0; a < 4; ++a) p_out[a] = pII[a];
                        fitted = true;
                    }
                    n_sweep_points += (long long)H * (rI.sweeps + rII.sweeps);
                }
                if (!fitted) {
                    status = H >= min_fit_points ? SLAQ_JOB_FIT_FAILED : SLAQ_JOB_SHORT;
                    const double y_new = win[H - 1];
                    p_out[0] = nz.rho;
                    p_out[1] = y_new > 0.0 ? y_new : CUDART_INF;
                    p_out[2] = p_out[3] = CUDART_NAN;
                }
            }
        }
        if (status == SLAQ_JOB_FITTED) {
            n_fit += 1;
            n_sub += family == 0;
            n_exp += family == 1;
        } else if (status == SLAQ_JOB_SHORT || status == SLAQ_JOB_NEW || status == SLAQ_JOB_FIT_FAILED) {
            n_fallback += 1;
        }
        if (lane == 0) {
            fit.status[j] = status;
            fit.family[j] = (int8_t)family;
#pragma unroll
            for (int a = 0; a < 4; ++a) fit.params[4 * (size_t)j + a] = p_out[a];
            fit.residual[2 * (size_t)j] = S_out[0];
            fit.residual[2 * (size_t)j + 1] = S_out[1];
            fit.sweeps[2 * (size_t)j] = sweeps[0];
            fit.sweeps[2 * (size_t)j + 1] = sweeps[1];
            fit.largest[j] = M;
            fit.span[j] = span;
        }
        __syncwarp();
    }
    if (lane == 0) {
        atomicAdd((unsigned long long*)&counters[0], (unsigned long long)n_points);
        atomicAdd((unsigned long long*)&counters[1], (unsigned long long)n_sweep_points);
        atomicAdd((unsigned long long*)&counters[2], (unsigned long long)n_fit);
        atomicAdd((unsigned long long*)&counters[3], (unsigned long long)n_sub);
        atomicAdd((unsigned long long*)&counters[4], (unsigned long long)n_exp);
        atomicAdd((unsigned long long*)&counters[5], (unsigned long long)n_fallback);
    }
}

// Normalisation only, written out for inspection: same staging and scaling code as the fit.
__global__ void __launch_bounds__(kMaxWarpsPerBlock * 32)
normalise_export_kernel(JobArrays job, const int32_t* __restrict__ ids, const int64_t* __restrict__ offsets, int n,
                        const double* __restrict__ g_wtab, int max_hist, double* changes, double* levels,
                        double* largest, int32_t* err_word) {
    extern __shared__ double smem[];
    double* wtab = smem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double* win = smem + max_hist + (size_t)warp * max_hist;
    for (int i = threadIdx.x; i < max_hist; i += blockDim.x) wtab[i] = g_wtab[i];
    __syncthreads();
    const int slot = blockIdx.x * (blockDim.x >> 5) + warp;
    if (slot >= n) return;
    const int j = ids[slot];
    const int H = stage_window(job, j, max_hist, win, lane, err_word);
    if (H <= 0) {
        if (lane == 0 && largest) largest[slot] = CUDART_NAN;
        return;
    }
    const int64_t base = offsets[slot];
    const Normalised nz = normalise_window(win, H, job.m_seen[j], wtab, lane, changes ? changes + base : nullptr);
    if (lane == 0 && largest) largest[slot] = nz.M;
    if (nz.status != SLAQ_JOB_FITTED) {   // nothing was scaled: report NaN levels and changes
        for (int i = lane; i < H; i += 32) {
            if (levels) levels[base + i] = CUDART_NAN;
            if (changes) changes[base + i] = CUDART_NAN;
        }
        return;
    }
    if (levels)
        for (int i = lane; i < H; i += 32) levels[base + i] = win[i];
}

size_t fit_smem_bytes(int32_t max_hist, int warps) { return sizeof(double) * (size_t)max_hist * (warps + 1); }

// Warps per block: as many as fit beside the weight table, each with a whole window.
int warps_for(int32_t max_hist) {
    int warps = kMaxWarpsPerBlock;
    while (warps > 1 && fit_smem_bytes(max_hist, warps) > kSmemLimit) --warps;
    return warps;
}

}  // namespace

int launch_fit(slaq_handle* h) {
    const int warps = warps_for(h->max_hist);
    const size_t smem = fit_smem_bytes(h->max_hist, warps);
    cudaError_t e = cudaFuncSetAttribute(fit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        h->err = std::string("fit kernel shared memory: ") + cudaGetErrorString(e);
        return -1;
    }
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fit_kernel, warps * 32, smem);
    if (per_sm < 1) per_sm = 1;
    const int n_work = h->max_jobs;
    int blocks = h->sm_count * per_sm;
    const int needed = (n_work + warps - 1) / warps;
    if (blocks > needed) blocks = needed;
    if (blocks < 1) blocks = 1;
    fit_kernel<<<blocks, warps * 32, smem, h->stream>>>(
        h->job, h->fit, h->wtab, nullptr, n_work, h->max_hist, h->lm_trials, h->min_fit_points,
        h->scratch.ticket, h->scratch.counters, h->err_word);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        h->err = std::string("fit kernel launch: ") + cudaGetErrorString(e);
        return -1;
    }
    return 1;
}

int launch_normalise_export(slaq_handle* h, int32_t n, const int64_t* d_offsets, double* d_changes,
                            double* d_levels, double* d_largest) {
    if (n <= 0) return 0;
    const int warps = warps_for(h->max_hist);
    const size_t smem = fit_smem_bytes(h->max_hist, warps);
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
