// The inner loop of the curve fit: one sweep over a job's window that evaluates both
// convergence families of "Predicting Quality Improvement" at their current points and
// accumulates the sums of their normal equations.  Kept in a header of its own so that the
// stand-alone timing program (bench_probes/fit_sweep_probe.cu) runs exactly this code.
#pragma once

#include <math_constants.h>

#include "slaq_bounds.cuh"

namespace slaq {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kParked = 12;                 // doubles per job and family kept in shared memory between sweeps

__device__ __forceinline__ bool finite_d(double v) { return fabs(v) <= 1.7976931348623157e308; }

// Reciprocal to about one ulp: hardware seed and two Newton steps (no special-case paths;
// a zero, subnormal or non-finite argument gives a non-finite or zero result, which the
// callers treat as "not usable").
__device__ __forceinline__ double fast_rcp(double q) {
    double x;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(x) : "d"(q));
    double e = fma(-q, x, 1.0);
    x = fma(x, e, x);
    e = fma(-q, x, 1.0);
    return fma(x, e, x);
}

// Shared-memory view of one warp.  Point m of a lane's job (m = distance from the newest
// point, m = l + L k for the lane with index l in its group) sits at y[k * 32 + lane]:
// every access of the sweeps is lane-private and free of bank conflicts.
struct Lanes {
    double* y;         // [k_cap + 1][32]
    double* park;      // this lane's family of its job in [kParked][2 * jobs per warp] (one column per job and family)
    const double* wtab;
    int lane, L, l;
    __device__ __forceinline__ int park_stride() const { return 64 >> (__ffs(L) - 1); }   // 2 * (32 / L), L a power of two
    // extents, read by the bounds build only: the warp's slice [slice, slice + slice_len) and the weight table
    const double* slice;
    int slice_len, wtab_len;
    int32_t* err_word;
    __device__ __forceinline__ bool holds(const double* p) const {
        return index_ok(p - slice, slice_len, kErrShared, err_word);
    }
    __device__ __forceinline__ double weight(int m) const {
        return index_ok(m, wtab_len, kErrShared, err_word) ? wtab[m] : 0.0;
    }
    __device__ __forceinline__ double level(int k) const {   // the lane's point of row k
        const double* p = y + k * 32 + lane;
        return holds(p) ? *p : 0.0;
    }
};

// The window value at distance m + 1 from the newest point, seen from the lane that owns m.
__device__ __forceinline__ double older_neighbour(const Lanes& S, int k) {
    const double* p = S.l + 1 < S.L ? S.y + k * 32 + S.lane + 1 : S.y + (k + 1) * 32 + S.lane - (S.L - 1);
    return S.holds(p) ? *p : 0.0;
}

// What a lane keeps of one sweep: the sums of ITS family over the whole window.
// Family I (u = 1/q^2, J = (-u x^2, -u x, -u, 1)): v[0..4] = sum w u^2 x^k, v[5..7] = sum w u x^k,
// v[8..10] = sum w u r x^k, v[11] = sum w r, v[12] = S.
// Family II (J = (e, -x e, 1)): v[0..2] = sum w e^2 x^k, v[3..4] = sum w e x^k, v[5..6] = sum w e r x^k,
// v[7] = sum w r, v[8] = S.
struct SweepSums {
    double v[13];
    bool usable;   // the model was defined at every point and all sums are finite
};

// One sweep over the window: both families at once, each at its own point.  A lane adds up
// both families over its points; the first reduction step hands each lane of a pair the other
// lane's partial sums of its own family, the remaining steps run over lanes of the same parity.
__device__ __forceinline__ void sweep(const Lanes& S, int fam, int H, int k_all, double inv_span,
                                      const double (&pI)[4], bool doI, const double (&pII)[4], bool doII,
                                      SweepSums& out) {
    double m0 = 0, m1 = 0, m2 = 0, m3 = 0, m4 = 0, n0 = 0, n1 = 0, n2 = 0, h0 = 0, h1 = 0, h2 = 0, gd = 0, sI = 0;
    double e0 = 0, e1 = 0, e2 = 0, f0 = 0, f1 = 0, k0 = 0, k1 = 0, gc = 0, sII = 0;
    int feasible = 1;
    // e = exp(alpha - beta x) with x = -m / span grows geometrically with m: one exact value at
    // the lane's newest point, then a constant ratio per step.  The rounding of the recurrence
    // accumulates towards the old points, whose weights gamma^m have long vanished.
    double e = 0.0, ratio = 1.0;
    if (doII) {
        e = exp(fma(pII[1], (double)S.l * inv_span, pII[0]));
        ratio = exp(pII[1] * ((double)S.L * inv_span));
    }
    double md = (double)S.l;
    const double dL = (double)S.L;
    const double* yp = S.y + S.lane;
#pragma unroll 1   // unrolling only adds register pressure here: the body already holds 22 independent sums
    for (int k = 0, m = S.l; k < k_all; ++k, m += S.L, md += dL, yp += 32) {
        if (m < H) {
            const double x = -md * inv_span;
            const double w = S.weight(m);
            const double y = S.holds(yp) ? *yp : 0.0;
            const double x2 = x * x;
            if (doI) {
                const double q = fma(fma(pI[0], x, pI[1]), x, pI[2]);
                feasible &= q > 0.0 ? 1 : 0;
                const double inv = fast_rcp(q);
                const double r = y - (inv + pI[3]);
                const double u = inv * inv;
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
                sI = fma(wr, r, sI);
            }
            if (doII) {
                const double r = y - (e + pII[2]);
                const double we = w * e, wee = we * e, wer = we * r, wr = w * r;
                e0 += wee;
                e1 = fma(wee, x, e1);
                e2 = fma(wee, x2, e2);
                f0 += we;
                f1 = fma(we, x, f1);
                k0 += wer;
                k1 = fma(wer, x, k1);
                gc += wr;
                sII = fma(wr, r, sII);
            }
        }
        e *= ratio;
    }
    // pair step: an even lane hands over its family-II partials and receives family-I ones, an odd lane the reverse
    const bool odd = fam != 0;
    double v[13];
#define SLAQ_PAIR(k, a, b) v[k] = (odd ? (b) : (a)) + __shfl_xor_sync(kFull, odd ? (a) : (b), 1)
    SLAQ_PAIR(0, m0, e0); SLAQ_PAIR(1, m1, e1); SLAQ_PAIR(2, m2, e2); SLAQ_PAIR(3, m3, f0); SLAQ_PAIR(4, m4, f1);
    SLAQ_PAIR(5, n0, k0); SLAQ_PAIR(6, n1, k1); SLAQ_PAIR(7, n2, gc); SLAQ_PAIR(8, h0, sII);
#undef SLAQ_PAIR
    v[9] = h1 + __shfl_xor_sync(kFull, h1, 1);    // family I only: odd lanes carry these along unused
    v[10] = h2 + __shfl_xor_sync(kFull, h2, 1);
    v[11] = gd + __shfl_xor_sync(kFull, gd, 1);
    v[12] = sI + __shfl_xor_sync(kFull, sI, 1);
    feasible &= __shfl_xor_sync(kFull, feasible, 1);
    for (int o = 2; o < S.L; o <<= 1) {
#pragma unroll
        for (int k = 0; k < 13; ++k) v[k] += __shfl_xor_sync(kFull, v[k], o);
        feasible &= __shfl_xor_sync(kFull, feasible, o);
    }
    double chk = 0.0;
#pragma unroll
    for (int k = 0; k < 13; ++k) {
        out.v[k] = v[k];
        if (k < 9 || !odd) chk += v[k];
    }
    out.usable = finite_d(chk) && (odd || feasible);
}

}  // namespace slaq
