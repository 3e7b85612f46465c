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
    __device__ __forceinline__ double weight(const double* p) const {   // p = wtab + m
        return index_ok(p - wtab, wtab_len, kErrShared, err_word) ? *p : 0.0;
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

// Running sums to sums of powers of x.  A lane walks its points from the oldest to the newest and keeps, for a
// weighted value a, the chain c0 += a, c1 += c0, c2 += c1, ... in which every link adds the value its
// predecessor had one step earlier; after the walk c_p = sum a_k C(k, p), k = the row of the point counted from
// the lane's newest.  Powers of k are fixed combinations with positive coefficients (k^2 = 2 C(k,2) + C(k,1),
// k^3 = 6 C(k,3) + 6 C(k,2) + C(k,1), k^4 = 24 C(k,4) + 36 C(k,3) + 14 C(k,2) + C(k,1)); with x = x_l + g k
// (x_l <= 0 the lane's newest point, g < 0 the row pitch) the powers of x follow from a scaling by g^p and a shift
// of the origin, all of whose terms have the sign of (-1)^p: nothing cancels, the sums are as accurate as if the
// powers had been multiplied out point by point.
template <int P>
__device__ __forceinline__ void chains_to_powers(double (&c)[P], double x_l, double g) {
    const double c1 = P > 1 ? c[1] : 0.0, c2 = P > 2 ? c[2] : 0.0, c3 = P > 3 ? c[3] : 0.0;
    if (P > 2) c[2] = fma(2.0, c2, c1);
    if (P > 3) c[3] = fma(6.0, c3, fma(6.0, c2, c1));
    if (P > 4) c[4] = fma(24.0, c[4], fma(36.0, c3, fma(14.0, c2, c1)));
    double gp = g;
#pragma unroll
    for (int i = 1; i < P; ++i, gp *= g) c[i] *= gp;
#pragma unroll
    for (int j = 1; j < P; ++j)
#pragma unroll
        for (int p = P - 1; p >= j; --p) c[p] = fma(x_l, c[p - 1], c[p]);
}

// The running sums of one lane: family I (m: w u^2, n: w u, h: w u r, gd: w r, sI: w r^2 with u = 1/q^2) and
// family II (ee: w e^2, f: w e, kk: w e r, gc: w r, sII: w r^2).
struct LaneSums {
    double m[5], n[3], h[3], gd, sI;
    double ee[3], f[2], kk[2], gc, sII;
    int q_signs;     // OR of the high words of family I's denominators: negative if one of them had its sign bit set
};

// One point of a lane's walk: both families' values at the point and their running sums.
template <bool kI, bool kII>
__device__ __forceinline__ void add_point(const Lanes& S, const double* wp, const double* yp, double x,
                                          const double (&pI)[4], const double (&pII)[4], double& e, double ratio,
                                          LaneSums& a) {
    const double w = S.weight(wp);
    const double y = S.holds(yp) ? *yp : 0.0;
    if (kI) {
        const double q = fma(fma(pI[0], x, pI[1]), x, pI[2]);
        a.q_signs |= __double2hiint(q);   // q = 0 or NaN makes the sums non-finite, which the caller sees
        const double inv = fast_rcp(q);
        const double r = y - (inv + pI[3]);
        const double u = inv * inv;
        const double wu = w * u, wuu = wu * u, wur = wu * r, wr = w * r;
        a.m[4] += a.m[3]; a.m[3] += a.m[2]; a.m[2] += a.m[1]; a.m[1] += a.m[0]; a.m[0] += wuu;
        a.n[2] += a.n[1]; a.n[1] += a.n[0]; a.n[0] += wu;
        a.h[2] += a.h[1]; a.h[1] += a.h[0]; a.h[0] += wur;
        a.gd += wr;
        a.sI = fma(wr, r, a.sI);
    }
    if (kII) {
        const double r = y - (e + pII[2]);
        const double we = w * e, wee = we * e, wer = we * r, wr = w * r;
        a.ee[2] += a.ee[1]; a.ee[1] += a.ee[0]; a.ee[0] += wee;
        a.f[1] += a.f[0]; a.f[0] += we;
        a.kk[1] += a.kk[0]; a.kk[0] += wer;
        a.gc += wr;
        a.sII = fma(wr, r, a.sII);
        e *= ratio;
    }
}

// The walk over a lane's rows, oldest first.  kI / kII: whether the family is evaluated at all - the same for
// the whole warp, so that the loop has no branch per family (a lane whose family has no trial computes it at
// parameters nobody uses and its sums are discarded).  Branches inside the loop cost issue slots on every row:
// the rows that every lane of the warp has are walked without a test, only the ragged rest with one.
template <bool kI, bool kII>
__device__ __forceinline__ void walk_rows(const Lanes& S, int k_last, int k_all, double inv_span,
                                          const double (&pI)[4], const double (&pII)[4], LaneSums& a) {
    const int mi = S.l + k_last * S.L;
    const double md = (double)mi;
    const double dL = (double)S.L;
    // x from the lane's oldest point by one addition per row (its rounding, at most a few 1e-15 absolute at the
    // newest point, moves the predictions as little as the exponential's recurrence does: measured)
    double x = -md * inv_span;
    const double hx = dL * inv_span;
    // e = exp(alpha - beta x) with x = -m / span falls geometrically towards the newest point: one
    // exact value at the lane's oldest point, then a constant ratio per step.  (Choosing the start such
    // that the recurrence lands on the exact value at the newest point was measured: the predictions stay
    // as close to the reference's either way, and the extra arithmetic costs 2 % of the kernel.)
    double e = 0.0, ratio = 1.0;
    if (kII) {
        e = exp(fma(pII[1], md * inv_span, pII[0]));
        ratio = exp(-pII[1] * (dL * inv_span));
    }
    const double* yp = S.y + S.lane + k_last * 32;
    const double* wp = S.wtab + mi;
    const int k_min = __reduce_min_sync(kFull, k_last);
    int i = 0;
#pragma unroll 1   // unrolling was measured (2 rows per step): slower, more spills
    for (; i <= k_min; ++i, x += hx, yp -= 32, wp -= S.L) add_point<kI, kII>(S, wp, yp, x, pI, pII, e, ratio, a);
#pragma unroll 1
    for (; i < k_all; ++i, x += hx, yp -= 32, wp -= S.L)
        if (i <= k_last) add_point<kI, kII>(S, wp, yp, x, pI, pII, e, ratio, a);   // row k_last - i >= 0
}

// One sweep over the window: both families at once, each at its own point.  A lane adds up
// both families over its points, oldest first, as running sums (see chains_to_powers: in the loop
// every accumulation but the two objectives is an addition of two registers, which the fp64 pipe
// issues in two cycles where a fused multiply-add on three registers takes three); the first
// reduction step hands each lane of a pair the other lane's partial sums of its own family, the
// remaining steps run over lanes of the same parity.
__device__ __forceinline__ void sweep(const Lanes& S, int fam, int H, int k_all, double inv_span,
                                      const double (&pI)[4], bool doI, const double (&pII)[4], bool doII,
                                      SweepSums& out) {
    LaneSums a = {};
    const int shift = __ffs(S.L) - 1;                                      // L is a power of two
    const int k_last = H - 1 - S.l >= 0 ? (H - 1 - S.l) >> shift : -1;     // the row of the lane's oldest point
    const bool anyI = __any_sync(kFull, doI), anyII = __any_sync(kFull, doII);
    if (anyI && anyII) {
        walk_rows<true, true>(S, k_last, k_all, inv_span, pI, pII, a);
    } else {   // one family has no trial left in the whole warp
        if (anyI) walk_rows<true, false>(S, k_last, k_all, inv_span, pI, pII, a);
        if (anyII) walk_rows<false, true>(S, k_last, k_all, inv_span, pI, pII, a);
    }
    double (&m)[5] = a.m, (&n)[3] = a.n, (&h)[3] = a.h, (&ee)[3] = a.ee, (&f)[2] = a.f, (&kk)[2] = a.kk;
    const double gd = a.gd, sI = a.sI, gc = a.gc, sII = a.sII;
    int feasible = a.q_signs >= 0 ? 1 : 0;
    const double dL = (double)S.L;
    const double x_l = -(double)S.l * inv_span, g = -dL * inv_span;
    chains_to_powers(m, x_l, g);
    chains_to_powers(n, x_l, g);
    chains_to_powers(h, x_l, g);
    chains_to_powers(ee, x_l, g);
    chains_to_powers(f, x_l, g);
    chains_to_powers(kk, x_l, g);
    // pair step: an even lane hands over its family-II partials and receives family-I ones, an odd lane the reverse
    const bool odd = fam != 0;
    double v[13];
#define SLAQ_PAIR(k, a, b) v[k] = (odd ? (b) : (a)) + __shfl_xor_sync(kFull, odd ? (a) : (b), 1)
    SLAQ_PAIR(0, m[0], ee[0]); SLAQ_PAIR(1, m[1], ee[1]); SLAQ_PAIR(2, m[2], ee[2]); SLAQ_PAIR(3, m[3], f[0]);
    SLAQ_PAIR(4, m[4], f[1]); SLAQ_PAIR(5, n[0], kk[0]); SLAQ_PAIR(6, n[1], kk[1]); SLAQ_PAIR(7, n[2], gc);
    SLAQ_PAIR(8, h[0], sII);
#undef SLAQ_PAIR
    v[9] = h[1] + __shfl_xor_sync(kFull, h[1], 1);    // family I only: odd lanes carry these along unused
    v[10] = h[2] + __shfl_xor_sync(kFull, h[2], 1);
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
