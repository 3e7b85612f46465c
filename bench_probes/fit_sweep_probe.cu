// The sweep of the curve fit, timed alone (a stand-alone program, not part of the library).
//
// Every warp of a 16-warp block per SM owns a slice of shared memory laid out as in the fit
// kernel, filled with a synthetic normalised window, and calls the library's own sweep function
// (paper_1802_04819_b200/csrc/slaq_fit_sweep.cuh) n_sweeps times at slowly moving parameters.
// Nothing else runs: no staging, no first guesses, no solver.  The SM cycles of the loop, read
// with clock64() around it, divided by (rows x sweeps x warps per sub-partition) give the cycles
// one sub-partition spends per warp row of 32 points when the fp64 pipe sees nothing but sweeps.
// Printed per (lanes per job L, rows per lane): cycles per warp row, and the same as a
// fraction of the 2-cycle issue rate of the variant's fp64 instructions (43 per point in the library's sweep).
//
//   fit_sweep_probe [n_sweeps]
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <vector>

#include <cuda_runtime.h>

#include "slaq_fit_sweep.cuh"

namespace {

// An alternative that was measured and not adopted: the same sweep with the powers of x taken out of the
// point loop (tables tab[p * ts + m] = gamma^m m^p, p = 0..4, in shared memory).  x = -m / span, so
// sum w v x^p = (-1 / span)^p sum (gamma^m m^p) v: with the weighted powers gamma^m m^p in shared-memory
// tables every accumulation is one fused multiply-add of (table entry, value, sum), the products with
// w, x and x^2 disappear from the loop, and the sums are scaled once after it.  q is evaluated in
// the point index as well: q = (a / span^2) m^2 - (b / span) m + c.
__device__ __forceinline__ void sweep_tables(const slaq::Lanes& S, int ts, int fam, int H, int k_all, double inv_span,
                                             const double (&pI)[4], bool doI, const double (&pII)[4], bool doII,
                                             slaq::SweepSums& out) {
    double m0 = 0, m1 = 0, m2 = 0, m3 = 0, m4 = 0, n0 = 0, n1 = 0, n2 = 0, h0 = 0, h1 = 0, h2 = 0, gd = 0, sI = 0;
    double e0 = 0, e1 = 0, e2 = 0, f0 = 0, f1 = 0, k0 = 0, k1 = 0, gc = 0, sII = 0;
    int feasible = 1;
    double e = 0.0, ratio = 1.0;
    if (doII) {
        e = exp(fma(pII[1], (double)S.l * inv_span, pII[0]));
        ratio = exp(pII[1] * ((double)S.L * inv_span));
    }
    const double qa = pI[0] * inv_span * inv_span, qb = -pI[1] * inv_span, qc = pI[2], dI = pI[3], cII = pII[2];
    double md = (double)S.l;
    const double dL = (double)S.L;
    const double* yp = S.y + S.lane;
    const double* tp = S.wtab + S.l;
#pragma unroll 1
    for (int k = 0, m = S.l; k < k_all; ++k, m += S.L, md += dL, yp += 32, tp += S.L) {
        if (m < H) {
            const bool ok = (m < S.wtab_len);
            const double t0 = ok ? tp[0] : 0.0, t1 = ok ? tp[ts] : 0.0, t2 = ok ? tp[2 * ts] : 0.0;
            const double y = S.holds(yp) ? *yp : 0.0;
            if (doI) {
                const double t3 = ok ? tp[3 * ts] : 0.0, t4 = ok ? tp[4 * ts] : 0.0;
                const double q = fma(fma(qa, md, qb), md, qc);
                feasible &= q > 0.0 ? 1 : 0;
                const double inv = slaq::fast_rcp(q);
                const double r = (y - dI) - inv;
                const double u = inv * inv;
                const double uu = u * u, ur = u * r;
                m0 = fma(t0, uu, m0);
                m1 = fma(t1, uu, m1);
                m2 = fma(t2, uu, m2);
                m3 = fma(t3, uu, m3);
                m4 = fma(t4, uu, m4);
                n0 = fma(t0, u, n0);
                n1 = fma(t1, u, n1);
                n2 = fma(t2, u, n2);
                h0 = fma(t0, ur, h0);
                h1 = fma(t1, ur, h1);
                h2 = fma(t2, ur, h2);
                gd = fma(t0, r, gd);
                sI = fma(t0 * r, r, sI);
            }
            if (doII) {
                const double r = (y - cII) - e;
                const double ee = e * e, er = e * r;
                e0 = fma(t0, ee, e0);
                e1 = fma(t1, ee, e1);
                e2 = fma(t2, ee, e2);
                f0 = fma(t0, e, f0);
                f1 = fma(t1, e, f1);
                k0 = fma(t0, er, k0);
                k1 = fma(t1, er, k1);
                gc = fma(t0, r, gc);
                sII = fma(t0 * r, r, sII);
            }
        }
        e *= ratio;
    }
    // back to powers of x = -m / span
    const double s1 = -inv_span, s2 = inv_span * inv_span, s3 = s1 * s2, s4 = s2 * s2;
    m1 *= s1; m2 *= s2; m3 *= s3; m4 *= s4;
    n1 *= s1; n2 *= s2;
    h1 *= s1; h2 *= s2;
    e1 *= s1; e2 *= s2;
    f1 *= s1;
    k1 *= s1;
    const bool odd = fam != 0;
    double v[13];
#define SLAQ_PAIR(k, a, b) v[k] = (odd ? (b) : (a)) + __shfl_xor_sync(slaq::kFull, odd ? (a) : (b), 1)
    SLAQ_PAIR(0, m0, e0); SLAQ_PAIR(1, m1, e1); SLAQ_PAIR(2, m2, e2); SLAQ_PAIR(3, m3, f0); SLAQ_PAIR(4, m4, f1);
    SLAQ_PAIR(5, n0, k0); SLAQ_PAIR(6, n1, k1); SLAQ_PAIR(7, n2, gc); SLAQ_PAIR(8, h0, sII);
#undef SLAQ_PAIR
    v[9] = h1 + __shfl_xor_sync(slaq::kFull, h1, 1);
    v[10] = h2 + __shfl_xor_sync(slaq::kFull, h2, 1);
    v[11] = gd + __shfl_xor_sync(slaq::kFull, gd, 1);
    v[12] = sI + __shfl_xor_sync(slaq::kFull, sI, 1);
    feasible &= __shfl_xor_sync(slaq::kFull, feasible, 1);
    for (int o = 2; o < S.L; o <<= 1) {
#pragma unroll
        for (int k = 0; k < 13; ++k) v[k] += __shfl_xor_sync(slaq::kFull, v[k], o);
        feasible &= __shfl_xor_sync(slaq::kFull, feasible, o);
    }
    double chk = 0.0;
#pragma unroll
    for (int k = 0; k < 13; ++k) {
        out.v[k] = v[k];
        if (k < 9 || !odd) chk += v[k];
    }
    out.usable = slaq::finite_d(chk) && (odd || feasible);
}

// A second alternative, the library's sweep until the running sums replaced it: the powers of x multiplied out
// point by point (x, x^2 and w u^2 x^2 formed in the loop, 13 of the 22 accumulations fused multiply-adds on three
// different registers): 46 fp64 instructions per point instead of 43, 19 fused multiply-adds instead of 8.
__device__ __forceinline__ void sweep_products(const slaq::Lanes& S, int fam, int H, int k_all, double inv_span,
                                               const double (&pI)[4], bool doI, const double (&pII)[4], bool doII,
                                               slaq::SweepSums& out) {
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
                const double inv = slaq::fast_rcp(q);
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
#define SLAQ_PAIR(k, a, b) v[k] = (odd ? (b) : (a)) + __shfl_xor_sync(slaq::kFull, odd ? (a) : (b), 1)
    SLAQ_PAIR(0, m0, e0); SLAQ_PAIR(1, m1, e1); SLAQ_PAIR(2, m2, e2); SLAQ_PAIR(3, m3, f0); SLAQ_PAIR(4, m4, f1);
    SLAQ_PAIR(5, n0, k0); SLAQ_PAIR(6, n1, k1); SLAQ_PAIR(7, n2, gc); SLAQ_PAIR(8, h0, sII);
#undef SLAQ_PAIR
    v[9] = h1 + __shfl_xor_sync(slaq::kFull, h1, 1);    // family I only: odd lanes carry these along unused
    v[10] = h2 + __shfl_xor_sync(slaq::kFull, h2, 1);
    v[11] = gd + __shfl_xor_sync(slaq::kFull, gd, 1);
    v[12] = sI + __shfl_xor_sync(slaq::kFull, sI, 1);
    feasible &= __shfl_xor_sync(slaq::kFull, feasible, 1);
    for (int o = 2; o < S.L; o <<= 1) {
#pragma unroll
        for (int k = 0; k < 13; ++k) v[k] += __shfl_xor_sync(slaq::kFull, v[k], o);
        feasible &= __shfl_xor_sync(slaq::kFull, feasible, o);
    }
    double chk = 0.0;
#pragma unroll
    for (int k = 0; k < 13; ++k) {
        out.v[k] = v[k];
        if (k < 9 || !odd) chk += v[k];
    }
    out.usable = slaq::finite_d(chk) && (odd || feasible);
}

constexpr int kWarps = 16;
constexpr int kSliceDoubles = 13824 / 8;
constexpr int kTable = 1000;

// kVariant 0: the library's sweep; 1: the weighted powers of the point index in shared-memory tables (5 tables,
// smaller slices); 2: the powers of x multiplied out in the loop
template <int kVariant>
__global__ void __launch_bounds__(kWarps * 32, 1)
sweep_loop_kernel(const double* __restrict__ g_wtab, int L, int rows, int n_sweeps, int warps_active, double* out,
                  long long* cycles, int slice_doubles, double* last_sums) {
    extern __shared__ double smem[];
    double* wtab = smem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kTabs = kVariant == 1 ? 5 : 1;
    for (int i = threadIdx.x; i < kTabs * kTable; i += blockDim.x) wtab[i] = g_wtab[i];
    double* const slice = smem + kTabs * kTable + (size_t)warp * slice_doubles;
    slaq::Lanes S;
    S.wtab = wtab;
    S.lane = lane;
    S.L = L;
    S.l = lane & (L - 1);
    const int G = 32 / L;
    S.park = slice + 2 * (lane / L) + (lane & 1);
    S.y = slice + slaq::kParked * 2 * G;
    S.slice = slice;
    S.slice_len = slice_doubles;
    S.wtab_len = kTable;
    S.err_word = nullptr;
    const int H = rows * L;
    const double span = (double)(H - 1), inv_span = 1.0 / span;
    // a window that falls like 1/(a k^2 + b k + c) + d, newest point last, in normalised units
    for (int k = 0; k < rows; ++k) {
        const int m = S.l + L * k;
        const double kk = (double)(H - 1 - m);
        S.y[k * 32 + lane] = 40.0 / (1e-3 * kk * kk + 0.2 * kk + 1.0) + 0.5 + 1e-3 * ((m * 37) % 11);
    }
    __syncthreads();
    double pI[4] = {1e-3 * span * span / 40.0, (2e-3 * span * span + 0.2 * span) / 40.0,
                    (1e-3 * span * span + 0.2 * span + 1.0) / 40.0, 0.45};   // the same curve in window coordinates
    double pII[4] = {-0.2, 3.0, 0.4, 0.0};
    const int fam = lane & 1;
    double check = 0.0;
    long long t0 = 0;
    if (threadIdx.x == 0) t0 = clock64();
    if (warp < warps_active) {
        for (int it = 0; it < n_sweeps; ++it) {
            slaq::SweepSums sums;
            if (kVariant == 1) sweep_tables(S, kTable, fam, H, rows, inv_span, pI, true, pII, true, sums);
            else if (kVariant == 2) sweep_products(S, fam, H, rows, inv_span, pI, true, pII, true, sums);
            else slaq::sweep(S, fam, H, rows, inv_span, pI, true, pII, true, sums);
            check += sums.v[fam ? 8 : 12];
            if (it == n_sweeps - 1 && blockIdx.x == 0 && warp == 0)
                for (int i = 0; i < 13; ++i) last_sums[lane * 13 + i] = (i < 9 || !fam) ? sums.v[i] : 0.0;
            // move the points a little, as accepted trials do (keeps every sweep's arithmetic live)
            pI[2] = fma(pI[2], 1.0 + 1e-9, sums.usable ? 0.0 : 1e-12);
            pII[0] = fma(pII[0], 1.0 - 1e-9, 0.0);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = clock64() - t0;
    out[blockIdx.x * blockDim.x + threadIdx.x] = check;
}

}  // namespace

int main(int argc, char** argv) {
    const int n_sweeps = argc > 1 ? atoi(argv[1]) : 400;
    int sm_count = 0;
    if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, 0) != cudaSuccess || sm_count <= 0) {
        fprintf(stderr, "fit_sweep_probe: no CUDA device\n");
        return 1;
    }
    std::vector<double> tab(5 * kTable);
    double wv = 1.0;
    for (int m = 0; m < kTable; ++m, wv *= 0.9) {
        double pw = wv;
        for (int p = 0; p < 5; ++p, pw *= (double)m) tab[p * kTable + m] = pw;
    }
    double *d_tab = nullptr, *d_out = nullptr;
    long long* d_cycles = nullptr;
    if (cudaMalloc(&d_tab, sizeof(double) * 5 * kTable) != cudaSuccess ||
        cudaMalloc(&d_out, sizeof(double) * sm_count * kWarps * 32) != cudaSuccess ||
        cudaMalloc(&d_cycles, sizeof(long long) * sm_count) != cudaSuccess)
        return 1;
    cudaMemcpy(d_tab, tab.data(), sizeof(double) * 5 * kTable, cudaMemcpyHostToDevice);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    printf("%d SMs, %d sweeps per warp, both families in every sweep\n", sm_count, n_sweeps);
    std::vector<long long> cyc(sm_count);
    double* d_last = nullptr;
    if (cudaMalloc(&d_last, sizeof(double) * 32 * 13) != cudaSuccess) return 1;
    std::vector<double> last_lib(5 * 32 * 13, 0.0), last(32 * 13);
    const char* const names[3] = {"the library's sweep (powers of x by running sums)", "weighted powers from tables",
                                  "powers of x multiplied in the loop"};
    const double kInstr[3] = {43.0, 41.0, 46.0};   // fp64 arithmetic instructions per point in the loop, from the source
    for (int variant = 0; variant < 3; ++variant) {
        // the tables take 4 x kTable doubles more of the SM's shared memory: the sixteen slices shrink accordingly
        const int slice_doubles = variant != 1 ? kSliceDoubles : (kSliceDoubles * kWarps - 4 * kTable) / kWarps / 32 * 32;
        const size_t smem = sizeof(double) * ((variant != 1 ? 1 : 5) * kTable + (size_t)kWarps * slice_doubles);
        auto kernel = variant == 0 ? sweep_loop_kernel<0> : variant == 1 ? sweep_loop_kernel<1> : sweep_loop_kernel<2>;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            fprintf(stderr, "fit_sweep_probe: cannot get %zu bytes of shared memory\n", smem);
            return 1;
        }
        printf("%s, %d doubles per slice\n", names[variant], slice_doubles);
        printf("%4s %5s %9s %22s %20s %14s\n", "L", "rows", "warps/SM", "cycles/warp row/SMSP", "of 2-cycle issue", "ms");
        // rows a slice holds at L lanes per job: (slice - parked sums of its 32/L jobs) / 32 - 1 spare row, as in the library
        const int Ls[5] = {2, 4, 8, 16, 32};
        for (int li = 0; li < 5; ++li) {
            const int L = Ls[li];
            int rows = (slice_doubles - slaq::kParked * (64 / L)) / 32 - 1;
            if (rows * L > kTable - 8) rows = (kTable - 8) / L;
            if (rows < 1 || slaq::kParked * (64 / L) + (rows + 1) * 32 > slice_doubles) {
                fprintf(stderr, "fit_sweep_probe: no room for L = %d\n", L);
                return 1;
            }
            for (int warps = 4; warps <= kWarps; warps += 4) {
                double best_cycles = 1e300;
                float best_ms = 1e30f;
                for (int rep = 0; rep < 4; ++rep) {   // the first repetition warms up
                    cudaEventRecord(e0);
                    kernel<<<sm_count, kWarps * 32, smem>>>(d_tab, L, rows, n_sweeps, warps, d_out, d_cycles, slice_doubles, d_last);
                    cudaEventRecord(e1);
                    const cudaError_t err = cudaDeviceSynchronize();
                    if (err != cudaSuccess) {
                        fprintf(stderr, "fit_sweep_probe: kernel failed: %s\n", cudaGetErrorString(err));
                        return 1;
                    }
                    float ms = 0.f;
                    cudaEventElapsedTime(&ms, e0, e1);
                    cudaMemcpy(cyc.data(), d_cycles, sizeof(long long) * sm_count, cudaMemcpyDeviceToHost);
                    double mean = 0.0;
                    for (long long v : cyc) mean += (double)v;
                    mean /= sm_count;
                    if (rep > 0 && mean < best_cycles) best_cycles = mean, best_ms = ms;
                }
                const double per_row = best_cycles / ((double)rows * n_sweeps * (warps / 4.0));
                printf("%4d %5d %9d %22.1f %20.3f %14.3f\n", L, rows, warps, per_row, 2.0 * kInstr[variant] / per_row, best_ms);
            }
            // the sums of the last sweep of block 0's first warp: the multiplied-out variant against the library's
            cudaMemcpy(last.data(), d_last, sizeof(double) * 32 * 13, cudaMemcpyDeviceToHost);
            if (variant == 0) std::copy(last.begin(), last.end(), last_lib.begin() + li * 32 * 13);
            if (variant == 2) {
                double worst = 0.0;
                for (int i = 0; i < 32 * 13; ++i) {
                    const double ref = last_lib[li * 32 * 13 + i];
                    if (ref != 0.0) worst = std::max(worst, std::fabs(last[i] - ref) / std::fabs(ref));
                }
                printf("     largest relative difference of a sum from the library's sweep: %.2e\n", worst);
            }
        }
    }
    cudaFree(d_tab);
    cudaFree(d_out);
    cudaFree(d_cycles);
    cudaFree(d_last);
    return 0;
}
