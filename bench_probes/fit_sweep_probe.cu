// The sweep of the curve fit, timed alone (a stand-alone program, not part of the library).
//
// Every warp of a 16-warp block per SM owns a slice of shared memory laid out as in the fit
// kernel, filled with a synthetic normalised window, and calls the library's own sweep function
// (paper_1802_04819_b200/csrc/slaq_fit_sweep.cuh) n_sweeps times at slowly moving parameters.
// Nothing else runs: no staging, no first guesses, no solver.  The SM cycles of the loop, read
// with clock64() around it, divided by (rows x sweeps x warps per sub-partition) give the cycles
// one sub-partition spends per warp row of 32 points when the fp64 pipe sees nothing but sweeps.
// Printed per (lanes per job L, rows per lane): cycles per warp row, and the same as a
// fraction of the 2-cycle issue rate of the sweep's fp64 instructions (46 per point).
//
//   fit_sweep_probe [n_sweeps]
#include <cstdio>
#include <cstdlib>
#include <vector>

#include <cuda_runtime.h>

#include "slaq_fit_sweep.cuh"

namespace {

constexpr int kWarps = 16;
constexpr int kSliceDoubles = 13824 / 8;
constexpr int kTable = 1000;

__global__ void __launch_bounds__(kWarps * 32, 1)
sweep_loop_kernel(const double* __restrict__ g_wtab, int L, int rows, int n_sweeps, int warps_active, double* out,
                  long long* cycles) {
    extern __shared__ double smem[];
    double* wtab = smem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kTable; i += blockDim.x) wtab[i] = g_wtab[i];
    double* const slice = smem + kTable + (size_t)warp * kSliceDoubles;
    slaq::Lanes S;
    S.wtab = wtab;
    S.lane = lane;
    S.L = L;
    S.l = lane & (L - 1);
    const int G = 32 / L;
    S.park = slice + 2 * (lane / L) + (lane & 1);
    S.y = slice + slaq::kParked * 2 * G;
    S.slice = slice;
    S.slice_len = kSliceDoubles;
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
            slaq::sweep(S, fam, H, rows, inv_span, pI, true, pII, true, sums);
            check += sums.v[fam ? 8 : 12];
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
    std::vector<double> tab(kTable);
    double wv = 1.0;
    for (int m = 0; m < kTable; ++m, wv *= 0.9) tab[m] = wv;
    double *d_tab = nullptr, *d_out = nullptr;
    long long* d_cycles = nullptr;
    const size_t smem = sizeof(double) * (kTable + (size_t)kWarps * kSliceDoubles);
    if (cudaMalloc(&d_tab, sizeof(double) * kTable) != cudaSuccess ||
        cudaMalloc(&d_out, sizeof(double) * sm_count * kWarps * 32) != cudaSuccess ||
        cudaMalloc(&d_cycles, sizeof(long long) * sm_count) != cudaSuccess)
        return 1;
    cudaMemcpy(d_tab, tab.data(), sizeof(double) * kTable, cudaMemcpyHostToDevice);
    if (cudaFuncSetAttribute(sweep_loop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        fprintf(stderr, "fit_sweep_probe: cannot get %zu bytes of shared memory\n", smem);
        return 1;
    }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    printf("%d SMs, %d sweeps per warp, both families in every sweep\n", sm_count, n_sweeps);
    printf("%4s %5s %9s %22s %20s %14s\n", "L", "rows", "warps/SM", "cycles/warp row/SMSP", "of 92 (2-cycle issue)", "ms");
    // rows a slice holds at L lanes per job: (slice - parked sums of its 32/L jobs) / 32 - 1 spare row, as in the library
    const int cases[][2] = {{2, 41}, {4, 47}, {8, 50}, {16, 51}, {32, 31}};
    std::vector<long long> cyc(sm_count);
    for (const auto& c : cases) {
        if (slaq::kParked * (64 / c[0]) + (c[1] + 1) * 32 > kSliceDoubles) {
            fprintf(stderr, "fit_sweep_probe: %d rows at L = %d do not fit a slice\n", c[1], c[0]);
            return 1;
        }
        for (int warps = 4; warps <= kWarps; warps += 4) {
            double best_cycles = 1e300;
            float best_ms = 1e30f;
            for (int rep = 0; rep < 4; ++rep) {   // the first repetition warms up
                cudaEventRecord(e0);
                sweep_loop_kernel<<<sm_count, kWarps * 32, smem>>>(d_tab, c[0], c[1], n_sweeps, warps, d_out, d_cycles);
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
            const double per_row = best_cycles / ((double)c[1] * n_sweeps * (warps / 4.0));
            printf("%4d %5d %9d %22.1f %20.3f %14.3f\n", c[0], c[1], warps, per_row, 92.0 / per_row, best_ms);
        }
    }
    cudaFree(d_tab);
    cudaFree(d_out);
    cudaFree(d_cycles);
    return 0;
}
