// Issue rate of the fp64 pipe for different operand patterns (a stand-alone program, not part
// of the library): the denominator behind the fit kernel's roofline.
//
// Every thread keeps 12 independent accumulators and updates them n_iter times with one
// instruction each, so the dependent-issue latency is covered and the time per warp
// instruction is what one SM sub-partition can issue.  Patterns:
//   fma3   acc = fma(a_i, b_i, acc)   three different registers per instruction
//   fma2   acc = fma(a_i, c,   acc)   one operand shared by all instructions
//   fma1   acc = fma(c,   d,   acc)   two operands shared
//   add    acc = acc + a_i
//   mul    acc = acc * a_i
// Prints cycles per warp instruction and sub-partition at the SM clock given on the command
// line (MHz, default 1965) for 4, 8 and 16 warps per SM.
#include <cstdio>
#include <cstdlib>

#include <cuda_runtime.h>

namespace {

constexpr int kAcc = 12;

template <int kPattern>
__global__ void __launch_bounds__(512, 1) probe_kernel(double* out, const double* in, int n_iter) {
    double acc[kAcc], a[kAcc], b[kAcc];
#pragma unroll
    for (int i = 0; i < kAcc; ++i) {
        acc[i] = in[i] * threadIdx.x;
        a[i] = in[kAcc + i] + threadIdx.x * 1e-9;
        b[i] = in[2 * kAcc + i] - threadIdx.x * 1e-9;
    }
    const double c = a[0], d = b[0];
    for (int it = 0; it < n_iter; ++it) {
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            if (kPattern == 0) acc[i] = fma(a[i], b[i], acc[i]);
            else if (kPattern == 1) acc[i] = fma(a[i], d, acc[i]);
            else if (kPattern == 2) acc[i] = fma(c, d, acc[i]);
            else if (kPattern == 3) acc[i] = acc[i] + a[i];
            else acc[i] = acc[i] * a[i];
        }
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < kAcc; ++i) s += acc[i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace

int main(int argc, char** argv) {
    const double mhz = argc > 1 ? atof(argv[1]) : 1965.0;
    const int n_iter = 20000;
    int sm_count = 0;
    if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, 0) != cudaSuccess || sm_count <= 0) {
        fprintf(stderr, "fp64_issue_probe: no CUDA device\n");
        return 1;
    }
    double h[3 * kAcc];
    for (int i = 0; i < 3 * kAcc; ++i) h[i] = 1.0 + 1e-3 * i;
    double *d_in = nullptr, *d_out = nullptr;
    if (cudaMalloc(&d_in, sizeof h) != cudaSuccess || cudaMalloc(&d_out, (size_t)sm_count * 512 * sizeof(double)) != cudaSuccess)
        return 1;
    cudaMemcpy(d_in, h, sizeof h, cudaMemcpyHostToDevice);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    void (*kernels[5])(double*, const double*, int) = {probe_kernel<0>, probe_kernel<1>, probe_kernel<2>, probe_kernel<3>,
                                                      probe_kernel<4>};
    const char* names[5] = {"fma3", "fma2", "fma1", "add", "mul"};
    printf("%d SMs, SM clock taken as %.0f MHz\n", sm_count, mhz);
    printf("%-6s %10s %22s %12s\n", "op", "warps/SM", "cycles/warp-instr/SMSP", "TFLOP/s");
    for (int warps = 4; warps <= 16; warps *= 2) {
        for (int v = 0; v < 5; ++v) {
            float best = 1e30f;
            for (int rep = 0; rep < 4; ++rep) {   // the first repetition warms up
                cudaEventRecord(e0);
                kernels[v]<<<sm_count, warps * 32>>>(d_out, d_in, n_iter);
                cudaEventRecord(e1);
                if (cudaDeviceSynchronize() != cudaSuccess) {
                    fprintf(stderr, "fp64_issue_probe: kernel failed\n");
                    return 1;
                }
                float ms = 0.f;
                cudaEventElapsedTime(&ms, e0, e1);
                if (rep > 0 && ms < best) best = ms;
            }
            const double instr_per_smsp = (double)n_iter * kAcc * warps / 4.0;
            const double flop = (double)n_iter * kAcc * warps * 32.0 * sm_count * (v <= 2 ? 2.0 : 1.0);
            printf("%-6s %10d %22.2f %12.2f\n", names[v], warps, best * 1e-3 * mhz * 1e6 / instr_per_smsp,
                   flop / (best * 1e-3) / 1e12);
        }
    }
    cudaFree(d_in);
    cudaFree(d_out);
    return 0;
}
