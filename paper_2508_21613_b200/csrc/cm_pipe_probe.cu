// Pipe-rate probe: how many scheduler cycles the recurrence cell of the plan search costs
// on this GPU.  Stand-alone program (not part of libchameleon.so); it backs the issue-bound
// peak that bench.py reports against: `python -m paper_2508_21613_b200.pipe_probe`.
//
// Every kernel runs 8 independent dependency chains per thread, 8 CTAs of 256 threads per SM,
// so the result is a throughput, not a latency.  Printed: items per clock per SM (at the
// SM clock given on the command line, default 1965 MHz) and scheduler cycles per warp-item
// (4 schedulers x 32 lanes per SM).
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#define CHAINS 8

template <int OP>
__global__ void probe(double *out, int iters, double seed) {
    double a[CHAINS], b = seed * 1e-3 + 1.0;
    long long ia[CHAINS], ib = (long long)(seed * 7) + 3;
#pragma unroll
    for (int u = 0; u < CHAINS; ++u) { a[u] = seed + u + threadIdx.x; ia[u] = (long long)(seed * 3) + u + threadIdx.x; }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < CHAINS; ++u) {
            const int v = (u + 1) % CHAINS;
            if (OP == 0) a[u] = a[u] + b;                                                        // fp64 add
            if (OP == 1) { const double s = a[u] + b; a[u] = s > a[v] ? s : a[v]; }              // add + max
            if (OP == 2) { const double d = a[v] + b; const double s = a[u] > d ? a[u] : d; a[u] = s + b; }  // cell, fp64
            if (OP == 3) { const long long x = __double_as_longlong(a[u]), y = __double_as_longlong(a[v] + b);
                           a[u] = __longlong_as_double(x > y ? x : y) + b; }                     // cell, max on bit patterns
            if (OP == 4) { const long long d = ia[v] + ib; const long long s = ia[u] > d ? ia[u] : d; ia[u] = s + ib; }  // cell, int64
        }
    }
    double s = 0;
    long long is = 0;
#pragma unroll
    for (int u = 0; u < CHAINS; ++u) { s += a[u]; is += ia[u]; }
    out[blockIdx.x * blockDim.x + threadIdx.x] = s + (double)is;
}

template <int OP>
static void run(const char *name, int n_sm, double mhz) {
    const int blocks = n_sm * 8, threads = 256, iters = 4096;
    double *out;
    cudaMalloc(&out, (size_t)blocks * threads * sizeof(double));
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    probe<OP><<<blocks, threads>>>(out, 64, 1.0);
    cudaEventRecord(e0);
    probe<OP><<<blocks, threads>>>(out, iters, 1.0);
    cudaEventRecord(e1);
    cudaDeviceSynchronize();
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    const double items = (double)blocks * threads * iters * CHAINS;
    const double per_clk_sm = items / (ms * 1e-3) / n_sm / (mhz * 1e6);
    printf("%-34s %8.3f ms  %7.2f items/clk/SM  %6.2f scheduler cycles per warp-item\n", name, ms, per_clk_sm, 128.0 / per_clk_sm);
    cudaFree(out);
}

int main(int argc, char **argv) {
    const double mhz = argc > 1 ? atof(argv[1]) : 1965.0;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { fprintf(stderr, "no CUDA device\n"); return 1; }
    printf("%s, %d SMs, assuming %.0f MHz\n", prop.name, prop.multiProcessorCount, mhz);
    run<0>("fp64 add", prop.multiProcessorCount, mhz);
    run<1>("fp64 add + max", prop.multiProcessorCount, mhz);
    run<2>("cell fp64 (add, max, add)", prop.multiProcessorCount, mhz);
    run<3>("cell fp64, max on bit patterns", prop.multiProcessorCount, mhz);
    run<4>("cell int64 (add, max, add)", prop.multiProcessorCount, mhz);
    return 0;
}
