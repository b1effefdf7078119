// Register-resident FP64 rate probes: the denominators of the base-product roofline.
// No memory traffic inside the loops; every thread keeps 8 independent accumulator chains.
#include "kernels.h"

namespace strassen {

namespace {

constexpr int PROBE_THREADS = 256;
constexpr int CHAINS = 8;

// Keeps the loops alive without an output buffer (so the probe allocates nothing): a thread stores its sum only
// if it equals a value the loops cannot produce.
__device__ double g_probe_sink;
constexpr double kNever = -1.2345678901234567e300;

__global__ void __launch_bounds__(PROBE_THREADS) probe_dfma_kernel(long long iters, double x, double y)
{
    double a[CHAINS];
#pragma unroll
    for (int c = 0; c < CHAINS; ++c) a[c] = double(threadIdx.x + c);
    for (long long i = 0; i < iters; ++i) {
#pragma unroll
        for (int c = 0; c < CHAINS; ++c) a[c] = fma(a[c], x, y);
    }
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < CHAINS; ++c) s += a[c];
    if (s == kNever) g_probe_sink = s;
}

template <int KIND>
__global__ void __launch_bounds__(PROBE_THREADS) probe_dmma_kernel(long long iters, double x, double y)
{
    double d[CHAINS][4];
#pragma unroll
    for (int c = 0; c < CHAINS; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) d[c][e] = double(threadIdx.x + c + e);
    const double a0 = x, a1 = x + 1, a2 = x + 2, a3 = x + 3, a4 = x + 4, a5 = x + 5, a6 = x + 6, a7 = x + 7;
    const double b0 = y, b1 = y + 1, b2 = y + 2, b3 = y + 3;
    for (long long i = 0; i < iters; ++i) {
#pragma unroll
        for (int c = 0; c < CHAINS; ++c) {
            if (KIND == 1)
                asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
                             : "+d"(d[c][0]), "+d"(d[c][1]) : "d"(a0), "d"(b0));
            else if (KIND == 2)
                asm volatile("mma.sync.aligned.m16n8k4.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
                             : "+d"(d[c][0]), "+d"(d[c][1]), "+d"(d[c][2]), "+d"(d[c][3]) : "d"(a0), "d"(a1), "d"(b0));
            else if (KIND == 3)
                asm volatile("mma.sync.aligned.m16n8k8.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                             : "+d"(d[c][0]), "+d"(d[c][1]), "+d"(d[c][2]), "+d"(d[c][3])
                             : "d"(a0), "d"(a1), "d"(a2), "d"(a3), "d"(b0), "d"(b1));
            else
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, {%12,%13,%14,%15}, {%0,%1,%2,%3};\n"
                             : "+d"(d[c][0]), "+d"(d[c][1]), "+d"(d[c][2]), "+d"(d[c][3])
                             : "d"(a0), "d"(a1), "d"(a2), "d"(a3), "d"(a4), "d"(a5), "d"(a6), "d"(a7), "d"(b0), "d"(b1),
                               "d"(b2), "d"(b3));
        }
    }
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < CHAINS; ++c) s += d[c][0] + d[c][1] + d[c][2] + d[c][3];
    if (s == kNever) g_probe_sink = s;
}

}  // namespace

cudaError_t probe_fp64(int kind, long long iters, cudaStream_t stream, double *tflops_out)
{
    if (kind < 0 || kind > 4 || iters < 1 || !tflops_out) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int blocks = sms * 4;
    cudaEvent_t t0, t1;
    cudaEventCreate(&t0);
    cudaEventCreate(&t1);
    float ms = 0.f;
    for (int rep = 0; rep < 2; ++rep) {   // first pass warms up, second is timed
        cudaEventRecord(t0, stream);
        switch (kind) {
        case 0: probe_dfma_kernel<<<blocks, PROBE_THREADS, 0, stream>>>(iters, 0.999999, 1e-9); break;
        case 1: probe_dmma_kernel<1><<<blocks, PROBE_THREADS, 0, stream>>>(iters, 1e-3, 1e-3); break;
        case 2: probe_dmma_kernel<2><<<blocks, PROBE_THREADS, 0, stream>>>(iters, 1e-3, 1e-3); break;
        case 3: probe_dmma_kernel<3><<<blocks, PROBE_THREADS, 0, stream>>>(iters, 1e-3, 1e-3); break;
        default: probe_dmma_kernel<4><<<blocks, PROBE_THREADS, 0, stream>>>(iters, 1e-3, 1e-3); break;
        }
        cudaEventRecord(t1, stream);
        e = cudaEventSynchronize(t1);
        if (e != cudaSuccess) break;
        cudaEventElapsedTime(&ms, t0, t1);
    }
    cudaEventDestroy(t0);
    cudaEventDestroy(t1);
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // flops per thread per iteration: 2 per fma chain; per warp-wide mma 2*m*n*k spread over 32 lanes
    static const double per_thread[5] = {2.0, 2.0 * 8 * 8 * 4 / 32, 2.0 * 16 * 8 * 4 / 32, 2.0 * 16 * 8 * 8 / 32,
                                         2.0 * 16 * 8 * 16 / 32};
    const double flops = double(blocks) * PROBE_THREADS * double(iters) * CHAINS * per_thread[kind];
    *tflops_out = flops / (double(ms) * 1e-3) / 1e12;
    return cudaSuccess;
}

}  // namespace strassen
