// Issue-rate probes for the roofline of the kernels that are bound by an arithmetic pipe rather than by HBM:
// sustained lane operations per second of integer max/min (the selection networks' instruction) and of fp32
// multiply-add, measured on the device the library runs on, with independent register chains and no memory traffic.
#include "sr_common.cuh"

namespace sr {

namespace {

constexpr int kChains = 8, kIters = 4096, kThreads = 256;

__device__ __forceinline__ void cx(int& a, int& b)
{
    const int hi = max(a, b), lo = min(a, b);
    a = hi;
    b = lo;
}

// The instruction mix of the selection networks themselves: the 19-exchange sorting network on eight registers, over
// and over (the data is sorted after the first pass, which the hardware does not care about and the compiler cannot
// know), two independent sets per thread. 38 max/min lane operations per set and pass, nothing else in the loop body.
__global__ void __launch_bounds__(kThreads) probe_minmax_kernel(const int* seed, int* sink)
{
    int k[2][8];
    const int s = __ldg(seed) + threadIdx.x;
#pragma unroll
    for (int q = 0; q < 2; ++q)
#pragma unroll
        for (int i = 0; i < 8; ++i) k[q][i] = (s + q) * (2 * i + 3) ^ (0x5bd1e995 * (i + 1));
#pragma unroll 1
    for (int it = 0; it < kIters / 8; ++it) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                int* v = k[q];
                cx(v[0], v[1]); cx(v[2], v[3]); cx(v[4], v[5]); cx(v[6], v[7]);
                cx(v[0], v[2]); cx(v[1], v[3]); cx(v[4], v[6]); cx(v[5], v[7]);
                cx(v[1], v[2]); cx(v[5], v[6]);
                cx(v[0], v[4]); cx(v[1], v[5]); cx(v[2], v[6]); cx(v[3], v[7]);
                cx(v[2], v[4]); cx(v[3], v[5]);
                cx(v[1], v[2]); cx(v[3], v[4]); cx(v[5], v[6]);
            }
        }
    }
    int acc = 0;
#pragma unroll
    for (int q = 0; q < 2; ++q)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc += k[q][i];
    if (acc == 0x7fffffff) sink[0] = acc;            // practically never: the result only has to look used
}

__global__ void __launch_bounds__(kThreads) probe_fma_kernel(const int* seed, float* sink)
{
    float a[kChains];
    const float x = 1.0f + 1e-7f * (float)(__ldg(seed) + threadIdx.x), y = 1e-9f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) a[i] = (float)i;
#pragma unroll 1
    for (int it = 0; it < kIters / 8; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < kChains; ++i) a[i] = fmaf(a[i], x, y);
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) acc += a[i];
    if (acc == -1.f) sink[0] = acc;
}

// The packed form (fma.rn.f32x2: two multiply-adds per lane and instruction), same chains.
__global__ void __launch_bounds__(kThreads) probe_fma2_kernel(const int* seed, float* sink)
{
    float2 a[kChains];
    const float xs = 1.0f + 1e-7f * (float)(__ldg(seed) + threadIdx.x);
    const float2 x = make_float2(xs, xs + 1e-7f), y = make_float2(1e-9f, 2e-9f);
#pragma unroll
    for (int i = 0; i < kChains; ++i) a[i] = make_float2((float)i, (float)(i + 1));
#pragma unroll 1
    for (int it = 0; it < kIters / 8; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < kChains; ++i) a[i] = __ffma2_rn(a[i], x, y);
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) acc += a[i].x + a[i].y;
    if (acc == -1.f) sink[0] = acc;
}

} // namespace

// kind 0: integer max/min, kind 1: fp32 multiply-add, kind 2: packed fp32 multiply-add (two per lane and instruction). Lane operations per second; synchronises the stream.
cudaError_t probe_rate(int kind, int* scratch2 /* two ints of device memory */, double* lane_ops_per_s, cudaStream_t st)
{
    const int ctas = sm_count() * 8;
    cudaEvent_t e0, e1;
    cudaError_t err = cudaEventCreate(&e0);
    if (err != cudaSuccess) return err;
    err = cudaEventCreate(&e1);
    if (err != cudaSuccess) { cudaEventDestroy(e0); return err; }
    float best_ms = 0.f;
    for (int rep = 0; rep < 4 && err == cudaSuccess; ++rep) {
        cudaEventRecord(e0, st);
        if (kind == 0) probe_minmax_kernel<<<ctas, kThreads, 0, st>>>(scratch2, scratch2 + 1);
        else if (kind == 1) probe_fma_kernel<<<ctas, kThreads, 0, st>>>(scratch2, reinterpret_cast<float*>(scratch2 + 1));
        else probe_fma2_kernel<<<ctas, kThreads, 0, st>>>(scratch2, reinterpret_cast<float*>(scratch2 + 1));
        count_launches(1);
        cudaEventRecord(e1, st);
        err = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;      // the first launch warms up
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess) return err;
    // max/min: (kIters / 8) trips x 2 passes x 2 sets x 38 operations per thread; multiply-add: kIters x kChains
    const double per_thread = kind == 0 ? (double)(kIters / 8) * 2 * 2 * 38 : (double)kIters * kChains * (kind == 2 ? 2 : 1);
    const double ops = (double)ctas * kThreads * per_thread;
    *lane_ops_per_s = ops / ((double)best_ms * 1e-3);
    return cudaSuccess;
}

} // namespace sr
