// Stage 1 alone: bicubic up-sampling of every LR plane (Keys a = -0.75, half-pixel centres, edge clamp).
// HBM-bound: one thread produces four consecutive HR pixels of a row and stores them as one 16-byte word
// when the row pitch allows it; the LR taps come through the read-only cache.
#include "sr_common.cuh"

namespace sr {

__global__ void __launch_bounds__(256) bicubic_kernel(const float* __restrict__ lr, float* __restrict__ hr,
                                                      const __grid_constant__ Problem pb)
{
    const int W = pb.W, H = pb.H;
    const int groups = (W + 3) >> 2;
    const int64_t total = (int64_t)pb.n * pb.c * H * groups;
    const bool vec = (W & 3) == 0 && ((reinterpret_cast<uintptr_t>(hr) & 15) == 0);
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(t % groups);
        const int64_t row = t / groups;          // plane * H + Y
        const int Y = (int)(row % H);
        const int64_t plane = row / H;
        const float* src = lr + plane * (int64_t)pb.h * pb.w;
        const int X0 = g * 4;
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = (X0 + i < W) ? bicubic_point(src, pb.h, pb.w, pb.r, pb.ph, Y, X0 + i) : 0.f;
        float* dst = hr + row * (int64_t)W + X0;
        if (vec) {
            *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (X0 + i < W) dst[i] = v[i];
        }
    }
}

cudaError_t launch_bicubic(const float* lr, float* hr, const Problem& pb, cudaStream_t st)
{
    const int64_t total = (int64_t)pb.n * pb.c * pb.H * ((pb.W + 3) >> 2);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = 148 * 8 * 4;
    if (blocks > cap) blocks = cap;
    bicubic_kernel<<<(unsigned)blocks, 256, 0, st>>>(lr, hr, pb);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace sr
