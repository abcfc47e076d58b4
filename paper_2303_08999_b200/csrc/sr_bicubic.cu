// Stage 1 alone: bicubic up-sampling of every LR plane (Keys a = -0.75, half-pixel centres, edge clamp).
// A thread produces a BS x BS block of HR pixels from one LR window, separably (bicubic_block_kernel): BS = 4 at scales
// 1, 2 and 4, BS = 6 at scale 3, BS = r above. The direct 4 x 4 form (bicubic_kernel: one thread, four consecutive
// pixels of a row) remains for scales the block kernel is not instantiated for.
// Vector stores when the row pitch allows it; the LR taps come through the read-only cache.
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

// First LR tap of phase p at scale r, relative to X / r (the same integer arithmetic as the host's phase table).
__host__ __device__ constexpr int phase_base(int p, int r)
{
    const int num = 2 * p + 1 - r;
    return (num >= 0 ? num / (2 * r) : -((-num + 2 * r - 1) / (2 * r))) - 1;
}

// One thread produces a BS x BS block of HR pixels, BS a multiple of the scale. The block starts on a multiple of the
// scale, so every pixel's phase and the offset of its taps inside the block's LR window are compile-time constants:
// the window (NWIN^2 values, indices clamped to the plane) is loaded once, a horizontal pass gives BS values per
// window row and a vertical pass the BS^2 outputs. About 6 instructions per HR pixel against ~80 for the direct
// 4 x 4 form, which made the stand-alone call issue-bound (scale 3, 1080p: 54 us in the direct form).
template <int R, int BS>
__global__ void __launch_bounds__(256) bicubic_block_kernel(const float* __restrict__ lr, float* __restrict__ hr,
                                                            const __grid_constant__ Problem pb)
{
    static_assert(BS % R == 0, "a block starts on a multiple of the scale");
    constexpr int B0 = phase_base(0, R);
    constexpr int NWIN = (BS - 1) / R + phase_base((BS - 1) % R, R) - B0 + 4;    // window side: last pixel's first tap + 4
    constexpr int VEC = BS % 4 == 0 ? 4 : (BS % 2 == 0 ? 2 : 1);                 // floats per store
    const int W = pb.W, H = pb.H, w = pb.w, h = pb.h;
    const int bw = (W + BS - 1) / BS, bh = (H + BS - 1) / BS;
    const int64_t total = (int64_t)pb.n * pb.c * bh * bw;
    const bool vec = VEC > 1 && (W % VEC) == 0 && ((reinterpret_cast<uintptr_t>(hr) & (4 * VEC - 1)) == 0);
    float wt[R][4];
#pragma unroll
    for (int p = 0; p < R; ++p)
#pragma unroll
        for (int b = 0; b < 4; ++b) wt[p][b] = pb.ph.w[p][b];
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int bx = (int)(t % bw);
        const int64_t rest = t / bw;
        const int by = (int)(rest % bh);
        const int64_t plane = rest / bh;
        const float* src = lr + plane * (int64_t)h * w;
        const int col0 = (BS * bx) / R + B0, row0 = (BS * by) / R + B0;
        int cx[NWIN];
#pragma unroll
        for (int c = 0; c < NWIN; ++c) cx[c] = clampi(col0 + c, 0, w - 1);
        float T[NWIN][BS];                                   // horizontal pass of every window row
#pragma unroll
        for (int j = 0; j < NWIN; ++j) {
            const float* row = src + (int64_t)clampi(row0 + j, 0, h - 1) * w;
            float L[NWIN];
#pragma unroll
            for (int c = 0; c < NWIN; ++c) L[c] = __ldg(row + cx[c]);
#pragma unroll
            for (int i = 0; i < BS; ++i) {
                const int off = i / R + phase_base(i % R, R) - B0;   // compile-time after unrolling
                float a = wt[i % R][0] * L[off];
                a = fmaf(wt[i % R][1], L[off + 1], a);
                a = fmaf(wt[i % R][2], L[off + 2], a);
                a = fmaf(wt[i % R][3], L[off + 3], a);
                T[j][i] = a;
            }
        }
        float* dst = hr + (plane * H + BS * by) * (int64_t)W + BS * bx;
#pragma unroll
        for (int k = 0; k < BS; ++k) {
            if (BS * by + k >= H) break;
            const int off = k / R + phase_base(k % R, R) - B0;
            float v[BS];
#pragma unroll
            for (int i = 0; i < BS; ++i) {
                float a = wt[k % R][0] * T[off][i];
                a = fmaf(wt[k % R][1], T[off + 1][i], a);
                a = fmaf(wt[k % R][2], T[off + 2][i], a);
                a = fmaf(wt[k % R][3], T[off + 3][i], a);
                v[i] = a;
            }
            float* o = dst + (int64_t)k * W;
            if (vec && BS * bx + BS <= W) {
#pragma unroll
                for (int i = 0; i < BS; i += VEC) {
                    if constexpr (VEC == 4) *reinterpret_cast<float4*>(o + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    else *reinterpret_cast<float2*>(o + i) = make_float2(v[i], v[i + 1]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < BS; ++i)
                    if (BS * bx + i < W) o[i] = v[i];
            }
        }
    }
}

template <int R, int BS>
static cudaError_t launch_block(const float* lr, float* hr, const Problem& pb, cudaStream_t st)
{
    const int64_t total = (int64_t)pb.n * pb.c * ((pb.H + BS - 1) / BS) * ((pb.W + BS - 1) / BS);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    bicubic_block_kernel<R, BS><<<(unsigned)blocks, 256, 0, st>>>(lr, hr, pb);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_bicubic(const float* lr, float* hr, const Problem& pb, cudaStream_t st)
{
    switch (pb.r) {
    case 1: return launch_block<1, 4>(lr, hr, pb, st);
    case 2: return launch_block<2, 4>(lr, hr, pb, st);
    case 3: return launch_block<3, 6>(lr, hr, pb, st);
    case 4: return launch_block<4, 4>(lr, hr, pb, st);
    case 5: return launch_block<5, 5>(lr, hr, pb, st);
    case 6: return launch_block<6, 6>(lr, hr, pb, st);
    default: break;
    }
    const int64_t total = (int64_t)pb.n * pb.c * pb.H * ((pb.W + 3) >> 2);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    bicubic_kernel<<<(unsigned)blocks, 256, 0, st>>>(lr, hr, pb);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace sr
