// Luma-only regression (SR_LUMA_ONLY) with fp32 output, composed from the ordinary kernels, frame by frame:
//   1. the luma of the LR frame, Y = 0.299 R + 0.587 G + 0.114 B, into plane 1 of the frame's output (scratch: it is
//      overwritten in step 3 and an LR plane is never larger than an HR plane);
//   2. the ordinary ONE-channel regression of that plane (whatever kernel the shape gets) into plane 0 of the output;
//   3. in place, per pixel: every channel = its up-sampled value + (plane 0 - luma of the up-sampled pixel), clamp.
// Stage 1 is linear, so the luma of the up-sampled frame is the up-sampled luma: step 2 filters exactly the image the
// definition names. The two small kernels of steps 1 and 3 are here; step 2 is the caller's.
#include "sr_common.cuh"

namespace sr {

namespace {

__global__ void __launch_bounds__(256) luma_lr_kernel(const float* __restrict__ lr, float* __restrict__ ylr, int hw)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < hw) ylr[i] = fmaf(0.299f, lr[i], fmaf(0.587f, lr[hw + i], 0.114f * lr[2 * hw + i]));
}

__global__ void __launch_bounds__(256) luma_combine_kernel(const float* __restrict__ lr, float* __restrict__ out,
                                                           const __grid_constant__ Problem pb)
{
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int64_t pix = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pix >= HW) return;
    const int Y = (int)(pix / pb.W), X = (int)(pix - (int64_t)Y * pb.W);
    const int hw = pb.h * pb.w;
    const float u0 = bicubic_point(lr, pb.h, pb.w, pb.r, pb.ph, Y, X);
    const float u1 = bicubic_point(lr + hw, pb.h, pb.w, pb.r, pb.ph, Y, X);
    const float u2 = bicubic_point(lr + 2 * hw, pb.h, pb.w, pb.r, pb.ph, Y, X);
    const float shift = out[pix] - fmaf(0.299f, u0, fmaf(0.587f, u1, 0.114f * u2));
    float v0 = u0 + shift, v1 = u1 + shift, v2 = u2 + shift;
    if (pb.flags & SR_CLAMP01) {
        v0 = fminf(fmaxf(v0, 0.f), 1.f);
        v1 = fminf(fmaxf(v1, 0.f), 1.f);
        v2 = fminf(fmaxf(v2, 0.f), 1.f);
    }
    out[pix] = v0;
    out[HW + pix] = v1;
    out[2 * HW + pix] = v2;
}

} // namespace

cudaError_t launch_luma_lr(const float* lr_frame, float* ylr, const Problem& pb, cudaStream_t st)
{
    const int hw = pb.h * pb.w;
    luma_lr_kernel<<<(hw + 255) / 256, 256, 0, st>>>(lr_frame, ylr, hw);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_luma_combine(const float* lr_frame, float* out_frame, const Problem& pb, cudaStream_t st)
{
    const int64_t HW = (int64_t)pb.H * pb.W;
    luma_combine_kernel<<<(unsigned)((HW + 255) / 256), 256, 0, st>>>(lr_frame, out_frame, pb);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace sr
