// Internal declarations shared by the translation units of libsr (not part of the public ABI).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sr.h"

namespace sr {

constexpr int kMaxScale = 8;
constexpr int kMaxK = 9;

// Per-phase taps of one axis of the up-sampling (Keys cubic convolution, a = -0.75, half-pixel centres; or the
// bilinear pair in the two middle taps).
// HR index X = q*scale + phase reads LR indices q + base[phase] + {0,1,2,3}, each clamped to the image.
struct BicubicPhases {
    float w[kMaxScale][4];
    int base[kMaxScale];
};

// Everything a regression kernel needs to know about the problem (passed by value).
struct Problem {
    int n, c, h, w, r, k, D;
    int H, W;
    int s;          // atoms per pixel on the selective paths (== D on the dense path)
    uint32_t flags; // SR_* flags
    BicubicPhases ph;
};

enum RegressMode {
    kModeDense = 0,       // every atom, coefficients [n][D][H][W]
    kModeIdx = 1,         // per-pixel idx given, coefficients gathered from [n][D][H][W]
    kModeCompact = 2,     // per-pixel idx given, coefficients [n][s][H][W]
    kModeGlobal = 3,      // one subset idx[s] (+gamma), coefficients [n][D][H][W] or compact [n][s][H][W]
    kModeFusedSelect = 4  // top-s chosen inside the kernel from [n][D][H][W]
};

BicubicPhases make_phases(int scale, bool bilinear);

// Address of the per-device status word (device memory; 0 = ok). Returns nullptr on a CUDA error.
int* device_status_word();

// Cycle budget of one device-side wait for the launches that follow (set by sr_set_wait_limit).
long long wait_cycle_limit();

// Test hook (sr_test_lose_arrival): true once per armed launch; the launch then leaves out one barrier arrival.
bool take_injected_lost_arrival();

// Multiprocessors of the current device (queried once per device; at least 1).
int sm_count();

// Adds to the process-wide count of kernels launched (read back by sr_launch_count).
void count_launches(int n);

// Issue-rate probe (sr_probe.cu): kind 0 integer max/min, 1 fp32 multiply-add; lane operations per second.
cudaError_t probe_rate(int kind, int* scratch2, double* lane_ops_per_s, cudaStream_t st);

// Launchers. Each returns a cudaError_t from the launch.
cudaError_t launch_bicubic(const float* lr, float* hr, const Problem& pb, cudaStream_t st);
cudaError_t launch_regress_fma(int mode, const float* lr, const void* coef, int coef_dtype, const uint8_t* idx,
                               const float* gamma, const float* dict, float* out, const Problem& pb, cudaStream_t st);
cudaError_t launch_select(const void* coef, int coef_dtype, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st);
// Steps 1 and 3 of the composed luma-only regression (sr_luma.cu), one frame at a time.
cudaError_t launch_luma_lr(const float* lr_frame, float* ylr, const Problem& pb, cudaStream_t st);
cudaError_t launch_luma_combine(const float* lr_frame, float* out_frame, const Problem& pb, cudaStream_t st);

// ---- device helpers ------------------------------------------------------------------------------------------------

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return min(max(v, lo), hi); }

// The fp32 result as it is stored: unchanged, or rounded to nearest binary16 (SR_OUT_F16).
template <typename OutT> __device__ __forceinline__ OutT to_out(float v);
template <> __device__ __forceinline__ float to_out<float>(float v) { return v; }
template <> __device__ __forceinline__ __half to_out<__half>(float v) { return __float2half_rn(v); }
// SR_OUT_U8: the value clamped to [0, 1], times 255, rounded to nearest (ties to even)
template <> __device__ __forceinline__ uint8_t to_out<uint8_t>(float v) { return (uint8_t)__float2int_rn(fminf(fmaxf(v, 0.f), 1.f) * 255.f); }

// Output element i of a frame buffer that holds fp32 or (f16) binary16 values; for kernels that are not tight on
// registers and take the output type at run time.
__device__ __forceinline__ void store_out(float* out, int64_t i, float v, uint32_t flags)
{
    if (flags & SR_OUT_U8) reinterpret_cast<uint8_t*>(out)[i] = to_out<uint8_t>(v);
    else if (flags & SR_OUT_F16) reinterpret_cast<__half*>(out)[i] = __float2half_rn(v);
    else out[i] = v;
}

__device__ __forceinline__ float load_coef(const float* p, int64_t i) { return __ldg(p + i); }
__device__ __forceinline__ float load_coef(const __half* p, int64_t i) { return __half2float(__ldg(p + i)); }

// Bit pattern with the sign cleared: the selection key's magnitude part.
__device__ __forceinline__ uint32_t mag_bits(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }
__device__ __forceinline__ uint32_t mag_bits(__half v) { return (uint32_t)(__half_as_ushort(v) & 0x7FFFu); }

// One up-sampled value of an LR plane, direct 4x4 form, fp32.
__device__ __forceinline__ float bicubic_point(const float* __restrict__ plane, int h, int w, int r,
                                               const BicubicPhases& ph, int Y, int X)
{
    const int qy = Y / r, py = Y - qy * r;
    const int qx = X / r, px = X - qx * r;
    const int y0 = qy + ph.base[py], x0 = qx + ph.base[px];
    float acc = 0.f;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const float* row = plane + (int64_t)clampi(y0 + a, 0, h - 1) * w;
        float t = 0.f;
#pragma unroll
        for (int b = 0; b < 4; ++b) t = fmaf(ph.w[px][b], __ldg(row + clampi(x0 + b, 0, w - 1)), t);
        acc = fmaf(ph.w[py][a], t, acc);
    }
    return acc;
}

} // namespace sr
