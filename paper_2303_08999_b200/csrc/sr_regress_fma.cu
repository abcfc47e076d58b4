// General regression kernel on the fp32 FMA pipe: every shape, fp32 or binary16 coefficients, all modes.
// It is the path for fp32 coefficients (where HBM traffic doubles and the FMA pipe keeps pace with it)
// and the fallback for shapes the tensor-core path does not take.
//
// One thread per HR pixel, 32 x 8 pixel tiles. Per pixel: assemble the filter F = Phi_i D in registers
// (dictionary rows broadcast from shared memory), then y_c = F . B_c against an up-sampled tile with a
// halo of p = (k-1)/2 that lives only in shared memory. Neither F nor the patch matrix B reaches HBM.
#include "sr_common.cuh"

namespace sr {

namespace {

constexpr int TX = 32, TY = 8, CCHUNK = 4;

template <int K> struct KK { static constexpr int value = K * K, padded = (K * K + 3) & ~3; };

// (magnitude, lower index first) as one ordered integer; unique per atom.
__device__ __forceinline__ long long select_key(uint32_t mag, int l) { return ((long long)mag << 8) | (long long)(255 - l); }

template <int K, typename CoefT, int MODE>
__global__ void __launch_bounds__(TX * TY)
regress_fma_kernel(const float* __restrict__ lr, const CoefT* __restrict__ coef, const uint8_t* __restrict__ idx,
                   const float* __restrict__ gamma, const float* __restrict__ dict, float* __restrict__ out,
                   const __grid_constant__ Problem pb)
{
    constexpr int kk = KK<K>::value, kkp = KK<K>::padded, P = (K - 1) / 2;
    constexpr int UW = TX + 2 * P, UH = TY + 2 * P;
    extern __shared__ __align__(16) float smem[];
    float* sdict = smem;                         // [D][kkp]
    float* sU = smem + (size_t)pb.D * kkp;       // [CCHUNK][UH][UW]

    const int tid = threadIdx.y * TX + threadIdx.x;
    const int X = blockIdx.x * TX + threadIdx.x, Y = blockIdx.y * TY + threadIdx.y;
    const int f = blockIdx.z;
    const int H = pb.H, W = pb.W, D = pb.D, s = pb.s;
    const int64_t HW = (int64_t)H * W;
    const bool valid = X < W && Y < H;
    const int64_t pix = (int64_t)min(Y, H - 1) * W + min(X, W - 1);

    for (int i = tid; i < D * kkp; i += TX * TY) {
        const int l = i / kkp, j = i - l * kkp;
        sdict[i] = j < kk ? __ldg(dict + (int64_t)l * kk + j) : 0.f;
    }
    __syncthreads();

    // ---- stage 3: F = sum_q weight_q * dict[atom_q]
    float F[kkp];
#pragma unroll
    for (int j = 0; j < kkp; ++j) F[j] = 0.f;
    auto accumulate = [&](int atom, float wgt) {
        const float4* row = reinterpret_cast<const float4*>(sdict + atom * kkp);
#pragma unroll
        for (int j4 = 0; j4 < kkp / 4; ++j4) {
            const float4 dv = row[j4];
            F[4 * j4 + 0] = fmaf(wgt, dv.x, F[4 * j4 + 0]);
            F[4 * j4 + 1] = fmaf(wgt, dv.y, F[4 * j4 + 1]);
            F[4 * j4 + 2] = fmaf(wgt, dv.z, F[4 * j4 + 2]);
            F[4 * j4 + 3] = fmaf(wgt, dv.w, F[4 * j4 + 3]);
        }
    };
    if (MODE == kModeDense) {
        const CoefT* cp = coef + (int64_t)f * D * HW + pix;
#pragma unroll 4
        for (int l = 0; l < D; ++l) accumulate(l, load_coef(cp, (int64_t)l * HW));
    } else if (MODE == kModeIdx) {
        for (int q = 0; q < s; ++q) {
            const int a = min((int)__ldg(idx + ((int64_t)f * s + q) * HW + pix), D - 1);
            accumulate(a, load_coef(coef, ((int64_t)f * D + a) * HW + pix));
        }
    } else if (MODE == kModeCompact) {
        for (int q = 0; q < s; ++q) {
            const int a = min((int)__ldg(idx + ((int64_t)f * s + q) * HW + pix), D - 1);
            accumulate(a, load_coef(coef, ((int64_t)f * s + q) * HW + pix));
        }
    } else if (MODE == kModeGlobal) {
        const bool compact = (pb.flags & SR_COEF_COMPACT) != 0;
        for (int q = 0; q < s; ++q) {
            const int a = min((int)__ldg(idx + q), D - 1);
            const float g = gamma ? __ldg(gamma + q) : 1.f;
            const int64_t plane = compact ? ((int64_t)f * s + q) : ((int64_t)f * D + a);
            accumulate(a, g * load_coef(coef, plane * HW + pix));
        }
    } else { // kModeFusedSelect: repeated scan for the next-largest key; any s, any D
        const CoefT* cp = coef + (int64_t)f * D * HW + pix;
        long long prev = 0x7FFFFFFFFFFFFFFFll;
        for (int q = 0; q < s; ++q) {
            long long best = -1;
            for (int l = 0; l < D; ++l) {
                const long long key = select_key(mag_bits(__ldg(cp + (int64_t)l * HW)), l);
                if (key < prev && key > best) best = key;
            }
            prev = best;
            const int a = 255 - (int)(best & 255);
            accumulate(a, load_coef(cp, (int64_t)a * HW));
        }
    }

    // ---- stages 1 + 4, CCHUNK channels at a time
    const int Y0 = blockIdx.y * TY - P, X0 = blockIdx.x * TX - P;
    for (int c0 = 0; c0 < pb.c; c0 += CCHUNK) {
        const int nc = min(CCHUNK, pb.c - c0);
        __syncthreads();
        for (int i = tid; i < nc * UH * UW; i += TX * TY) {
            const int ch = i / (UH * UW), rem = i - ch * (UH * UW);
            const int uy = rem / UW, ux = rem - uy * UW;
            const float* plane = lr + ((int64_t)f * pb.c + c0 + ch) * pb.h * pb.w;
            sU[i] = bicubic_point(plane, pb.h, pb.w, pb.r, pb.ph, clampi(Y0 + uy, 0, H - 1), clampi(X0 + ux, 0, W - 1));
        }
        __syncthreads();
        if (pb.flags & SR_LUMA_ONLY) {
            // c = 3 (checked by the caller): the fourth slot takes the luma of the tile, the filter runs on it once,
            // and every channel moves by the same amount, so the chroma differences stay those of stage 1.
            float* sY = sU + 3 * UH * UW;
            for (int i = tid; i < UH * UW; i += TX * TY)
                sY[i] = fmaf(0.299f, sU[i], fmaf(0.587f, sU[UH * UW + i], 0.114f * sU[2 * UH * UW + i]));
            __syncthreads();
            const float* u = sY + threadIdx.y * UW + threadIdx.x;
            float acc = 0.f;
#pragma unroll
            for (int a = 0; a < K; ++a)
#pragma unroll
                for (int b = 0; b < K; ++b) acc = fmaf(F[a * K + b], u[a * UW + b], acc);
            const float shift = acc - u[P * UW + P];
            for (int ch = 0; ch < 3; ++ch) {
                float v = sU[ch * UH * UW + (threadIdx.y + P) * UW + threadIdx.x + P] + shift;
                if (pb.flags & SR_CLAMP01) v = fminf(fmaxf(v, 0.f), 1.f);
                if (valid) store_out(out, ((int64_t)f * 3 + ch) * HW + pix, v, pb.flags);
            }
            break;
        }
        for (int ch = 0; ch < nc; ++ch) {
            const float* u = sU + ch * UH * UW + threadIdx.y * UW + threadIdx.x;
            float acc = 0.f;
#pragma unroll
            for (int a = 0; a < K; ++a)
#pragma unroll
                for (int b = 0; b < K; ++b) acc = fmaf(F[a * K + b], u[a * UW + b], acc);
            if (pb.flags & SR_CLAMP01) acc = fminf(fmaxf(acc, 0.f), 1.f);
            if (valid) store_out(out, ((int64_t)f * pb.c + c0 + ch) * HW + pix, acc, pb.flags);
        }
    }
}

template <int K, typename CoefT, int MODE>
cudaError_t launch_t(const float* lr, const void* coef, const uint8_t* idx, const float* gamma, const float* dict,
                     float* out, const Problem& pb, cudaStream_t st)
{
    constexpr int P = (K - 1) / 2;
    const size_t smem = ((size_t)pb.D * KK<K>::padded + (size_t)CCHUNK * (TY + 2 * P) * (TX + 2 * P)) * sizeof(float);
    auto kern = regress_fma_kernel<K, CoefT, MODE>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((pb.W + TX - 1) / TX, (pb.H + TY - 1) / TY, pb.n), block(TX, TY);
    if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidConfiguration;
    kern<<<grid, block, smem, st>>>(lr, (const CoefT*)coef, idx, gamma, dict, out, pb);
    count_launches(1);
    return cudaGetLastError();
}

template <int K, typename CoefT>
cudaError_t launch_m(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                     const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    switch (mode) {
    case kModeDense: return launch_t<K, CoefT, kModeDense>(lr, coef, idx, gamma, dict, out, pb, st);
    case kModeIdx: return launch_t<K, CoefT, kModeIdx>(lr, coef, idx, gamma, dict, out, pb, st);
    case kModeCompact: return launch_t<K, CoefT, kModeCompact>(lr, coef, idx, gamma, dict, out, pb, st);
    case kModeGlobal: return launch_t<K, CoefT, kModeGlobal>(lr, coef, idx, gamma, dict, out, pb, st);
    default: return launch_t<K, CoefT, kModeFusedSelect>(lr, coef, idx, gamma, dict, out, pb, st);
    }
}

template <typename CoefT>
cudaError_t launch_k(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                     const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    switch (pb.k) {
    case 1: return launch_m<1, CoefT>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    case 3: return launch_m<3, CoefT>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    case 5: return launch_m<5, CoefT>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    case 7: return launch_m<7, CoefT>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    default: return launch_m<9, CoefT>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    }
}

} // namespace

cudaError_t launch_regress_fma(int mode, const float* lr, const void* coef, int coef_dtype, const uint8_t* idx,
                               const float* gamma, const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    if (coef_dtype == SR_F16) return launch_k<__half>(mode, lr, coef, idx, gamma, dict, out, pb, st);
    return launch_k<float>(mode, lr, coef, idx, gamma, dict, out, pb, st);
}

} // namespace sr
