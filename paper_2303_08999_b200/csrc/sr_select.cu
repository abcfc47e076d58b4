// Per-pixel top-s selection by coefficient magnitude, ties to the lower atom index, rank order out.
// Key of atom l = (bit pattern with the sign cleared) * 256 + (255 - l): one integer whose order is
// exactly "larger magnitude first, then lower index"; keys of one pixel are distinct.
#include "sr_common.cuh"

namespace sr {

namespace {

template <typename CoefT> struct KeyOf;
template <> struct KeyOf<__half> { using type = int; };          // 15 + 8 bits
template <> struct KeyOf<float> { using type = long long; };     // 31 + 8 bits

template <typename CoefT>
__device__ __forceinline__ typename KeyOf<CoefT>::type make_key(CoefT v, int l)
{
    using KeyT = typename KeyOf<CoefT>::type;
    return (KeyT)(((KeyT)mag_bits(v) << 8) | (KeyT)(255 - l));
}

// s <= SMAX: sorted list in registers, one branch-free insertion per atom.
template <typename CoefT, int SMAX>
__global__ void __launch_bounds__(256)
select_insert_kernel(const CoefT* __restrict__ coef, uint8_t* __restrict__ idx, CoefT* __restrict__ sel,
                     const __grid_constant__ Problem pb)
{
    using KeyT = typename KeyOf<CoefT>::type;
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int64_t total = (int64_t)pb.n * HW;
    const int D = pb.D, s = pb.s;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t f = t / HW, pix = t - f * HW;
        const CoefT* cp = coef + f * D * HW + pix;
        KeyT top[SMAX];
#pragma unroll
        for (int i = 0; i < SMAX; ++i) top[i] = (KeyT)-1;
#pragma unroll 4
        for (int l = 0; l < D; ++l) {
            KeyT x = make_key<CoefT>(__ldg(cp + (int64_t)l * HW), l);
#pragma unroll
            for (int i = 0; i < SMAX; ++i) {
                const KeyT hi = max(top[i], x);
                x = min(top[i], x);
                top[i] = hi;
            }
        }
#pragma unroll
        for (int q = 0; q < SMAX; ++q) {
            if (q < s) {
                const int a = 255 - (int)(top[q] & 255);
                idx[(f * s + q) * HW + pix] = (uint8_t)a;
                if (sel) sel[(f * s + q) * HW + pix] = __ldg(cp + (int64_t)a * HW);
            }
        }
    }
}

// Any s: rank q is the largest key below rank q-1's key.
template <typename CoefT>
__global__ void __launch_bounds__(256)
select_scan_kernel(const CoefT* __restrict__ coef, uint8_t* __restrict__ idx, CoefT* __restrict__ sel,
                   const __grid_constant__ Problem pb)
{
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int64_t total = (int64_t)pb.n * HW;
    const int D = pb.D, s = pb.s;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t f = t / HW, pix = t - f * HW;
        const CoefT* cp = coef + f * D * HW + pix;
        long long prev = 0x7FFFFFFFFFFFFFFFll;
        for (int q = 0; q < s; ++q) {
            long long best = -1;
            for (int l = 0; l < D; ++l) {
                const long long key = (long long)make_key<CoefT>(__ldg(cp + (int64_t)l * HW), l);
                if (key < prev && key > best) best = key;
            }
            prev = best;
            const int a = 255 - (int)(best & 255);
            idx[(f * s + q) * HW + pix] = (uint8_t)a;
            if (sel) sel[(f * s + q) * HW + pix] = __ldg(cp + (int64_t)a * HW);
        }
    }
}

template <typename CoefT>
cudaError_t launch_sel(const void* coef, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st)
{
    const int64_t total = (int64_t)pb.n * pb.H * pb.W;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    const CoefT* c = (const CoefT*)coef;
    CoefT* sl = (CoefT*)sel;
    if (pb.s <= 4) select_insert_kernel<CoefT, 4><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else if (pb.s <= 8) select_insert_kernel<CoefT, 8><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else if (pb.s <= 16) select_insert_kernel<CoefT, 16><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else select_scan_kernel<CoefT><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace

cudaError_t launch_select(const void* coef, int coef_dtype, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st)
{
    if (coef_dtype == SR_F16) return launch_sel<__half>(coef, idx, sel, pb, st);
    return launch_sel<float>(coef, idx, sel, pb, st);
}

} // namespace sr
