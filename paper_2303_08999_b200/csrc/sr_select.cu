// Per-pixel top-s selection by coefficient magnitude, ties to the lower atom index, rank order out.
// Key of atom l = (bit pattern with the sign cleared) * 256 + (255 - l): one integer whose order is
// exactly "larger magnitude first, then lower index"; keys of one pixel are distinct.
//
// Fast path (binary16 coefficients, s <= 16, even W): one thread owns two neighbouring pixels (one 4-byte load per
// plane, a full 128-byte line per warp), keeps their s best keys sorted in registers and merges every group of S
// planes with branch-free sorting networks of integer max / min:
//   sort the S new keys (19 compare-exchanges for S = 8), max against the reversed running list (S ops, gives a
//   bitonic sequence holding the S best of both), bitonic-merge it back to sorted order (S/2 * log2 S exchanges).
// Per pixel and plane that is about 8.75 min/max for S = 8 (630 per pixel at D = 72) against 16 for plain insertion.
// The kernel is bound by the integer ALU rate or by HBM, whichever is slower for the shape.
// With 16-byte aligned planes the block first stages its 256 pixels x D planes in shared memory (select_tilef_kernel)
// and the threads read their words, and at the end the selected values, from there.
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

// ---- sorting networks on int keys (descending) -----------------------------------------------------------------------

__device__ __forceinline__ void cx(int& a, int& b)    // afterwards a >= b
{
    const int hi = max(a, b), lo = min(a, b);
    a = hi;
    b = lo;
}

template <int S> __device__ __forceinline__ void sort_desc(int* k);

template <> __device__ __forceinline__ void sort_desc<4>(int* k)
{
    cx(k[0], k[1]); cx(k[2], k[3]);
    cx(k[0], k[2]); cx(k[1], k[3]);
    cx(k[1], k[2]);
}

template <> __device__ __forceinline__ void sort_desc<8>(int* k)   // 19 exchanges
{
    cx(k[0], k[1]); cx(k[2], k[3]); cx(k[4], k[5]); cx(k[6], k[7]);
    cx(k[0], k[2]); cx(k[1], k[3]); cx(k[4], k[6]); cx(k[5], k[7]);
    cx(k[1], k[2]); cx(k[5], k[6]);
    cx(k[0], k[4]); cx(k[1], k[5]); cx(k[2], k[6]); cx(k[3], k[7]);
    cx(k[2], k[4]); cx(k[3], k[5]);
    cx(k[1], k[2]); cx(k[3], k[4]); cx(k[5], k[6]);
}

// Sorts a bitonic sequence of S keys into descending order.
template <int S> __device__ __forceinline__ void bitonic_merge_desc(int* k)
{
#pragma unroll
    for (int d = S / 2; d >= 1; d >>= 1)
#pragma unroll
        for (int i = 0; i < S; ++i)
            if ((i & d) == 0) cx(k[i], k[i + d]);
}

template <> __device__ __forceinline__ void sort_desc<16>(int* k)   // two sorted halves, then a bitonic merge
{
    sort_desc<8>(k);
    sort_desc<8>(k + 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const int t = k[8 + i]; k[8 + i] = k[15 - i]; k[15 - i] = t; }   // second half ascending
    bitonic_merge_desc<16>(k);
}

// top[] (sorted) <- the S best of top[] and grp[] (grp sorted descending)
template <int S> __device__ __forceinline__ void merge_top(int* top, const int* grp)
{
#pragma unroll
    for (int i = 0; i < S; ++i) top[i] = max(top[i], grp[S - 1 - i]);
    bitonic_merge_desc<S>(top);
}

// Two pixels per thread, binary16, s <= S, W even.
template <int S>
__global__ void __launch_bounds__(256)
select_pair_kernel(const __half* __restrict__ coef, uint8_t* __restrict__ idx, __half* __restrict__ sel,
                   const __grid_constant__ Problem pb)
{
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int64_t pairs_per_frame = HW / 2;
    const int64_t total = (int64_t)pb.n * pairs_per_frame;
    const int D = pb.D, s = pb.s;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t f = t / pairs_per_frame, pix = (t - f * pairs_per_frame) * 2;
        const __half* cp = coef + f * D * HW + pix;
        int ta[S], tb[S];
#pragma unroll
        for (int i = 0; i < S; ++i) ta[i] = tb[i] = -1;
        const uint32_t* wp = reinterpret_cast<const uint32_t*>(cp);      // one word = the pair's coefficients of a plane
        const int64_t wstride = HW / 2;                                   // words between planes (W is even)
        int l0 = 0;
        for (; l0 + S <= D; l0 += S) {                                   // whole groups: no per-key guards
            uint32_t w[S];
#pragma unroll
            for (int i = 0; i < S; ++i) w[i] = __ldg(wp + (int64_t)(l0 + i) * wstride);
            int ga[S], gb[S];
#pragma unroll
            for (int i = 0; i < S; ++i) {
                // key = 0 | magnitude (2 bytes) | tag: one byte permute per pixel out of (signs cleared, tag)
                const uint32_t tag = (uint32_t)(255 - (l0 + i)), m2 = w[i] & 0x7FFF7FFFu;
                ga[i] = (int)__byte_perm(m2, tag, 0x5104);
                gb[i] = (int)__byte_perm(m2, tag, 0x5324);
            }
            sort_desc<S>(ga);
            sort_desc<S>(gb);
            merge_top<S>(ta, ga);
            merge_top<S>(tb, gb);
        }
        if (l0 < D) {                                                     // last, partial group
            int ga[S], gb[S];
#pragma unroll
            for (int i = 0; i < S; ++i) {
                ga[i] = gb[i] = -1;
                if (l0 + i < D) {
                    const uint32_t tag = (uint32_t)(255 - (l0 + i)), m2 = __ldg(wp + (int64_t)(l0 + i) * wstride) & 0x7FFF7FFFu;
                    ga[i] = (int)__byte_perm(m2, tag, 0x5104);
                    gb[i] = (int)__byte_perm(m2, tag, 0x5324);
                }
            }
            sort_desc<S>(ga);
            sort_desc<S>(gb);
            merge_top<S>(ta, ga);
            merge_top<S>(tb, gb);
        }
#pragma unroll
        for (int q = 0; q < S; ++q) {
            if (q < s) {
                const int a = 255 - (ta[q] & 255), b = 255 - (tb[q] & 255);
                const int64_t o = (f * s + q) * HW + pix;
                *reinterpret_cast<uchar2*>(idx + o) = make_uchar2((unsigned char)a, (unsigned char)b);
                if (sel) {
                    const __half va = __ldg(cp + (int64_t)a * HW), vb = __ldg(cp + (int64_t)b * HW + 1);
                    *reinterpret_cast<__half2*>(sel + o) = __halves2half2(va, vb);
                }
            }
        }
    }
}

// Same selection with the block's coefficients staged in shared memory first: a block owns TP = 256 consecutive pixels
// of a frame, copies their D planes with 16-byte asynchronous copies ([D][TP] binary16), and every thread then reads
// its pixel pair's words from there. The selected values are picked out of the same tile at the end, so no
// coefficient is fetched from global memory twice (on frames whose planes are many megabytes apart the re-read of
// the selected values used to miss the L2 and cost half as much again as the selection itself).
// Needs 16-byte aligned planes (H * W a multiple of 8) and D / 2 KiB of shared memory. Shared memory, not registers,
// limits the resident pixels (2 D bytes each: about 1500 per SM at D = 72 whatever the tile size); the smaller tile
// gives more, shorter load and compute phases to interleave (six blocks per SM instead of three: 3 % faster at s = 8,
// 8 % at s = 16 on the 1080p frame).
constexpr int kSelTilePixels = 256;

// Byte permute with the full selector: bit 3 of a selector nibble replicates the sign bit of the selected byte instead
// of copying it (the intrinsic only documents the low three bits).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__device__ __forceinline__ void sel_cp_async_16(uint32_t dst_smem, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}

// ---- the same networks on keys held as fp32 numbers -------------------------------------------------------------------
// A key (23 bits) is exactly representable in fp32, so a compare-exchange can run on either arithmetic pipe:
//   ALU pipe:  hi = max(a, b), lo = min(a, b)                                    (2 operations, 64 lanes/clk/SM)
//   FMA pipe:  d = a - b, s = a + b, hi = (s + |d|) / 2, lo = s - hi             (5 operations, 128 lanes/clk/SM)
// every step of the second form is exact (integers below 2^24). The integer networks saturate the ALU pipe while the FMA
// pipe idles. By pipe and issue-slot counts two exchanges in seven on the FMA pipe would be the balance; measured on the
// 1080p frame the longer dependency chain of the second form matters as much: every fifth exchange, spread evenly, was
// the fastest of eleven placements tried (118 us against 130 us with none; whole first layers on the FMA pipe: 131 us).
__device__ __forceinline__ void cxf_alu(float& a, float& b)
{
    const float hi = fmaxf(a, b), lo = fminf(a, b);
    a = hi;
    b = lo;
}
__device__ __forceinline__ void cxf_fma(float& a, float& b)
{
    const float d = a - b, s = a + b;
    const float hi = (s + fabsf(d)) * 0.5f;
    b = s - hi;
    a = hi;
}
// exchange number N of a network: which pipe takes it
template <int N> __device__ __forceinline__ void cxf(float& a, float& b)
{
    if constexpr (N % 5 == 1) cxf_fma(a, b);
    else cxf_alu(a, b);
}

__device__ __forceinline__ void sort8_desc_f(float* k)   // 19 exchanges
{
    cxf<0>(k[0], k[1]); cxf<1>(k[2], k[3]); cxf<2>(k[4], k[5]); cxf<3>(k[6], k[7]);
    cxf<4>(k[0], k[2]); cxf<5>(k[1], k[3]); cxf<6>(k[4], k[6]); cxf<7>(k[5], k[7]);
    cxf<8>(k[1], k[2]); cxf<9>(k[5], k[6]);
    cxf<10>(k[0], k[4]); cxf<11>(k[1], k[5]); cxf<12>(k[2], k[6]); cxf<13>(k[3], k[7]);
    cxf<14>(k[2], k[4]); cxf<15>(k[3], k[5]);
    cxf<16>(k[1], k[2]); cxf<17>(k[3], k[4]); cxf<18>(k[5], k[6]);
}

// top[] (sorted) <- the 8 best of top[] and grp[] (grp sorted descending): 8 max, then a 12-exchange bitonic merge
__device__ __forceinline__ void merge_top8_f(float* top, const float* grp)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = fmaxf(top[i], grp[7 - i]);
    cxf<19>(top[0], top[4]); cxf<20>(top[1], top[5]); cxf<21>(top[2], top[6]); cxf<22>(top[3], top[7]);
    cxf<23>(top[0], top[2]); cxf<24>(top[1], top[3]); cxf<25>(top[4], top[6]); cxf<26>(top[5], top[7]);
    cxf<27>(top[0], top[1]); cxf<28>(top[2], top[3]); cxf<29>(top[4], top[5]); cxf<30>(top[6], top[7]);
}

// Lists of 4 and 16: the same split, the exchange number taken from its place in the network.
__device__ __forceinline__ void sort4_desc_f(float* k)
{
    cxf<0>(k[0], k[1]); cxf<1>(k[2], k[3]);
    cxf<2>(k[0], k[2]); cxf<3>(k[1], k[3]);
    cxf<4>(k[1], k[2]);
}
__device__ __forceinline__ void merge_top4_f(float* top, const float* grp)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) top[i] = fmaxf(top[i], grp[3 - i]);
    cxf<5>(top[0], top[2]); cxf<6>(top[1], top[3]);
    cxf<7>(top[0], top[1]); cxf<8>(top[2], top[3]);
}
template <int BASE>
__device__ __forceinline__ void bitonic16_desc_f(float* k)   // 32 exchanges, numbered from BASE
{
    cxf<BASE + 0>(k[0], k[8]); cxf<BASE + 1>(k[1], k[9]); cxf<BASE + 2>(k[2], k[10]); cxf<BASE + 3>(k[3], k[11]);
    cxf<BASE + 4>(k[4], k[12]); cxf<BASE + 5>(k[5], k[13]); cxf<BASE + 6>(k[6], k[14]); cxf<BASE + 7>(k[7], k[15]);
    cxf<BASE + 8>(k[0], k[4]); cxf<BASE + 9>(k[1], k[5]); cxf<BASE + 10>(k[2], k[6]); cxf<BASE + 11>(k[3], k[7]);
    cxf<BASE + 12>(k[8], k[12]); cxf<BASE + 13>(k[9], k[13]); cxf<BASE + 14>(k[10], k[14]); cxf<BASE + 15>(k[11], k[15]);
    cxf<BASE + 16>(k[0], k[2]); cxf<BASE + 17>(k[1], k[3]); cxf<BASE + 18>(k[4], k[6]); cxf<BASE + 19>(k[5], k[7]);
    cxf<BASE + 20>(k[8], k[10]); cxf<BASE + 21>(k[9], k[11]); cxf<BASE + 22>(k[12], k[14]); cxf<BASE + 23>(k[13], k[15]);
    cxf<BASE + 24>(k[0], k[1]); cxf<BASE + 25>(k[2], k[3]); cxf<BASE + 26>(k[4], k[5]); cxf<BASE + 27>(k[6], k[7]);
    cxf<BASE + 28>(k[8], k[9]); cxf<BASE + 29>(k[10], k[11]); cxf<BASE + 30>(k[12], k[13]); cxf<BASE + 31>(k[14], k[15]);
}
__device__ __forceinline__ void sort16_desc_f(float* k)   // two sorted halves, then a bitonic merge
{
    sort8_desc_f(k);
    sort8_desc_f(k + 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float t = k[8 + i]; k[8 + i] = k[15 - i]; k[15 - i] = t; }   // second half ascending
    bitonic16_desc_f<19>(k);
}
__device__ __forceinline__ void merge_top16_f(float* top, const float* grp)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) top[i] = fmaxf(top[i], grp[15 - i]);
    bitonic16_desc_f<51>(top);
}
template <int S> __device__ __forceinline__ void sort_desc_f(float* k)
{
    if constexpr (S == 4) sort4_desc_f(k);
    else if constexpr (S == 8) sort8_desc_f(k);
    else sort16_desc_f(k);
}
template <int S> __device__ __forceinline__ void merge_top_f(float* top, const float* grp)
{
    if constexpr (S == 4) merge_top4_f(top, grp);
    else if constexpr (S == 8) merge_top8_f(top, grp);
    else merge_top16_f(top, grp);
}

constexpr float kKeyMagic = 8388608.f;   // 2^23: the bits 0x4B000000 | key are the fp32 number 2^23 + key

template <int S, int TP>   // TP: pixels per tile (512 or 256), two per thread
__global__ void __launch_bounds__(TP / 2)
select_tilef_kernel(const __half* __restrict__ coef, uint8_t* __restrict__ idx, __half* __restrict__ sel,
                    const __grid_constant__ Problem pb, int tiles_per_frame)
{
    constexpr int NT = (S + 2) / 3;                          // tag registers: three tags each
    extern __shared__ __align__(16) uint8_t tile[];          // [D][TP] binary16
    const int64_t HW = (int64_t)pb.H * pb.W;
    const int D = pb.D, s = pb.s, tid = threadIdx.x;
    const int64_t f = blockIdx.x / tiles_per_frame;
    const int64_t p0 = (int64_t)(blockIdx.x - f * tiles_per_frame) * TP;   // first pixel of the tile
    const __half* cp = coef + f * D * HW + p0;
    {
        const uint32_t tile_s = (uint32_t)__cvta_generic_to_shared(tile);
        const int chunk = tid & (TP / 8 - 1);                // 16-byte chunk (8 pixels) of a plane's row of TP pixels
        const uint32_t bytes = p0 + chunk * 8 < HW ? 16u : 0u;   // chunks beyond the frame are zero-filled
        const __half* src = cp + (bytes ? chunk * 8 : 0);
        for (int l = tid / (TP / 8); l < D; l += 4)
            sel_cp_async_16(tile_s + (uint32_t)l * (uint32_t)(2 * TP) + (uint32_t)chunk * 16u, src + (int64_t)l * HW, bytes);
        asm volatile("cp.async.wait_all;" ::: "memory");
    }
    __syncthreads();
    const int64_t pix = p0 + 2 * tid;
    if (pix >= HW) return;
    const uint32_t* wp = reinterpret_cast<const uint32_t*>(tile) + tid;   // + TP / 2 words per plane
    float ta[S], tb[S];
#pragma unroll
    for (int i = 0; i < S; ++i) ta[i] = tb[i] = -1.f;
    // byte j (j < 3) of tags[q] = 255 - (l0 + 3 q + j), byte 3 = 0x4B; a group moves the tags down by S with one
    // subtraction per register (no byte ever borrows: a tag is at least 255 - 199)
    uint32_t tags[NT];
#pragma unroll
    for (int q = 0; q < NT; ++q) tags[q] = 0x4B000000u | (255u - 3u * q) | ((254u - 3u * q) << 8) | ((253u - 3u * q) << 16);
    int l0 = 0;
    for (; l0 + S <= D; l0 += S) {                           // whole groups: no per-key guards
        uint32_t w[S];
#pragma unroll
        for (int i = 0; i < S; ++i) w[i] = wp[(l0 + i) * (TP / 2)];
        float ga[S], gb[S];
#pragma unroll
        for (int i = 0; i < S; ++i) {
            // bits (tag, magnitude low byte, magnitude high byte, 0x4B) = the fp32 number 2^23 + key
            const uint32_t m2 = w[i] & 0x7FFF7FFFu;
            ga[i] = __uint_as_float(prmt(m2, tags[i / 3], 0x7100u | (uint32_t)(4 + i % 3))) - kKeyMagic;
            gb[i] = __uint_as_float(prmt(m2, tags[i / 3], 0x7320u | (uint32_t)(4 + i % 3))) - kKeyMagic;
        }
        sort_desc_f<S>(ga);
        sort_desc_f<S>(gb);
        merge_top_f<S>(ta, ga);
        merge_top_f<S>(tb, gb);
#pragma unroll
        for (int q = 0; q < NT; ++q) tags[q] -= 0x00010101u * (uint32_t)S;
    }
    if (l0 < D) {                                            // last, partial group
        float ga[S], gb[S];
#pragma unroll
        for (int i = 0; i < S; ++i) {
            ga[i] = gb[i] = -1.f;
            if (l0 + i < D) {
                const uint32_t m2 = wp[(l0 + i) * (TP / 2)] & 0x7FFF7FFFu;
                ga[i] = __uint_as_float(prmt(m2, tags[i / 3], 0x7100u | (uint32_t)(4 + i % 3))) - kKeyMagic;
                gb[i] = __uint_as_float(prmt(m2, tags[i / 3], 0x7320u | (uint32_t)(4 + i % 3))) - kKeyMagic;
            }
        }
        sort_desc_f<S>(ga);
        sort_desc_f<S>(gb);
        merge_top_f<S>(ta, ga);
        merge_top_f<S>(tb, gb);
    }
    const __half* th = reinterpret_cast<const __half*>(tile) + 2 * tid;
#pragma unroll
    for (int q = 0; q < S; ++q) {
        if (q < s) {
            const int a = 255 - (int)(__float_as_uint(ta[q] + kKeyMagic) & 255u), b = 255 - (int)(__float_as_uint(tb[q] + kKeyMagic) & 255u);
            const int64_t o = (f * s + q) * HW + pix;
            *reinterpret_cast<uchar2*>(idx + o) = make_uchar2((unsigned char)a, (unsigned char)b);
            if (sel) *reinterpret_cast<__half2*>(sel + o) = __halves2half2(th[a * TP], th[b * TP + 1]);
        }
    }
}

// s <= SMAX: sorted list in registers, one branch-free insertion per atom (any dtype, any W).
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
    const int64_t cap = (int64_t)sm_count() * 64;
    if (blocks > cap) blocks = cap;
    const CoefT* c = (const CoefT*)coef;
    CoefT* sl = (CoefT*)sel;
    if (pb.s <= 4) select_insert_kernel<CoefT, 4><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else if (pb.s <= 8) select_insert_kernel<CoefT, 8><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else if (pb.s <= 16) select_insert_kernel<CoefT, 16><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else select_scan_kernel<CoefT><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    count_launches(1);
    return cudaGetLastError();
}

// binary16 fast path: needs 4-byte aligned pixel pairs in every plane and in the outputs
bool pair_path_ok(const void* coef, const uint8_t* idx, const void* sel, const Problem& pb)
{
    return pb.s <= 16 && (pb.W & 1) == 0 && (reinterpret_cast<uintptr_t>(coef) & 3) == 0 &&
           (reinterpret_cast<uintptr_t>(idx) & 1) == 0 && (reinterpret_cast<uintptr_t>(sel) & 3) == 0;
}

// The tile kernel additionally needs 16-byte aligned planes and its tile in shared memory.
bool tile_path_ok(const void* coef, const Problem& pb)
{
    const int64_t HW = (int64_t)pb.H * pb.W;
    return (HW & 7) == 0 && (reinterpret_cast<uintptr_t>(coef) & 15) == 0 && pb.D <= 200 &&
           (HW + kSelTilePixels - 1) / kSelTilePixels * pb.n <= 0x7FFFFFFF;
}

template <int S, int TP>
cudaError_t launch_tilef_s(const __half* c, uint8_t* idx, __half* sl, const Problem& pb, cudaStream_t st)
{
    const size_t smem = (size_t)pb.D * TP * sizeof(__half);
    auto kern = select_tilef_kernel<S, TP>;
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * TP * (int)sizeof(__half));
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int64_t tiles_per_frame = ((int64_t)pb.H * pb.W + TP - 1) / TP;
    if (tiles_per_frame * pb.n > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
    kern<<<(unsigned)(tiles_per_frame * pb.n), TP / 2, smem, st>>>(c, idx, sl, pb, (int)tiles_per_frame);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_tile(const void* coef, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st)
{
    const __half* c = (const __half*)coef;
    __half* sl = (__half*)sel;
    if (pb.s <= 4) return launch_tilef_s<4, kSelTilePixels>(c, idx, sl, pb, st);
    if (pb.s <= 8) return launch_tilef_s<8, kSelTilePixels>(c, idx, sl, pb, st);
    return launch_tilef_s<16, kSelTilePixels>(c, idx, sl, pb, st);
}

cudaError_t launch_pair(const void* coef, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st)
{
    // One block per 256 pixel pairs, launched in order, so that the resident blocks sweep the planes as one
    // contiguous window (a capped grid with a grid-stride loop keeps every block on several far-apart windows at
    // once: 72 planes x that many pages in flight, which cost 60 % more time per pixel on 4K frames).
    const int64_t total = (int64_t)pb.n * pb.H * pb.W / 2;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = 0x7FFFFFFF;
    if (blocks > cap) blocks = cap;
    const __half* c = (const __half*)coef;
    __half* sl = (__half*)sel;
    if (pb.s <= 4) select_pair_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else if (pb.s <= 8) select_pair_kernel<8><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    else select_pair_kernel<16><<<(unsigned)blocks, 256, 0, st>>>(c, idx, sl, pb);
    count_launches(1);
    return cudaGetLastError();
}

} // namespace

cudaError_t launch_select(const void* coef, int coef_dtype, uint8_t* idx, void* sel, const Problem& pb, cudaStream_t st)
{
    if (coef_dtype == SR_F16) {
        if (pair_path_ok(coef, idx, sel, pb)) return tile_path_ok(coef, pb) ? launch_tile(coef, idx, sel, pb, st) : launch_pair(coef, idx, sel, pb, st);
        return launch_sel<__half>(coef, idx, sel, pb, st);
    }
    return launch_sel<float>(coef, idx, sel, pb, st);
}

} // namespace sr
