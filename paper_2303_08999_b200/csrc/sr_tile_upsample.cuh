// Up-sampled tile in shared memory, shared by the regression kernels that walk HR tiles of tw x th pixels (tw = 128
// unless a kernel asks otherwise):
// tile geometry, the LR window a tile needs, its asynchronous fetch, and the two separable passes (stage 1 of the
// method, Section II-A; bicubic or bilinear taps come from the per-phase table in Problem).
//   sL [c * nrows][tcols]   LR window (rows flattened as ch * nrows + j)
//   sV [c][uh][tcols]       after the vertical pass (HR rows, LR columns)
//   sU [c][uh][UW]          the up-sampled tile with a halo of P = (k-1)/2 pixels, patch positions clamped in HR
//                           coordinates (edge replicate)
// All three buffers must start as zeros (or hold finite values): the horizontal pass reads a few staged values beyond
// the ones it weights and multiplies them by zero.
#pragma once

#include "sr_common.cuh"

namespace sr {
namespace tile {

constexpr int TW = 128;   // default tile width in HR pixels

struct Geom {
    Problem pb;
    int tw;               // tile width
    int th, uh;           // tile height, and th + 2 P (rows allocated for the U tile)
    int trows, tcols;     // LR rows / columns a tile can need (tcols a multiple of 4)
    int lr_vec;           // 1: LR rows are 16-byte aligned (16-byte copies for the inner part of the window)
    uint32_t r_magic;     // ceil(2^32 / r): floor(x / r) == umulhi(x, r_magic) for 0 <= x < 2^29 (r >= 2)
    uint32_t tc4_magic;   // same for tcols / 4
    int tiles_x, tiles_y, num_tiles;
    int gps, num_groups;  // 8-row groups per column strip (ceil(H / 8)) and in all strips of all frames
};

// U tile width for patch radius P: tile + halo, rounded up to 4 for 16-byte rows.
__host__ __device__ constexpr int tile_uw(int P, int tw = TW) { return (tw + 2 * P + 3) & ~3; }

// Host side: fills th-dependent sizes; returns the floats the three buffers need.
inline size_t plan_geom(Geom& g, const Problem& pb, int th, const float* lr, int tw = TW)
{
    const int P = (pb.k - 1) / 2, UW = tile_uw(P, tw);
    g.pb = pb;
    g.tw = tw;
    g.th = th;
    g.uh = th + 2 * P;
    g.trows = (g.uh - 1) / pb.r + 5;
    g.tcols = ((UW - 1) / pb.r + 5 + 3 /* window start rounded down to 4 */ + 3) & ~3;
    g.lr_vec = ((reinterpret_cast<uintptr_t>(lr) & 15) == 0 && (pb.w & 3) == 0) ? 1 : 0;
    g.r_magic = pb.r > 1 ? (uint32_t)((0x100000000ull + pb.r - 1) / pb.r) : 0u;
    const int tc4 = g.tcols / 4;
    g.tc4_magic = (uint32_t)((0x100000000ull + tc4 - 1) / tc4);
    g.tiles_x = (pb.W + tw - 1) / tw;
    g.tiles_y = (pb.H + th - 1) / th;
    g.num_tiles = g.tiles_x * g.tiles_y * pb.n;
    g.gps = (pb.H + 7) / 8;
    g.num_groups = g.gps * g.tiles_x * pb.n;
    return (size_t)pb.c * g.uh * UW + (size_t)pb.c * g.uh * g.tcols + (size_t)pb.c * g.trows * g.tcols;
}

#ifdef __CUDACC__

__device__ __forceinline__ int fast_div(int x, int d, uint32_t magic) { return d == 1 ? x : (int)__umulhi((uint32_t)x, magic); }

__device__ __forceinline__ void decode_tile(const Geom& p, int t, int& f, int& y0, int& x0, int& rows)
{
    const int tx = t % p.tiles_x;
    const int rest = t / p.tiles_x;
    const int ty = rest % p.tiles_y;
    f = rest / p.tiles_y;
    y0 = ty * p.th;
    x0 = tx * p.tw;
    rows = min(p.th, p.pb.H - y0);
}

// A worker's share of the image as a run of consecutive 8-row groups [cur, end) of the flattened space
// [frame][column strip][group of 8 rows]: worker j of nworkers takes [j T / nworkers, (j + 1) T / nworkers), T =
// num_groups, so that every worker filters the same number of rows to within one group, whatever the frame height.
// next_tile_of_run cuts the next tile off the run: up to th rows (th a multiple of 8), never across a strip's end.
__device__ __forceinline__ int run_bound(const Geom& p, int j, int nworkers)
{
    return (int)(((long long)j * p.num_groups) / nworkers);
}

__device__ __forceinline__ bool next_tile_of_run(const Geom& p, int& cur, int end, int& f, int& y0, int& x0, int& rows)
{
    if (cur >= end) return false;
    const int strip = cur / p.gps, gy = cur - strip * p.gps;
    const int ng = min(min(p.th >> 3, p.gps - gy), end - cur);
    f = strip / p.tiles_x;
    x0 = (strip - f * p.tiles_x) * p.tw;
    y0 = gy * 8;
    rows = min(ng * 8, p.pb.H - y0);
    cur += ng;
    return true;
}

// LR pixels a tile (plus patch halo) needs for its taps: rows lr_lo .. lr_lo + nrows - 1 and columns
// col_a .. col_a + 4 nc4 - 1 (col_a a multiple of 4, possibly negative; reads clamp to the image).
struct LrWindow { int f, y0, x0, rows, lr_lo, nrows, col_a, nc4; };

// First tap of HR coordinate Z (already clamped to the image) along one axis, and its phase.
__device__ __forceinline__ int first_tap(const Geom& p, int Z, int& phase)
{
    const int q = fast_div(Z, p.pb.r, p.r_magic);
    phase = Z - q * p.pb.r;
    return q + p.pb.ph.base[phase];
}

// Fills the window fields of g from its tile fields (f, y0, x0, rows).
template <int P, int TWD = TW>
__device__ __forceinline__ void lr_window_of_tile(const Geom& p, LrWindow& g)
{
    constexpr int UW = tile_uw(P, TWD);
    const Problem& pb = p.pb;
    int ph;
    g.lr_lo = first_tap(p, clampi(g.y0 - P, 0, pb.H - 1), ph);
    g.nrows = first_tap(p, clampi(g.y0 + g.rows - 1 + P, 0, pb.H - 1), ph) + 3 - g.lr_lo + 1;      // <= trows
    const int col_lo = first_tap(p, clampi(g.x0 - P, 0, pb.W - 1), ph);
    const int col_hi = first_tap(p, clampi(g.x0 - P + UW - 1, 0, pb.W - 1), ph) + 3;
    g.col_a = col_lo & ~3;                                       // rounds down, also for negative values
    g.nc4 = (col_hi - g.col_a) / 4 + 1;                          // <= tcols / 4
}

template <int P, int TWD = TW>
__device__ __forceinline__ void lr_window(const Geom& p, int t, LrWindow& g)
{
    decode_tile(p, t, g.f, g.y0, g.x0, g.rows);
    lr_window_of_tile<P, TWD>(p, g);
}

__device__ __forceinline__ void cp_async_4(float* dst_smem, const float* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_16(float* dst_smem, const float* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

// Fetches the LR window of tile t into dstL with asynchronous copies: 16 bytes where the four columns lie inside the
// image and the row is aligned, single clamped elements at the borders. Thread `me` of `nthr`; the caller waits for
// the copies (cp.async.wait_all or an mbarrier arrival).
__device__ __forceinline__ void prefetch_lr_window_of(const Geom& p, const float* lr, const LrWindow& g, float* dstL, int me, int nthr)
{
    const Problem& pb = p.pb;
    const int C = pb.c;
    const int tc4 = p.tcols >> 2;
    const int total = C * g.nrows * tc4;
    for (int e = me; e < total; e += nthr) {
        const int row = fast_div(e, tc4, p.tc4_magic), c4 = e - row * tc4;
        if (c4 < g.nc4) {
            const int ch = (row >= g.nrows) + (row >= 2 * g.nrows) + (row >= 3 * g.nrows);
            const int j = row - ch * g.nrows;
            const float* src_row = lr + (((int64_t)g.f * C + ch) * pb.h + clampi(g.lr_lo + j, 0, pb.h - 1)) * pb.w;
            const int col = g.col_a + 4 * c4;
            float* dst = dstL + row * p.tcols + 4 * c4;
            if (p.lr_vec && col >= 0 && col + 3 < pb.w) {
                cp_async_16(dst, src_row + col);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) cp_async_4(dst + i, src_row + clampi(col + i, 0, pb.w - 1));
            }
        }
    }
}

template <int P, int TWD = TW>
__device__ __forceinline__ void prefetch_lr_window(const Geom& p, const float* lr, int t, float* dstL, int me, int nthr)
{
    LrWindow g;
    lr_window<P, TWD>(p, t, g);
    prefetch_lr_window_of(p, lr, g, dstL, me, nthr);
}

// Vertical pass on the LR columns of the window: V[ch][uy][i] = sum_a wy[a] * L[ch][first tap of row uy + a][i], four
// LR columns per trip. A thread keeps its column group i4 and walks the rows row_lane, row_lane + row_lanes, ...
__device__ __forceinline__ void vertical_pass(const Geom& p, const LrWindow& g, int uh, int P, const float* sL, float* sV,
                                              int i4, int row_lane, int row_lanes)
{
    const Problem& pb = p.pb;
    if (i4 >= 4 * g.nc4) return;
    for (int row = row_lane; row < pb.c * uh; row += row_lanes) {
        const int ch = (row >= uh) + (row >= 2 * uh) + (row >= 3 * uh);
        const int uy = row - ch * uh;
        int py;
        const int off = first_tap(p, clampi(g.y0 - P + uy, 0, pb.H - 1), py) - g.lr_lo;
        const float w0 = pb.ph.w[py][0], w1 = pb.ph.w[py][1], w2 = pb.ph.w[py][2], w3 = pb.ph.w[py][3];
        const float* src = sL + (ch * g.nrows + off) * p.tcols + i4;
        const float4 t0 = *reinterpret_cast<const float4*>(src);
        const float4 t1 = *reinterpret_cast<const float4*>(src + p.tcols);
        const float4 t2 = *reinterpret_cast<const float4*>(src + 2 * p.tcols);
        const float4 t3 = *reinterpret_cast<const float4*>(src + 3 * p.tcols);
        float4 v;
        v.x = fmaf(w3, t3.x, fmaf(w2, t2.x, fmaf(w1, t1.x, w0 * t0.x)));
        v.y = fmaf(w3, t3.y, fmaf(w2, t2.y, fmaf(w1, t1.y, w0 * t0.y)));
        v.z = fmaf(w3, t3.z, fmaf(w2, t2.z, fmaf(w1, t1.z, w0 * t0.z)));
        v.w = fmaf(w3, t3.w, fmaf(w2, t2.w, fmaf(w1, t1.w, w0 * t0.w)));
        *reinterpret_cast<float4*>(sV + (ch * p.uh + uy) * p.tcols + i4) = v;
    }
}

// The four tap weights of every phase between zeros (0 0 0 w0 w1 w2 w3 0 0 0 ..): row `phase` of wpad, 12 floats.
__device__ __forceinline__ void fill_wpad(const Problem& pb, float (*wpad)[12], int me, int nthr)
{
    for (int i = me; i < kMaxScale * 12; i += nthr) {
        const int phs = i / 12, j = i - phs * 12;
        wpad[phs][j] = (j >= 3 && j < 7) ? pb.ph.w[phs][j - 3] : 0.f;
    }
}

// Horizontal pass: U[ch][uy][ux] = sum_b wx[b] * V[ch][uy][first tap of column ux + b]. A thread keeps the four
// neighbouring columns 4 cg .. 4 cg + 3 for the whole tile. Their first taps are at most three LR columns apart, so
// the four outputs are one 4 x 7 matrix (taps shifted by each column's offset, zeros elsewhere; read from the
// zero-padded weight table) times the seven values V[first .. first + 6]: seven shared loads per four outputs.
template <int P, int TWD = TW>
__device__ __forceinline__ void horizontal_pass(const Geom& p, const float (*wpad)[12], const LrWindow& g, int uh, const float* sV,
                                                float* sU, int cg, int row_lane, int row_lanes)
{
    constexpr int UW = tile_uw(P, TWD);
    const Problem& pb = p.pb;
    float wm[4][7];
    int first = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int px;
        const int off = first_tap(p, clampi(g.x0 - P + 4 * cg + i, 0, pb.W - 1), px) - g.col_a;
        if (i == 0) first = off;
        const float* wrow = &wpad[px][3 - (off - first)];        // column j of the matrix row: tap j - (off - first)
#pragma unroll
        for (int j = 0; j < 7; ++j) wm[i][j] = wrow[j];
    }
    for (int row = row_lane; row < pb.c * uh; row += row_lanes) {
        const int ch = (row >= uh) + (row >= 2 * uh) + (row >= 3 * uh);
        const int uy = row - ch * uh;
        const float* src = sV + (ch * p.uh + uy) * p.tcols + first;
        float v[7];
#pragma unroll
        for (int j = 0; j < 7; ++j) v[j] = src[j];
        float o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float a = wm[i][0] * v[0];
#pragma unroll
            for (int j = 1; j < 7; ++j) a = fmaf(wm[i][j], v[j], a);
            o[i] = a;
        }
        *reinterpret_cast<float4*>(sU + (ch * p.uh + uy) * UW + 4 * cg) = make_float4(o[0], o[1], o[2], o[3]);
    }
}

#endif // __CUDACC__

} // namespace tile
} // namespace sr
