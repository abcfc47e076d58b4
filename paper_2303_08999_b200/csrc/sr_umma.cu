// Fused regression kernel for sm_100a: coefficient planes streamed into shared memory (TMA boxes for the leading
// planes of a stage, 16-byte asynchronous copies for the rest, so that both load paths of the SM work side by side),
// dictionary assembly F = Phi D on the tcgen05 tensor cores with fp32 accumulators in tensor memory, bicubic tile +
// patch dot product + clamp in the epilogue. The filter matrix F (TMEM / registers), the up-sampled image U and its
// patches (shared memory) never reach HBM: per HR pixel the kernel reads its coefficients once and writes its c
// output values once.
//
// One persistent CTA per SM walks HR tiles of 128 x 16 (or 128 x 8) pixels. A tile row (128 pixels of one HR row) is
// one pipeline stage [atoms][128 pixels] binary16 in the 128-byte-swizzled MN-major layout the tensor core reads
// (pixels are M, atoms are K), so the planar [n][D][H][W] coefficient tensor needs no transpose. The dictionary is
// the B operand (K-major): its fp32 values are split into binary16 hi + lo parts (~22 bits kept) that sit side by
// side along N, so one MMA per 16 atoms reads the coefficient stage once and yields both partial filters; the
// epilogue adds them. N = 2 x (k*k padded to 16).
//
// Shared-memory bandwidth and per-warp latency are the scarce on-chip resources, so the epilogue keeps a sliding
// k x k x 3 window of U in registers and reads each U row once per pixel column.
//
// Warp roles, dense and global-subset modes (640 threads = five warpgroups; the register file is re-balanced between
// them with setmaxnreg):
//   warps 0-3    coefficient producers (two groups, alternate rows)   full[stage] <- copy arrivals when the data
//                has landed; wait empty[stage]
//   warps 4-5    MMA issuers (warp 4 owns TMEM): one thread each, alternate rows, because the issue loop of a
//                single thread (~600 cycles per row alone, twice that on a busy SM) would otherwise pace the kernel;
//                acc_full[a], empty[stage] <- tcgen05.commit; wait full[stage] (ready[stage] when selecting), acc_empty[a]
//   warps 6-11   U producers             bicubic (separable) of the tile + halo into a double-buffered tile
//   warps 12-19  epilogue (2 x 4 warps)  TMEM -> registers (one pixel's filter per thread), patch dot, clamp, store;
//                                        the two groups own the upper and the lower half of a tile
// Selective modes (768 threads): warps 6-7 idle, warps 8-15 are select warps that mask each landed stage in place
// (two per stage, one 64-pixel chunk each; ready[stage] <- 64 arrivals), warps 16-23 are the epilogue, which also
// builds its own U tile before each tile's rows.
// Every wait is bounded; on expiry the CTA raises its abort flag, sets the device status word and drains.
#include <stdlib.h>

#include "sr_ptx.cuh"
#include "sr_umma.cuh"

namespace sr {

namespace {

using namespace ptx;

// The kernel is instantiated for two tile heights: 16 rows (less halo work per pixel) and 8 rows, for selective
// launches whose U tile would otherwise leave fewer than eight coefficient stages.
namespace th16 {
#define SR_UMMA_TH 16
#include "sr_umma_impl.inc"
#undef SR_UMMA_TH
} // namespace th16

namespace th8 {
#define SR_UMMA_TH 8
#include "sr_umma_impl.inc"
#undef SR_UMMA_TH
} // namespace th8

} // namespace

// Tile height per mode: 16 rows wherever the shape still leaves the selective pipeline its eight stages (dense and
// global-subset modes always; the in-kernel selection when the single U buffer it needs fits), else 8 rows.
static bool tall_tiles(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    if (!th8::is_selective(mode)) return true;
    // (compact values: nothing streams into the stages, four are enough)
    return th16::supported(mode, coef, coef_dtype, pb) && th16::stage_count(mode, pb) >= (mode == kModeCompact ? 4 : 8);
}

bool umma_supported(int mode, const void* coef, int coef_dtype, const Problem& pb)
{
    return tall_tiles(mode, coef, coef_dtype, pb) ? th16::supported(mode, coef, coef_dtype, pb) : th8::supported(mode, coef, coef_dtype, pb);
}

cudaError_t launch_regress_umma(int mode, const float* lr, const void* coef, const uint8_t* idx, const float* gamma,
                                const float* dict, float* out, const Problem& pb, cudaStream_t st)
{
    return tall_tiles(mode, coef, SR_F16, pb) ? th16::launch(mode, lr, coef, idx, gamma, dict, out, pb, st)
                                               : th8::launch(mode, lr, coef, idx, gamma, dict, out, pb, st);
}

} // namespace sr
