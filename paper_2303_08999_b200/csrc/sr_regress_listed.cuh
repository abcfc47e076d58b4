// Regression from per-pixel lists (index planes + value planes) on the fp32 FMA pipe: declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// True when this path can run the problem: compact mode (idx [n][s][H][W] uint8 with its binary16 values
// [n][s][H][W]), s <= 16, k in {3, 5, 7}, c in {1, 3}, W even, idx rows 2-byte aligned, value rows 4-byte aligned,
// output rows aligned for one store per pixel pair, and the replicated dictionary plus two tile sets fit shared memory.
bool regress_listed_supported(int mode, const void* coef, int coef_dtype, const uint8_t* idx, const void* out, const Problem& pb);

cudaError_t launch_regress_listed(const float* lr, const void* val, const uint8_t* idx, const float* dict, float* out,
                                  const Problem& pb, cudaStream_t st, int th_forced = 0);

// Tile heights (8, 16, 24) the problem admits; returns how many were written.
int regress_listed_candidates(const Problem& pb, int* ths, int max_out);

} // namespace sr
