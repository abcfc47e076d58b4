// Global-subset regression with at most eight atoms on the fp32 FMA pipe: declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// True when this path can run the problem (global subset, s <= 8, binary16 coefficients, c in {1, 3}, W % 4 == 0,
// coefficient rows 8-byte aligned, output rows 16-byte aligned (8 with binary16 output)).
bool regress_subset_supported(int mode, const void* coef, int coef_dtype, const void* out, const Problem& pb);

cudaError_t launch_regress_subset(const float* lr, const void* coef, const uint8_t* idx, const float* gamma, const float* dict,
                                  float* out, const Problem& pb, cudaStream_t st, int th_forced = 0);

// Tile heights (8, 16, 24) the problem admits; returns how many were written.
int regress_subset_candidates(const Problem& pb, int* ths, int max_out);

} // namespace sr
