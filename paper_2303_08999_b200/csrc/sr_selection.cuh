// Dictionary selection search (Section III-A, Algorithm 1) on the device: declarations.
#pragma once
#include "sr_common.cuh"

namespace sr {

// Scratch of the Gram kernel: one fp64 slot per CTA.
int selection_gram_slots();
size_t selection_gram_slot_bytes(int D);

cudaError_t launch_selection_gram(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                                  const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const Problem& pb,
                                  double* slots, int nslots, cudaStream_t st);

// The same with the slots in a device array that is part of the library (at most selection_gram_static_max_atoms()
// atoms): nothing is allocated and the caller passes no scratch.
int selection_gram_static_max_atoms();
cudaError_t launch_selection_gram_static(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                                         const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const Problem& pb,
                                         cudaStream_t st);

// Scratch of the search kernel: the matrix its Cholesky factorisation works in.
size_t selection_search_scratch_bytes(int L);

cudaError_t launch_selection_search(const double* G, const double* b, const double* hh, double nrows, int L, const sr_search_opts& o,
                                    uint8_t* idx_out, float* gamma_out, int* count_out, double* trace, int* steps_out, double* chol,
                                    cudaStream_t st);

} // namespace sr
