// Internal helpers shared by the translation units of libdynbatch.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "dynbatch.h"

namespace dynbatch {

// Records the runtime's message for db_last_cuda_error() and returns DB_ERR_CUDA.
db_status record_cuda_error(cudaError_t err, const char* where);

// Stores a plain message for db_last_cuda_error() (non-CUDA failures that need explaining).
void record_message(const char* text);

// Number of SMs of the current device (queried once per device, then cached).
int sm_count();

// Pieces of the aggregation step used by the host pipeline (defined in aggregate.cu).
// aggregate_chunk enqueues only the aggregation kernel for N elements; each of its CTAs leaves the sum
// of its squared aggregated gradients in partials[0 .. *ctas) (partials may be NULL: no norm).
// finalize_norm folds n partials in index order into *sq_out with one more small kernel.
long long aggregate_cta_bound(int64_t N);
db_status aggregate_chunk(const void* const* grads, db_dtype grad_dtype, const int32_t* b, int32_t K, int64_t N,
                          float* params, float* momentum, float lr, float mu, double* partials, long long* ctas,
                          void* cuda_stream);
db_status finalize_norm(const double* partials, long long n, double* sq_out, cudaStream_t stream);

#define DB_CUDA_TRY(expr)                                              \
    do {                                                               \
        cudaError_t db_err__ = (expr);                                 \
        if (db_err__ != cudaSuccess)                                   \
            return ::dynbatch::record_cuda_error(db_err__, #expr);     \
    } while (0)

}  // namespace dynbatch
