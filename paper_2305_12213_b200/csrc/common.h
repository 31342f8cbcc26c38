// Internal helpers shared by the translation units of libdynbatch.
#pragma once
#include <cuda_runtime.h>

#include "dynbatch.h"

namespace dynbatch {

// Records the runtime's message for db_last_cuda_error() and returns DB_ERR_CUDA.
db_status record_cuda_error(cudaError_t err, const char* where);

// Stores a plain message for db_last_cuda_error() (non-CUDA failures that need explaining).
void record_message(const char* text);

// Number of SMs of the current device (queried once per device, then cached).
int sm_count();

#define DB_CUDA_TRY(expr)                                              \
    do {                                                               \
        cudaError_t db_err__ = (expr);                                 \
        if (db_err__ != cudaSuccess)                                   \
            return ::dynbatch::record_cuda_error(db_err__, #expr);     \
    } while (0)

}  // namespace dynbatch
