// Status strings, per-thread CUDA error text and device-attribute cache.
#include <cstdio>

#include "common.h"

namespace dynbatch {

static thread_local char g_cuda_msg[256] = "";

db_status record_cuda_error(cudaError_t err, const char* where) {
    std::snprintf(g_cuda_msg, sizeof g_cuda_msg, "%s: %s (%s)", where,
                  cudaGetErrorName(err), cudaGetErrorString(err));
    (void)cudaGetLastError();  // clear the sticky-less error state for the next call
    return DB_ERR_CUDA;
}

void record_message(const char* text) { std::snprintf(g_cuda_msg, sizeof g_cuda_msg, "%s", text); }

int sm_count() {
    constexpr int kMaxDev = 64;
    static int cache[kMaxDev] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return 148;
    int n = cache[dev];
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
            n = 148;
        cache[dev] = n;  // benign race: every thread writes the same value
    }
    return n;
}

}  // namespace dynbatch

extern "C" const char* db_status_string(db_status s) {
    switch (s) {
        case DB_OK: return "ok";
        case DB_ERR_NULL: return "required pointer is NULL";
        case DB_ERR_ARG: return "argument out of range";
        case DB_ERR_UNSUPPORTED: return "unsupported dtype or configuration";
        case DB_ERR_INFEASIBLE: return "batch-size bounds cannot sum to the global batch";
        case DB_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

extern "C" const char* db_last_cuda_error(void) { return dynbatch::g_cuda_msg; }
