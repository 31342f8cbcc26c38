// The parameter-server step for gradients that arrive in HOST memory.
//
// The arithmetic is db_aggregate_update_ex's (Section 3.1, Eq. 2-3 + momentum);
// this file only moves data: the parameter range is cut into chunks and three
// streams overlap, chunk by chunk, the host->device copy of the K gradient
// slices (copy-in stream), the fused aggregate/update kernel (the caller's
// stream) and the device->host copy of the updated parameters (copy-out
// stream), so that PCIe runs in both directions while the kernel works on the
// previous chunk.  Two staging slots in device memory hold the chunks in flight.
#include <cstdint>
#include <cmath>
#include <new>

#include "common.h"

struct db_host_pipeline {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, loaded[2] = {nullptr, nullptr}, computed[2] = {nullptr, nullptr},
                drained = nullptr;
    int device = -1;
};

namespace dynbatch {
namespace {

constexpr int64_t kDefaultChunk = 1 << 21;  // elements per chunk
constexpr int kSlots = 2;

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

int64_t chunk_or_default(int64_t chunk_elems) {
    if (chunk_elems <= 0) return kDefaultChunk;
    return (chunk_elems + 7) / 8 * 8;  // keeps every chunk start on a 16-byte boundary (fp32 and bf16)
}

struct StagingLayout {
    size_t slot_bytes, slots_off, partials_off, total_off, end;
};

StagingLayout layout(int32_t K, db_dtype dt, int64_t N, int64_t chunk) {
    StagingLayout L;
    const size_t gsize = dt == DB_F32 ? 4 : 2;
    L.slot_bytes = round256(static_cast<size_t>(K) * chunk * gsize);
    L.slots_off = 0;
    // every CTA of every chunk leaves one partial sum of the squared norm; one kernel folds them at the end
    L.partials_off = L.slots_off + kSlots * L.slot_bytes;
    const int64_t nchunks = N > 0 ? (N + chunk - 1) / chunk : 1;
    L.total_off = L.partials_off +
                  round256(sizeof(double) * static_cast<size_t>(nchunks * aggregate_cta_bound(chunk)));
    L.end = L.total_off + 256;
    return L;
}

}  // namespace
}  // namespace dynbatch

extern "C" size_t db_host_staging_bytes(int32_t K, db_dtype grad_dtype, int64_t N, int64_t chunk_elems) {
    using namespace dynbatch;
    if (K < 1 || K > DB_MAX_K || N < 0 || (grad_dtype != DB_F32 && grad_dtype != DB_BF16)) return 0;
    return layout(K, grad_dtype, N, chunk_or_default(chunk_elems)).end;
}

extern "C" db_status db_host_pipeline_destroy(db_host_pipeline* h) {
    if (!h) return DB_OK;
    if (h->in) cudaStreamSynchronize(h->in);
    if (h->out) cudaStreamSynchronize(h->out);
    cudaEvent_t evs[] = {h->start, h->loaded[0], h->loaded[1], h->computed[0], h->computed[1], h->drained};
    for (cudaEvent_t e : evs)
        if (e) cudaEventDestroy(e);
    if (h->in) cudaStreamDestroy(h->in);
    if (h->out) cudaStreamDestroy(h->out);
    delete h;
    return DB_OK;
}

extern "C" db_status db_host_pipeline_create(db_host_pipeline** out) {
    using namespace dynbatch;
    if (!out) return DB_ERR_NULL;
    *out = nullptr;
    db_host_pipeline* h = new (std::nothrow) db_host_pipeline();
    if (!h) return DB_ERR_ARG;
    cudaError_t err = cudaGetDevice(&h->device);
    if (err == cudaSuccess) err = cudaStreamCreateWithFlags(&h->in, cudaStreamNonBlocking);
    if (err == cudaSuccess) err = cudaStreamCreateWithFlags(&h->out, cudaStreamNonBlocking);
    cudaEvent_t* evs[] = {&h->start, &h->loaded[0], &h->loaded[1], &h->computed[0], &h->computed[1], &h->drained};
    for (cudaEvent_t* e : evs)
        if (err == cudaSuccess) err = cudaEventCreateWithFlags(e, cudaEventDisableTiming);
    if (err != cudaSuccess) {
        const db_status st = record_cuda_error(err, "db_host_pipeline_create");
        db_host_pipeline_destroy(h);
        return st;
    }
    *out = h;
    return DB_OK;
}

extern "C" db_status db_aggregate_update_host(db_host_pipeline* h, const void* const* host_grads,
                                              db_dtype grad_dtype, const int32_t* b, int32_t K, int64_t N,
                                              float* params, float* momentum, float lr, float mu,
                                              float* host_params_out, double* host_sqnorm_out,
                                              void* staging, size_t staging_bytes, int64_t chunk_elems,
                                              void* cuda_stream) {
    using namespace dynbatch;
    if (!h || !host_grads || !b) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || N < 0) return DB_ERR_ARG;
    if (grad_dtype != DB_F32 && grad_dtype != DB_BF16) return DB_ERR_UNSUPPORTED;
    long long total = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        if (b[k] > 0 && !host_grads[k]) return DB_ERR_NULL;
        total += b[k];
    }
    if (total <= 0) return DB_ERR_ARG;
    if (N == 0) return DB_OK;
    if (!params || !momentum || !staging) return DB_ERR_NULL;
    const int64_t chunk = chunk_or_default(chunk_elems);
    const StagingLayout L = layout(K, grad_dtype, N, chunk);
    if (reinterpret_cast<uintptr_t>(staging) % 256 || staging_bytes < L.end) return DB_ERR_ARG;
    int dev = -1;
    DB_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != h->device) return DB_ERR_ARG;

    cudaStream_t compute = static_cast<cudaStream_t>(cuda_stream);
    const size_t gsize = grad_dtype == DB_F32 ? 4 : 2;
    char* base = static_cast<char*>(staging);
    double* partials = reinterpret_cast<double*>(base + L.partials_off);
    long long n_partials = 0;
    double* total_norm = reinterpret_cast<double*>(base + L.total_off);
    const int64_t nchunks = (N + chunk - 1) / chunk;

    // Everything that can be rejected is rejected here, before the first event is recorded: an error
    // from an argument leaves nothing enqueued on any stream.
    if (!std::isfinite(lr) || !std::isfinite(mu)) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(params) % 4 || reinterpret_cast<uintptr_t>(momentum) % 4) return DB_ERR_ARG;
    {
        const uintptr_t p0 = reinterpret_cast<uintptr_t>(params), v0 = reinterpret_cast<uintptr_t>(momentum);
        const uintptr_t s0 = reinterpret_cast<uintptr_t>(staging);
        const size_t state_bytes = static_cast<size_t>(N) * 4;
        auto overlap = [](uintptr_t a, size_t an, uintptr_t c, size_t cn) { return a < c + cn && c < a + an; };
        if (overlap(p0, state_bytes, v0, state_bytes) || overlap(p0, state_bytes, s0, L.end) ||
            overlap(v0, state_bytes, s0, L.end))
            return DB_ERR_ARG;
    }

    // Everything below is ordered after the caller's earlier work on its stream.
    DB_CUDA_TRY(cudaEventRecord(h->start, compute));
    DB_CUDA_TRY(cudaStreamWaitEvent(h->in, h->start, 0));
    DB_CUDA_TRY(cudaStreamWaitEvent(h->out, h->start, 0));

    auto enqueue_chunks = [&]() -> db_status {
        for (int64_t c = 0; c < nchunks; ++c) {
            const int s = static_cast<int>(c % kSlots);
            const int64_t off = c * chunk;
            const int64_t len = (N - off < chunk) ? (N - off) : chunk;
            char* slot = base + L.slots_off + s * L.slot_bytes;
            const void* slices[DB_MAX_K];

            // copy-in: the slot is free once the kernel that read it two chunks ago has finished
            if (c >= kSlots) DB_CUDA_TRY(cudaStreamWaitEvent(h->in, h->computed[s], 0));
            for (int k = 0; k < K; ++k) {
                char* dst = slot + static_cast<size_t>(k) * chunk * gsize;
                slices[k] = dst;
                if (b[k] == 0) continue;  // weight 0: neither copied nor read
                DB_CUDA_TRY(cudaMemcpyAsync(dst, static_cast<const char*>(host_grads[k]) + off * gsize,
                                            static_cast<size_t>(len) * gsize, cudaMemcpyHostToDevice, h->in));
            }
            DB_CUDA_TRY(cudaEventRecord(h->loaded[s], h->in));

            // compute on the caller's stream
            DB_CUDA_TRY(cudaStreamWaitEvent(compute, h->loaded[s], 0));
            long long ctas = 0;
            const db_status st = aggregate_chunk(slices, grad_dtype, b, K, len, params + off, momentum + off, lr, mu,
                                                 host_sqnorm_out ? partials + n_partials : nullptr, &ctas, compute);
            if (st != DB_OK) return st;
            n_partials += ctas;
            DB_CUDA_TRY(cudaEventRecord(h->computed[s], compute));

            // copy-out of the updated parameters
            if (host_params_out) {
                DB_CUDA_TRY(cudaStreamWaitEvent(h->out, h->computed[s], 0));
                DB_CUDA_TRY(cudaMemcpyAsync(host_params_out + off, params + off, static_cast<size_t>(len) * 4,
                                            cudaMemcpyDeviceToHost, h->out));
            }
        }
        if (host_sqnorm_out) {
            const db_status st = finalize_norm(partials, n_partials, total_norm, compute);
            if (st != DB_OK) return st;
            DB_CUDA_TRY(cudaMemcpyAsync(host_sqnorm_out, total_norm, sizeof(double), cudaMemcpyDeviceToHost, compute));
        }
        return DB_OK;
    };
    const db_status st = enqueue_chunks();
    // The caller's stream completes only after everything queued on the two copy streams has: the last
    // parameter chunk has reached the host, and -- should a CUDA call have failed half way -- no copy of this
    // call is still in flight when the caller's stream moves on.
    cudaError_t join = cudaEventRecord(h->loaded[0], h->in);
    if (join == cudaSuccess) join = cudaStreamWaitEvent(compute, h->loaded[0], 0);
    if (join == cudaSuccess) join = cudaEventRecord(h->drained, h->out);
    if (join == cudaSuccess) join = cudaStreamWaitEvent(compute, h->drained, 0);
    if (st != DB_OK) return st;
    DB_CUDA_TRY(join);
    return DB_OK;
}
