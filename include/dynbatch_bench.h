/*
 * Measurement helpers of libdynbatch.  None of these is part of the training
 * step's API and the paper has no counterpart for any of them: they exist so
 * that the bandwidth figures and the design comparisons reported for the
 * aggregation kernel (Section 3.1, Eq. 2-3) can be reproduced from this tree.
 *
 * Conventions are those of dynbatch.h: caller-owned device memory, work is
 * enqueued on `cuda_stream` without synchronising, a db_status comes back,
 * arguments are validated before anything is enqueued.
 */
#ifndef DYNBATCH_BENCH_H_
#define DYNBATCH_BENCH_H_

#include "dynbatch.h"

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

/* Read-only bandwidth probe: one kernel streams `bytes` bytes of `src` (device,
 * 16-byte aligned, bytes a multiple of 16) through registers with the loads
 * the aggregation kernel uses for its gradients (128-bit, streaming) and
 * writes an 8-byte checksum per CTA to `sink` (device, >=
 * db_bench_read_probe_sink_bytes(bytes) bytes).  bytes / time is the rate at
 * which this GPU delivers a pure read stream: the second denominator, beside a
 * device-to-device copy, for a step that is 75-94 % reads. */
size_t db_bench_read_probe_sink_bytes(size_t bytes);
db_status db_bench_read_probe(const void* src, size_t bytes, void* sink,
                              void* cuda_stream);

/* The aggregation + momentum step in the two shapes that were measured against
 * the kept kernel and not adopted, with the same per-element arithmetic
 * (results are bit-identical to db_aggregate_update_ex):
 *   DB_BENCH_PERSISTENT   a grid of SMs x resident CTAs, each striding over the
 *                         tiles (the "persistent grid-stride" launch);
 *   DB_BENCH_BULK_STAGED  every stream's tile is staged in shared memory by
 *                         cp.async.bulk on one mbarrier, combined from there and
 *                         stored back by cp.async.bulk; `stage_floats` floats per
 *                         stream and CTA (512, 1024 or 2048).
 * Restricted to what the comparison needs: fp32 gradients, no norm, K in
 * {2, 4, 8, 16} all with b[k] > 0, N a multiple of 4, every buffer 16-byte
 * aligned; anything else is DB_ERR_UNSUPPORTED.  `status` (device int32,
 * zeroed by the caller, or NULL) is set non-zero if a staged CTA's bounded
 * wait for its copies ran out; that CTA then stores nothing. */
typedef enum { DB_BENCH_PERSISTENT = 1, DB_BENCH_BULK_STAGED = 2 } db_bench_variant;

db_status db_bench_aggregate_variant(db_bench_variant variant, int32_t stage_floats,
                                     const float* const* grads, const int32_t* b,
                                     int32_t K, int64_t N, float* params,
                                     float* momentum, float lr, float mu,
                                     int32_t* status, void* cuda_stream);

/* The time-limited wait of the tensor-core kernels, made to run out: one CTA
 * waits on an mbarrier that nothing ever arrives on, gives up after limit_ns
 * nanoseconds (at most 2e9), writes `code` to *status (device int32, zeroed by
 * the caller) and returns normally.  This is how those kernels report a wait
 * that never ends -- a status word the host reads, the context stays usable --
 * and the only way to see that path taken without a faulty kernel. */
db_status db_bench_wait_timeout(int32_t* status, int32_t code, uint64_t limit_ns,
                                void* cuda_stream);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif

#ifdef __cplusplus
}
#endif

#endif /* DYNBATCH_BENCH_H_ */
