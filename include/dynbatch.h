/*
 * libdynbatch -- the parameter-server step of dynamic-batching BSP training
 * (Tyagi & Sharma, "Taming Resource Heterogeneity In Distributed ML Training
 * With Dynamic Batching"), as CUDA kernels for NVIDIA B200 (sm_100a) behind a
 * plain C ABI.
 *
 * Conventions shared by every entry point
 *   - "device" pointers are CUDA device memory owned by the caller; "host"
 *     pointers are ordinary host memory.  The library allocates no device
 *     memory: scratch space is a caller-provided workspace sized by the
 *     matching *_workspace_bytes query.
 *   - Device work is enqueued on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL is the legacy default stream) and the call returns without
 *     synchronising.  Host arrays (batch sizes, pointer tables) are consumed
 *     before the call returns.
 *   - Every call returns a db_status.  Arguments are validated before any
 *     launch; on an argument error (DB_ERR_NULL / ARG / UNSUPPORTED /
 *     INFEASIBLE) nothing has been enqueued and no output is touched.
 *     Nothing throws, aborts or traps.  After DB_ERR_CUDA,
 *     db_last_cuda_error() returns the runtime's message for this thread; an
 *     entry point that enqueues several operations may then have enqueued
 *     some of them, and outputs are unspecified.
 *   - NaN/Inf in the inputs propagate by IEEE rules; they are not checked.
 */
#ifndef DYNBATCH_H_
#define DYNBATCH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

typedef enum {
    DB_OK = 0,
    DB_ERR_NULL = 1,        /* a required pointer is NULL */
    DB_ERR_ARG = 2,         /* a value is out of its documented range */
    DB_ERR_UNSUPPORTED = 3, /* unknown dtype / configuration */
    DB_ERR_INFEASIBLE = 4,  /* batch-size bounds cannot sum to the global batch */
    DB_ERR_CUDA = 5         /* the CUDA runtime reported an error */
} db_status;

typedef enum {
    DB_F32 = 0,  /* IEEE binary32 */
    DB_BF16 = 1  /* bfloat16 (upper half of a binary32) */
} db_dtype;

/* Largest number of workers one call combines. */
#define DB_MAX_K 64

/* ------------------------------------------------------------------------
 * Weighted aggregation + momentum-SGD update      (Section 3.1, Eq. 2-3;
 * momentum optimizer of the ResNet-50 workload, Section 4)
 *
 * For every parameter j, in one pass over memory:
 *     g    = sum_k lambda_k * grads[k][j],  lambda_k = b[k] / sum_i b[i]
 *     v[j] = mu * v[j] + g
 *     p[j] = p[j] - lr * v[j]
 * and, optionally, grad_sqnorm = sum_j g^2.
 *
 * grads[k] is worker k's MEAN gradient over its b[k] samples.  The sum runs
 * over k ascending with fp32 fused multiply-adds from a zero accumulator, so
 * results are bit-reproducible and independent of launch geometry (the
 * squared norm is reproducible for a fixed device and K).  Eq. 3's printed
 * 1/K factor is not applied (with sum lambda = 1 it would break the stated
 * equivalence with uniform batching); pass lr/K to get it.
 *
 *   grads          host array of K device pointers, each to N contiguous
 *                  elements of grad_dtype; read-only.  A worker with
 *                  b[k] == 0 has weight 0 and its buffer is never read.
 *   b              host, K mini-batch sizes, each >= 0, sum > 0
 *   K              1..DB_MAX_K
 *   N              number of parameters, >= 0 (0: DB_OK, nothing enqueued,
 *                  *grad_sqnorm left as it was)
 *   params         device, N fp32, updated in place
 *   momentum       device, N fp32, updated in place
 *   lr, mu         finite learning rate and momentum coefficient
 *   grad_sqnorm    device, one double, or NULL to skip the norm
 *   workspace      device scratch of >= db_aggregate_workspace_bytes(K, N)
 *                  bytes, 16-byte aligned; needs no initialisation; may be
 *                  NULL when grad_sqnorm is NULL.  Calls that may overlap on
 *                  the device need distinct workspaces.
 *
 * Any pointer alignment (down to the element size) and any N are accepted;
 * the 128-bit path is taken when params, momentum and all gradient buffers
 * reach a 16-byte boundary after the same number of leading elements,
 * otherwise an element-wise kernel runs.  Gradient buffers must not overlap
 * params or momentum, nor params momentum (DB_ERR_ARG).
 *
 * db_aggregate_update is the fp32, no-norm, default-stream short form.
 * ------------------------------------------------------------------------ */
db_status db_aggregate_update(const float* const* grads, const int32_t* b,
                              int32_t K, int64_t N, float* params,
                              float* momentum, float lr, float mu);

db_status db_aggregate_update_ex(const void* const* grads, db_dtype grad_dtype,
                                 const int32_t* b, int32_t K, int64_t N,
                                 float* params, float* momentum, float lr,
                                 float mu, double* grad_sqnorm, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

size_t db_aggregate_workspace_bytes(int32_t K, int64_t N);

/* ------------------------------------------------------------------------
 * Weighted aggregation + Adam update   (Section 3.1, Eq. 2; Adam is the
 * optimizer of the paper's MNIST workload, Section 4, which prints no formula:
 * this is the textbook rule with bias correction)
 *
 * Same aggregate g as above, then per parameter, with t = step >= 1:
 *     m <- beta1 m + (1 - beta1) g        u <- beta2 u + (1 - beta2) g^2
 *     p <- p - lr * (m / (1 - beta1^t)) / (sqrt(u / (1 - beta2^t)) + eps)
 * first_moment and second_moment are device fp32 buffers of N elements updated
 * in place (zero before step 1).  0 <= beta1, beta2 < 1, eps >= 0.  Every other
 * argument, the alignment rules, the norm and the workspace are those of
 * db_aggregate_update_ex; the pass reads K gradients + 3 state arrays and
 * writes 3: K * sizeof(grad) + 24 bytes per parameter.
 * ------------------------------------------------------------------------ */
db_status db_aggregate_adam_ex(const void* const* grads, db_dtype grad_dtype,
                               const int32_t* b, int32_t K, int64_t N,
                               float* params, float* first_moment,
                               float* second_moment, float lr, float beta1,
                               float beta2, float eps, int64_t step,
                               double* grad_sqnorm, void* workspace,
                               size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------
 * The momentum step over a list of tensors        (Section 3.1, Eq. 2-3)
 *
 * For models whose T parameter tensors (and their gradients and momentum
 * buffers) are separate allocations rather than one arena.  A plan is built
 * once for a fixed set of tensors; each step is then one launch over all of
 * them, with results bit-identical to db_aggregate_update_ex applied tensor by
 * tensor (the squared norm is the sum over all tensors).
 *
 *   grads        host array of K*T device pointers, grads[k*T + t] = worker k's
 *                gradient of tensor t (sizes[t] elements of grad_dtype)
 *   sizes        host, T element counts >= 0
 *   params, momentum   host arrays of T device pointers (fp32, sizes[t] each)
 *   device_table device scratch of >= db_multi_plan_device_bytes(...) bytes,
 *                256-byte aligned; the plan keeps one record per CTA (the
 *                pointers of its tile of one tensor) and the norm's partial
 *                sums there until it is destroyed.  Must outlive the plan.
 *   cuda_stream  (create) the tables are uploaded on it and the call waits for
 *                the upload; (step) the launch stream
 * A tensor whose buffers are all 16-byte aligned takes 128-bit accesses,
 * otherwise element-wise ones.  b[k] == 0: worker k's buffers are not read.
 * The buffers of different tensors must not overlap; steps on one plan must not
 * overlap on the device.
 * ------------------------------------------------------------------------ */
typedef struct db_multi_plan db_multi_plan;

size_t db_multi_plan_device_bytes(int32_t K, db_dtype grad_dtype,
                                  const int64_t* sizes, int32_t T);
db_status db_multi_plan_create(db_multi_plan** out, const void* const* grads,
                               db_dtype grad_dtype, int32_t K,
                               const int64_t* sizes, int32_t T,
                               float* const* params, float* const* momentum,
                               void* device_table, size_t device_table_bytes,
                               void* cuda_stream);
db_status db_aggregate_update_multi(db_multi_plan* plan, const int32_t* b,
                                    float lr, float mu, double* grad_sqnorm,
                                    void* cuda_stream);
db_status db_multi_plan_destroy(db_multi_plan* plan);

/* ------------------------------------------------------------------------
 * The same step for callers that cannot provide scratch memory
 * (the paper has no counterpart; this is a packaging variant of the call above)
 *
 * db_aggregate_update_ex needs a device workspace for the gradient norm, so
 * somebody has to allocate one.  Some callers cannot: a plug-in running inside
 * a host application that has already handed all device memory to its own
 * pool and exposes no allocator to plug-ins; a latency-critical loop in which
 * cudaMalloc is forbidden because it may synchronise the whole device; code
 * that only ever receives raw input/output pointers from its framework.  For
 * them this entry point keeps the scratch inside the library, in a fixed
 * array in device global memory (DB_STATIC_SCRATCH_BYTES = 1 MiB, resident on every
 * GPU that loads the library until the process exits).  It calls no
 * cudaMalloc/cudaFree and no allocating library routine.
 *
 * Arguments and results are those of db_aggregate_update_ex without the
 * workspace pair; results are bit-identical to it.
 *
 *   - The first call on each device looks up the array's device address
 *     (once per device, with that device current).  Make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array.  It keeps the previous
 *     call's contents; nothing in it has to start at zero, since every CTA
 *     of a launch overwrites its own slot before the fold reads it.  Two calls
 *     whose kernels may run at the same time on one device (different
 *     streams, different threads) race on it and return a wrong norm:
 *     serialise them, or use db_aggregate_update_ex with separate workspaces.
 *   - The scratch holds one double per CTA, i.e. per 1024 parameters, so the
 *     built-in 1 MiB serves N up to 134,215,680 parameters when the norm is
 *     requested (any N without it).  Beyond that the call returns
 *     DB_ERR_UNSUPPORTED and enqueues nothing; db_last_cuda_error() then says
 *     how many bytes were needed.
 * ------------------------------------------------------------------------ */
#define DB_STATIC_SCRATCH_BYTES 1048576

db_status db_aggregate_update_static(const void* const* grads,
                                     db_dtype grad_dtype, const int32_t* b,
                                     int32_t K, int64_t N, float* params,
                                     float* momentum, float lr, float mu,
                                     double* grad_sqnorm, void* cuda_stream);

/* ------------------------------------------------------------------------
 * Several parameter servers      (Section 4, experimental setup: the number
 * of parameter servers is scaled so that they are not the bottleneck)
 *
 * The step is element-wise over the parameters, so G servers can each own a
 * contiguous slice of params and momentum and run db_aggregate_update_ex on
 * it, with grads[k] pointing at the same slice of worker k's buffer (on
 * another GPU of the node: a peer mapping; the kernel reads it with ordinary
 * loads).  db_shard_range gives the slice of server r: equal chunks of
 * ceil(N / G) elements rounded up to a multiple of `align` (use 8: slices of
 * 16-byte-aligned fp32 and bf16 buffers then stay on the 128-bit path), the
 * last ones shorter or empty.  The union of the G slices is [0, N) and the
 * results are bit-identical to one call over all N (the norm is the sum of
 * the slices' norms).
 *   N >= 0, G >= 1, 0 <= r < G, align >= 1, else DB_ERR_ARG; begin, end: host.
 * ------------------------------------------------------------------------ */
db_status db_shard_range(int64_t N, int32_t G, int32_t r, int32_t align,
                         int64_t* begin, int64_t* end);

/* ------------------------------------------------------------------------
 * The same step with the gradients in HOST memory   (Section 3.1, Eq. 2-3;
 * in the paper's system the parameter server receives the workers' gradients
 * over the network, i.e. in host buffers, and sends the new model back)
 *
 * db_aggregate_update_host cuts the N parameters into chunks and overlaps,
 * chunk by chunk, the host->device copy of the K gradient slices, the fused
 * aggregate/update kernel and the device->host copy of the updated
 * parameters on three streams.  params/momentum stay resident on the device
 * and are updated in place exactly as by db_aggregate_update_ex (bit-identical:
 * the update is element-wise); the squared norm is the sum of the per-chunk
 * norms in chunk order (same value to rounding).
 *
 *   pipeline         from db_host_pipeline_create on the current device; holds
 *                    two side streams and events, no device memory.  One call at
 *                    a time per pipeline.
 *   host_grads       host array of K HOST pointers, N elements each; page-locked
 *                    memory is needed for the copies to overlap (pageable memory
 *                    works, serialised by the runtime).  b[k] == 0: never read.
 *   params, momentum device, N fp32, in/out
 *   host_params_out  host, N fp32, receives the updated parameters, or NULL
 *   host_sqnorm_out  host, one double, or NULL
 *   staging          device scratch of >= db_host_staging_bytes(K, dtype, N,
 *                    chunk_elems) bytes, 256-byte aligned, uninitialised
 *   chunk_elems      elements per chunk (rounded up to a multiple of 8);
 *                    <= 0 selects the default of 2^21
 *   cuda_stream      the kernels run here; the call is ordered after earlier work
 *                    on it, and work enqueued on it afterwards starts only when
 *                    every copy of this call has finished.  Host outputs are valid
 *                    after synchronising this stream; host_grads must stay
 *                    unchanged until then.
 * ------------------------------------------------------------------------ */
typedef struct db_host_pipeline db_host_pipeline;

db_status db_host_pipeline_create(db_host_pipeline** out);
db_status db_host_pipeline_destroy(db_host_pipeline* pipeline);

size_t db_host_staging_bytes(int32_t K, db_dtype grad_dtype, int64_t N,
                             int64_t chunk_elems);

db_status db_aggregate_update_host(db_host_pipeline* pipeline,
                                   const void* const* host_grads,
                                   db_dtype grad_dtype, const int32_t* b,
                                   int32_t K, int64_t N, float* params,
                                   float* momentum, float lr, float mu,
                                   float* host_params_out,
                                   double* host_sqnorm_out, void* staging,
                                   size_t staging_bytes, int64_t chunk_elems,
                                   void* cuda_stream);

/* ------------------------------------------------------------------------
 * Ragged per-worker gradient of a linear-softmax classifier
 *
 * The model on which the batch-proportional weighting of Eq. 2 is checked
 * against the gradient of the whole global batch (Section 3.1: the weights
 * keep variable batching equivalent to uniform batching).  For worker i with
 * b_i samples:
 *     Z = X W;  P = softmax over each row of Z;  G = X^T (P - Y) / b_i
 * with Y the one-hot labels; no bias; loss = mean cross-entropy.
 *
 *   X     device [b_i, D] row-major fp32
 *   y     device [b_i] int32 labels in [0, C) (a label outside the range
 *         contributes no one-hot term and a zero loss; not an error)
 *   W     device [D, C] row-major fp32
 *   b_i   1..65535,  D >= 1,  C >= 1
 *   G     device [D, C] row-major fp32, overwritten
 *   loss  device, one float (mean cross-entropy), or NULL
 *   workspace  device scratch of >= db_worker_grad_workspace_bytes(b_i, D, C)
 *         bytes, 16-byte aligned, uninitialised.  Its first 32-bit word is a
 *         status word the call clears and the tensor-core kernels set to a
 *         non-zero code if one of their (time-limited) internal waits ever
 *         gives up; it stays 0 in correct operation.  Calls enqueued on one
 *         stream may share a workspace (none of a call's kernels touches it
 *         before the previous call's have finished); calls that may overlap
 *         on the device need distinct workspaces.
 *   flags 0, or DB_WORKER_GRAD_FFMA to run both contractions as plain fp32
 *         FFMA instead of on the tensor cores (the accuracy reference; also
 *         taken automatically for b_i > 4096)
 * Any D, C and alignment down to 4 bytes are accepted; 16-byte aligned X with
 * D a multiple of 4 takes 128-bit loads.
 *
 * On the tensor cores every fp32 product is formed from three TF32 products
 * (operands split into two TF32 halves, fp32 accumulation), which keeps the
 * result within 1e-5 of an fp64 evaluation.  The tensor-core path is the grouped
 * call below with one worker.
 * db_worker_grad is db_worker_grad_ex with flags = 0.
 * ------------------------------------------------------------------------ */
#define DB_WORKER_GRAD_FFMA 1u

db_status db_worker_grad(const float* X, const int32_t* y, const float* W,
                         int32_t b_i, int32_t D, int32_t C, float* G,
                         float* loss, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);

db_status db_worker_grad_ex(const float* X, const int32_t* y, const float* W,
                            int32_t b_i, int32_t D, int32_t C, float* G,
                            float* loss, void* workspace,
                            size_t workspace_bytes, uint32_t flags,
                            void* cuda_stream);

size_t db_worker_grad_workspace_bytes(int32_t b_i, int32_t D, int32_t C);

/* ------------------------------------------------------------------------
 * All K workers' ragged gradients in three launches
 *
 * The workers of one iteration share W, so their logits are one contraction
 * over the concatenated mini-batches; only the 1/b_w scale and the final
 * reduction over each worker's own rows differ.  The last launch computes all
 * K gradients; its operands (the softmax residual and X, split into TF32
 * halves, every worker's rows padded with zero rows to a multiple of 8) reach
 * the tensor cores by TMA.  Worker w owns rows
 * [offsets[w], offsets[w+1]) of X and y (its b_w = their number, Eq. 2's b_k)
 * and receives G[w] = X_w^T (softmax(X_w W) - Y_w) / b_w and losses[w].
 *
 *   X        device [offsets[K], D] row-major fp32, the workers' rows in order
 *   y        device [offsets[K]] int32
 *   W        device [D, C] row-major fp32
 *   offsets  host, K + 1 entries, offsets[0] = 0, strictly increasing (every
 *            worker has at least one sample; at most 4096 per worker:
 *            DB_ERR_UNSUPPORTED beyond)
 *   K        1..DB_MAX_K
 *   G        host array of K device pointers, each [D, C] fp32, overwritten
 *   losses   device, K floats (mean cross-entropy per worker), or NULL
 *   workspace  device scratch of >= db_worker_grad_grouped_workspace_bytes(
 *            offsets[K], K, D, C) bytes, 16-byte aligned, uninitialised; its
 *            first word is the status word described for db_worker_grad_ex
 * Tensor-core path only; results equal db_worker_grad's on each worker to
 * within the fp32 rounding of a differently split reduction over D.  NaN/Inf
 * in one worker's samples stay in that worker's gradient and loss.
 * ------------------------------------------------------------------------ */
db_status db_worker_grad_grouped(const float* X, const int32_t* y,
                                 const float* W, const int32_t* offsets,
                                 int32_t K, int32_t D, int32_t C,
                                 float* const* G, float* losses,
                                 void* workspace, size_t workspace_bytes,
                                 void* cuda_stream);

size_t db_worker_grad_grouped_workspace_bytes(int32_t total_rows, int32_t K,
                                              int32_t D, int32_t C);

/* ------------------------------------------------------------------------
 * The dense fp32 contraction db_worker_grad is built from (both Z = X W and
 * G = X^T E are instances), exposed so that it can be checked in isolation:
 *     out(m, n) = sum_{k < K} A(m, k) * B(n, k)
 * on the tensor cores with three TF32 products per fp32 product.
 *
 *   A(m, k) = A[m * a_row + k * a_k],  B(n, k) = B[n * b_row + k * b_k]
 *   out(m, n) at out[m * o_m + n * o_n]       all device fp32, strides in
 *   elements, >= 0 (outputs >= 1); either operand may be contiguous along k or
 *   along its rows, which selects 128-bit loads when 16-byte aligned.  With A
 *   contiguous along m, B along k and out along m (a_row = b_k = o_m = 1, bases
 *   16-byte aligned, a_k and b_row multiples of 4) the operands travel by TMA,
 *   as for the logits of db_worker_grad.
 *   M, N >= 1, K >= 0 (K = 0 writes zeros)
 *   status   device, one int32 the caller has cleared; set non-zero if a
 *            time-limited wait inside the kernel gave up
 * The tensor core truncates when it adds into its fp32 accumulator (measured
 * bias 7e-9 * chain length, relative), so the reduction is dealt round-robin to
 * up to 15 accumulators in tensor memory that are added at the end in fp32.
 * ------------------------------------------------------------------------ */
db_status db_contract_f32(const float* A, int64_t a_row, int64_t a_k,
                          const float* B, int64_t b_row, int64_t b_k,
                          float* out, int64_t o_m, int64_t o_n, int32_t M,
                          int32_t N, int32_t K, int32_t* status,
                          void* cuda_stream);

/* ------------------------------------------------------------------------
 * Proportional batch-size controller, host side   (Section 3.3, Eq. 4-5)
 *
 * One adjustment from per-worker throughputs X_k (samples per unit time):
 *     t_k = b_k / X_k;  tbar = mean_k t_k;  Db_k = -X_k (t_k - tbar)   (Eq. 4)
 *     bt_k = b_k + kp * Db_k                                           (Eq. 5)
 * kp = 1 is the paper's rule (equivalently b_k * tbar / t_k); kp in (0,1)
 * damps it.  The targets are rescaled so that the global batch sum_k b_k is
 * unchanged (the invariant Section 3.2 states for variable batching), then
 * made integer within [b_min_k, b_max_k] (bounds: Section 3.3.1) by the
 * largest-remainder rule: start from floor, hand missing units to the worker
 * furthest below its target (ties: lowest index), take surplus units from
 * the worker furthest above.  All arithmetic is IEEE fp64 in a fixed order,
 * so the integer result is deterministic.
 *
 *   b            host, K batch sizes >= 0 with sum > 0; overwritten on DB_OK
 *   throughputs  host, K finite values > 0
 *   K            1..DB_MAX_K
 *   kp           0 < kp <= 1
 *   b_min,b_max  host, K each, or NULL for 1 and sum(b); 0 <= min <= max
 * DB_ERR_INFEASIBLE (b untouched) if the bounds cannot sum to sum(b).
 * ------------------------------------------------------------------------ */
db_status db_controller_step(int32_t* b, const double* throughputs, int32_t K,
                             double kp);

db_status db_controller_step_ex(int32_t* b, const double* throughputs,
                                int32_t K, double kp, const int32_t* b_min,
                                const int32_t* b_max);

/* ------------------------------------------------------------------------
 * Static open-loop allocation                               (Section 3.2)
 *
 * b_k proportional to the throughput estimate X_k with the global batch K*b0
 * kept: b_k = K * b0 * X_k / sum X (the printed b0 * X_k / sum X sums to b0,
 * not to the K*b0 the text requires), made integer within the bounds by the
 * same largest-remainder rule as the controller.
 *   throughputs host, K finite values > 0 (e.g. core counts or FLOPs)
 *   b0          the uniform per-worker batch it replaces, >= 1
 *   b_min,b_max host, K each, or NULL for 1 and K*b0
 *   b           host, K, written on DB_OK
 * ------------------------------------------------------------------------ */
db_status db_static_allocate(const double* throughputs, int32_t K, int32_t b0,
                             const int32_t* b_min, const int32_t* b_max,
                             int32_t* b);

/* ------------------------------------------------------------------------
 * Stabilised controller, host side        (Section 3.3.1, the 4-step listing)
 *
 * A controller object keeps the current batch sizes and, per observation of
 * the workers' iteration times t_k (any unit, > 0):
 *   1. smooths them with an EWMA over the iterations since the last
 *      readjustment, mu_k <- alpha t_k + (1 - alpha) mu_k (the first sample
 *      after a readjustment initialises mu_k; the paper gives no alpha);
 *   2. applies db_controller_step_ex with X_k = b_k / mu_k and gain kp;
 *   3. within [b_min, b_max]; with adaptive_b_max != 0 the upper bound also
 *      learns: when a worker whose batch was raised at the previous
 *      readjustment (from b0 to b) now shows a lower smoothed throughput than
 *      it had then, its upper bound becomes b0.  If the learnt bounds cannot
 *      hold the global batch, the user's bounds alone are used for that step;
 *   4. dead-band: the new sizes are adopted for all workers only if
 *      max_k |b'_k - b_k| / b_k > dead_band (the paper uses 0.05), else none.
 *
 *   b0          host, K initial batch sizes >= 1
 *   kp          0 < kp <= 1;  alpha 0 < alpha <= 1;  dead_band >= 0
 *   b_min,b_max host, K each, or NULL for 1 and sum(b0); b_min[k] >= 1 (a
 *               worker at batch 0 would have no iteration time to observe)
 *               and b_max[k] >= b_min[k], else DB_ERR_ARG
 * db_controller_observe: b_out (host, K, nullable) receives the batch sizes in
 * force after the observation, *changed (nullable) whether they moved.
 * Not thread-safe per object.  All arithmetic is IEEE fp64 in a fixed order.
 * ------------------------------------------------------------------------ */
typedef struct db_controller db_controller;

db_status db_controller_create(db_controller** out, const int32_t* b0,
                               int32_t K, double kp, double alpha,
                               double dead_band, const int32_t* b_min,
                               const int32_t* b_max, int32_t adaptive_b_max);
db_status db_controller_observe(db_controller* controller,
                                const double* iteration_times, int32_t* b_out,
                                int32_t* changed);
db_status db_controller_destroy(db_controller* controller);

/* Static text for a status code. */
const char* db_status_string(db_status s);

/* Message of the last CUDA error seen by this thread ("" if none). */
const char* db_last_cuda_error(void);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif

#ifdef __cplusplus
}
#endif
#endif /* DYNBATCH_H_ */
