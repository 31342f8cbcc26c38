// Fused K-way weighted gradient aggregation + momentum-SGD update
// (Section 3.1, Eq. 2-3; momentum optimizer of Section 4's ResNet-50 workload).
//
// One pass over HBM: each thread owns one 16-byte vector position per step,
// issues the loads of all K gradient slices and of the parameter/momentum
// vectors before the first use, folds the slices with fp32 FMAs in worker
// order, applies v = mu v + g, p = p - lr v and streams both back.  Nothing
// else touches N-sized data; the squared gradient norm rides along in
// registers.  A CTA handles one to four consecutive tiles of 256 x UNROLL vectors and
// exits: the hardware hands out CTAs in index order as others retire, so the SMs
// stay inside one narrow moving window of each stream and their load and store
// phases are staggered.  Measured on B200 this beats a persistent grid-stride grid
// of SMs x occupancy CTAs by 2-14 % (K = 16 .. 2), whose CTAs move in lock step.
#include <cuda_bf16.h>

#include <cmath>
#include <cstdint>
#include <cstdio>

#include "agg_device.cuh"
#include "agg_kernels.cuh"
#include "common.h"

namespace dynbatch {
namespace {

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
using KernelFn = void (*)(const AggArgs);

template <typename GT, int KT, bool NORM, int OPT>
KernelFn pick_unroll(int* vectors_per_cta, int* block) {
    // Launch shapes measured on B200 (with the norm), fp32 and bf16 gradients:
    //   up to 8 workers   256 threads, two vector positions per thread, one tile per CTA
    //                     (2 (K + 2) independent 16-byte loads in flight per thread);
    //   9 to 16 workers   128 threads, two positions, two consecutive tiles per CTA: the smaller CTA
    //                     keeps two resident per SM despite ~40 loads per thread, and the second tile
    //                     amortises the norm epilogue (bf16, K = 16: 6.9 TB/s against 6.3-6.6 for
    //                     every 256-thread shape); Adam, with a third state stream, does better with 256
    //                     threads and one position (BERT-base shapes, K = 16, bf16: 872 against 886 us;
    //                     one tile per CTA 908, four 895);
    //   more workers      the chunked kernel, 256 threads, one position, one tile (more tiles per CTA
    //                     cost it 30 %).
    constexpr int kThreads = (KT >= 9 && OPT != kAdam) ? 128 : kBlock;
    constexpr int kUnroll = (KT >= 1 && !(KT >= 9 && OPT == kAdam)) ? 2 : 1;
    constexpr int kTiles = (KT >= 9) ? 2 : 1;
    *vectors_per_cta = kThreads * kUnroll * kTiles;
    *block = kThreads;
    return agg_vec_kernel<GT, KT, kThreads, kUnroll, kTiles, NORM, OPT>;
}

template <typename GT, bool NORM, int OPT>
KernelFn pick_vec_kernel(int K, int* unroll_out, int* block) {
    switch (K) {
#define DB_CASE(n) case n: return pick_unroll<GT, n, NORM, OPT>(unroll_out, block);
        DB_CASE(1) DB_CASE(2) DB_CASE(3) DB_CASE(4) DB_CASE(5) DB_CASE(6) DB_CASE(7) DB_CASE(8)
        DB_CASE(9) DB_CASE(10) DB_CASE(11) DB_CASE(12) DB_CASE(13) DB_CASE(14) DB_CASE(15) DB_CASE(16)
#undef DB_CASE
        default: return pick_unroll<GT, 0, NORM, OPT>(unroll_out, block);
    }
}

bool ranges_overlap(const void* a, size_t abytes, const void* b, size_t bbytes) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

// CTAs any launch of this file can use for N elements: one per 256 vectors of 4 elements (the
// smallest tile), plus one for a ragged last tile and one so that the bound is never zero.
long long cta_bound(long long n) { return (n + 1023) / 1024 + 2; }

// Resident CTAs of the element-wise kernel (grid-stride), capped by the workspace bound.
int scalar_grid(KernelFn fn, long long n) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kBlock, 0) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    long long g = static_cast<long long>(sm_count()) * per_sm;
    const long long need = (n + kBlock - 1) / kBlock;
    if (g > need) g = need;
    if (g > cta_bound(n)) g = cta_bound(n);
    return static_cast<int>(g < 1 ? 1 : g);
}

}  // namespace
}  // namespace dynbatch

extern "C" size_t db_aggregate_workspace_bytes(int32_t K, int64_t N) {
    (void)K;
    // one double per CTA
    return sizeof(double) * static_cast<size_t>(dynbatch::cta_bound(N < 0 ? 0 : N));
}

namespace dynbatch {
namespace {

template <int OPT>
KernelFn pick_kernel(bool vector_ok, db_dtype dt, bool norm, int active, int* vectors_per_cta, int* block) {
    *block = kBlock;
    if (vector_ok) {
        if (dt == DB_F32)
            return norm ? pick_vec_kernel<float, true, OPT>(active, vectors_per_cta, block)
                        : pick_vec_kernel<float, false, OPT>(active, vectors_per_cta, block);
        return norm ? pick_vec_kernel<__nv_bfloat16, true, OPT>(active, vectors_per_cta, block)
                    : pick_vec_kernel<__nv_bfloat16, false, OPT>(active, vectors_per_cta, block);
    }
    if (dt == DB_F32) return norm ? agg_scalar_kernel<float, true, OPT> : agg_scalar_kernel<float, false, OPT>;
    return norm ? agg_scalar_kernel<__nv_bfloat16, true, OPT> : agg_scalar_kernel<__nv_bfloat16, false, OPT>;
}

// Validation, weights, alignment analysis and launch shared by the momentum and Adam entry points.
// `a` arrives with the optimizer's scalars set; `second` is Adam's second-moment buffer (else NULL).
db_status aggregate_launch(AggArgs a, int opt, const void* const* grads, db_dtype grad_dtype, const int32_t* b,
                           int32_t K, int64_t N, float* params, float* first, float* second,
                           double* grad_sqnorm, void* workspace, size_t workspace_bytes, void* cuda_stream,
                           double* chunk_partials = nullptr, long long* chunk_ctas = nullptr) {
    if (!grads || !b) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || N < 0) return DB_ERR_ARG;
    if (grad_dtype != DB_F32 && grad_dtype != DB_BF16) return DB_ERR_UNSUPPORTED;
    long long total = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        total += b[k];
    }
    if (total <= 0) return DB_ERR_ARG;
    if (N == 0) return DB_OK;
    float* state[3] = {params, first, second};
    const int n_state = opt == kAdam ? 3 : 2;
    const size_t gsize = grad_dtype == DB_F32 ? 4 : 2;
    const size_t state_bytes = static_cast<size_t>(N) * 4, grad_bytes = static_cast<size_t>(N) * gsize;
    for (int i = 0; i < n_state; ++i) {
        if (!state[i]) return DB_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(state[i]) % 4) return DB_ERR_ARG;
        for (int j = 0; j < i; ++j)
            if (ranges_overlap(state[i], state_bytes, state[j], state_bytes)) return DB_ERR_ARG;
    }

    int active = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] == 0) continue;  // weight 0: the buffer is not read
        if (!grads[k]) return DB_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(grads[k]) % gsize) return DB_ERR_ARG;
        for (int i = 0; i < n_state; ++i)
            if (ranges_overlap(grads[k], grad_bytes, state[i], state_bytes)) return DB_ERR_ARG;
        a.g[active] = grads[k];
        a.lambda[active] = static_cast<float>(static_cast<double>(b[k]) / static_cast<double>(total));
        ++active;
    }
    a.K = active;
    a.p = params;
    a.v = first;
    a.u = second;
    a.n = N;

    // chunk mode (the host pipeline): only the partial sums are produced, at a place the caller chose
    const bool norm = grad_sqnorm != nullptr || chunk_partials != nullptr;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (chunk_partials) {
        a.partials = chunk_partials;
    } else if (norm) {
        if (!workspace) return DB_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(workspace) % 16 || workspace_bytes < db_aggregate_workspace_bytes(K, N))
            return DB_ERR_ARG;
        a.partials = static_cast<double*>(workspace);
        a.sq_out = grad_sqnorm;
    }

    // Leading elements until params reaches a 16-byte boundary; the vector body needs the other
    // state buffers and every gradient buffer on a boundary at the same element.
    const int lanes = grad_dtype == DB_F32 ? 4 : 8;
    long long head = static_cast<long long>(((16 - reinterpret_cast<uintptr_t>(params) % 16) % 16) / 4);
    bool vector_ok = true;
    for (int i = 1; i < n_state; ++i)
        vector_ok = vector_ok && (reinterpret_cast<uintptr_t>(state[i]) + head * 4) % 16 == 0;
    if (vector_ok && grad_dtype == DB_BF16) {
        // bf16 vectors hold 8 elements: pick the head in {head, head + 4} that aligns the gradients
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(a.g[0]);
        if ((g0 + head * 2) % 16 != 0) head += 4;
    }
    for (int k = 0; vector_ok && k < active; ++k)
        vector_ok = (reinterpret_cast<uintptr_t>(a.g[k]) + head * gsize) % 16 == 0;
    if (head > N) head = N;
    a.head = head;
    a.nvec = (N - head) / lanes;

    int vectors_per_cta = kBlock, block = kBlock;
    const KernelFn fn = opt == kAdam
                            ? pick_kernel<kAdam>(vector_ok, grad_dtype, norm, active, &vectors_per_cta, &block)
                            : pick_kernel<kMomentum>(vector_ok, grad_dtype, norm, active, &vectors_per_cta, &block);
    int grid;
    if (vector_ok) {
        const long long tiles = (a.nvec + vectors_per_cta - 1) / vectors_per_cta;
        if (tiles > 0x7fffffffLL) return DB_ERR_ARG;
        grid = static_cast<int>(tiles < 1 ? 1 : tiles);
        // Grids of at most one wave (what an SM's 2048 threads hold of this CTA size, on every SM) of a launch
        // that may be scheduled under its predecessor: every CTA asks the L2 for its state vectors before it
        // waits.  Measured on B200, steps back to back: 7.7 -> 6.8 us for N = 2^20, K = 3; 49.9 -> 44.0 us for
        // N = 2^22, K = 16; 44.7 -> 42.5 us for the 2,048,000-parameter step behind the worker-gradient kernels.
        // Larger grids lose: at 1.7 waves (N = 2^22, K = 2) 18.4 -> 19.1 us, and on the large workloads even the
        // first wave alone doing so costs 3 % (ResNet-50 shapes 173.1 -> 178.8 us, BERT-base 738 -> 772 us): its
        // CTAs then start their gradient loads in lock step.
        const int first_wave = sm_count() * (2048 / block);
        if (!chunk_partials && !chunk_ctas && active <= 16 && grid <= first_wave) a.prefetch_ctas = grid;
    } else {
        grid = scalar_grid(fn, N);
    }
    // A whole-array step may be scheduled while its predecessor in the stream (typically the previous
    // step's norm fold) still runs; the kernel waits for it before its first access.  The chunks of the
    // host pipeline are ordered by events across streams and take ordinary launches.
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1]{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (chunk_partials || chunk_ctas) ? 0 : 1;
    DB_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, a));
    DB_CUDA_TRY(cudaGetLastError());
    if (chunk_ctas) *chunk_ctas = grid;
    if (norm && !chunk_partials) DB_CUDA_TRY(agg::launch_norm_finalize(a.partials, grid, a.sq_out, stream, true));
    return DB_OK;
}

}  // namespace

long long aggregate_cta_bound(int64_t N) { return cta_bound(N < 0 ? 0 : N); }

db_status aggregate_chunk(const void* const* grads, db_dtype grad_dtype, const int32_t* b, int32_t K, int64_t N,
                          float* params, float* momentum, float lr, float mu, double* partials, long long* ctas,
                          void* cuda_stream) {
    if (ctas) *ctas = 0;
    AggArgs a{};
    a.lr = lr;
    a.mu = mu;
    return aggregate_launch(a, kMomentum, grads, grad_dtype, b, K, N, params, momentum, nullptr, nullptr, nullptr, 0,
                            cuda_stream, partials, ctas);
}

db_status finalize_norm(const double* partials, long long n, double* sq_out, cudaStream_t stream) {
    DB_CUDA_TRY(agg::launch_norm_finalize(partials, n, sq_out, stream, false));
    return DB_OK;
}

}  // namespace dynbatch

extern "C" db_status db_aggregate_update_ex(const void* const* grads, db_dtype grad_dtype,
                                            const int32_t* b, int32_t K, int64_t N,
                                            float* params, float* momentum, float lr, float mu,
                                            double* grad_sqnorm, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream) {
    using namespace dynbatch;
    if (!isfinite(lr) || !isfinite(mu)) return DB_ERR_ARG;
    AggArgs a{};
    a.lr = lr;
    a.mu = mu;
    return aggregate_launch(a, kMomentum, grads, grad_dtype, b, K, N, params, momentum, nullptr, grad_sqnorm,
                            workspace, workspace_bytes, cuda_stream);
}

extern "C" db_status db_aggregate_adam_ex(const void* const* grads, db_dtype grad_dtype, const int32_t* b,
                                          int32_t K, int64_t N, float* params, float* first_moment,
                                          float* second_moment, float lr, float beta1, float beta2, float eps,
                                          int64_t step, double* grad_sqnorm, void* workspace,
                                          size_t workspace_bytes, void* cuda_stream) {
    using namespace dynbatch;
    if (!isfinite(lr) || !isfinite(eps) || !(eps >= 0.0f)) return DB_ERR_ARG;
    if (!(beta1 >= 0.0f) || !(beta1 < 1.0f) || !(beta2 >= 0.0f) || !(beta2 < 1.0f) || step < 1) return DB_ERR_ARG;
    AggArgs a{};
    a.lr = lr;
    a.mu = beta1;
    a.beta2 = beta2;
    a.eps = eps;
    // bias corrections in fp64 on the host, once per call
    a.inv_c1 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta1), static_cast<double>(step))));
    a.inv_c2 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta2), static_cast<double>(step))));
    return aggregate_launch(a, kAdam, grads, grad_dtype, b, K, N, params, first_moment, second_moment,
                            grad_sqnorm, workspace, workspace_bytes, cuda_stream);
}

extern "C" db_status db_aggregate_update(const float* const* grads, const int32_t* b, int32_t K,
                                         int64_t N, float* params, float* momentum, float lr, float mu) {
    return db_aggregate_update_ex(reinterpret_cast<const void* const*>(grads), DB_F32, b, K, N, params,
                                  momentum, lr, mu, nullptr, nullptr, 0, nullptr);
}

// ---------------------------------------------------------------------------
// Variant with library-owned scratch, for callers that cannot allocate.
// ---------------------------------------------------------------------------
namespace dynbatch {
namespace {

// Per-CTA partials of the norm.  Lives in every device's global memory
// for the life of the process.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is never passed to a kernel as a pointer.
static __device__ __align__(256) unsigned char g_static_scratch[DB_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, looked up once per device.
db_status static_scratch_address(void** out) {
    constexpr int kMaxDev = 64;
    static void* cache[kMaxDev] = {nullptr};
    int dev = 0;
    DB_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return DB_ERR_UNSUPPORTED;
    void* ptr = __atomic_load_n(&cache[dev], __ATOMIC_ACQUIRE);
    if (!ptr) {
        DB_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return DB_ERR_CUDA;
        __atomic_store_n(&cache[dev], ptr, __ATOMIC_RELEASE);  // every thread stores the same address
    }
    *out = ptr;
    return DB_OK;
}

}  // namespace
}  // namespace dynbatch

extern "C" db_status db_aggregate_update_static(const void* const* grads, db_dtype grad_dtype,
                                                const int32_t* b, int32_t K, int64_t N, float* params,
                                                float* momentum, float lr, float mu,
                                                double* grad_sqnorm, void* cuda_stream) {
    using namespace dynbatch;
    // the cheap argument checks first, so that a bad call is reported as what it is, not as too large
    if (!grads || !b || !params || !momentum) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || N < 0) return DB_ERR_ARG;
    if (grad_dtype != DB_F32 && grad_dtype != DB_BF16) return DB_ERR_UNSUPPORTED;
    long long total = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        total += b[k];
    }
    if (total <= 0 || !isfinite(lr) || !isfinite(mu)) return DB_ERR_ARG;
    void* scratch = nullptr;
    if (grad_sqnorm && N > 0) {
        const size_t need = db_aggregate_workspace_bytes(K, N);
        if (need > DB_STATIC_SCRATCH_BYTES) {
            char msg[256];
            snprintf(msg, sizeof msg,
                     "db_aggregate_update_static: this device needs %zu bytes of scratch, the built-in "
                     "array holds %d; use db_aggregate_update_ex with a workspace",
                     need, DB_STATIC_SCRATCH_BYTES);
            record_message(msg);
            return DB_ERR_UNSUPPORTED;
        }
        const db_status st = static_scratch_address(&scratch);
        if (st != DB_OK) return st;
    }
    return db_aggregate_update_ex(grads, grad_dtype, b, K, N, params, momentum, lr, mu, grad_sqnorm,
                                  scratch, scratch ? DB_STATIC_SCRATCH_BYTES : 0, cuda_stream);
}
