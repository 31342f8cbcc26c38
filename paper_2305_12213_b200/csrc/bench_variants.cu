// Measurement helpers: a read-only bandwidth probe, and the aggregation step (Section 3.1, Eq. 2-3 with
// the momentum update) in the two launch / staging shapes that were measured against the kept kernel of
// aggregate.cu and not adopted.  Same per-element arithmetic as the kept kernel -- a zero accumulator,
// fmaf in worker order, v = fma(mu, v, g), p = fma(-lr, v, p) -- so the results are bit-identical and only
// the way the bytes move differs.
#include <cmath>
#include <cstdint>

#include "agg_device.cuh"
#include "common.h"
#include "dynbatch_bench.h"
#include "tc_gemm.cuh"

namespace dynbatch {
namespace {

using agg::kBlock;

// ---------------------------------------------------------------------------------------------
// read probe
// ---------------------------------------------------------------------------------------------
constexpr int kProbeVecPerThread = 8;                                   // independent 16-byte loads in flight
constexpr long long kProbeVecPerCta = static_cast<long long>(kBlock) * kProbeVecPerThread;   // 32 KB per CTA

__global__ void __launch_bounds__(kBlock) read_probe_kernel(const uint4* __restrict__ src, long long nvec,
                                                            unsigned long long* __restrict__ sink) {
    const long long base = static_cast<long long>(blockIdx.x) * kProbeVecPerCta + threadIdx.x;
    uint4 r[kProbeVecPerThread];
#pragma unroll
    for (int u = 0; u < kProbeVecPerThread; ++u) {
        const long long i = base + static_cast<long long>(u) * kBlock;
        r[u] = i < nvec ? __ldcs(src + i) : make_uint4(0u, 0u, 0u, 0u);
    }
    unsigned int x = 0;
#pragma unroll
    for (int u = 0; u < kProbeVecPerThread; ++u) x ^= r[u].x ^ r[u].y ^ r[u].z ^ r[u].w;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x ^= __shfl_xor_sync(0xffffffffu, x, off);
    __shared__ unsigned int warp_x[kBlock / 32];
    if ((threadIdx.x & 31) == 0) warp_x[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0;
        for (int w = 0; w < kBlock / 32; ++w) s = s * 31u + warp_x[w];
        sink[blockIdx.x] = s;
    }
}

long long probe_ctas(size_t bytes) {
    const long long nvec = static_cast<long long>(bytes / 16);
    const long long ctas = (nvec + kProbeVecPerCta - 1) / kProbeVecPerCta;
    return ctas < 1 ? 1 : ctas;
}

// ---------------------------------------------------------------------------------------------
// the step, other shapes
// ---------------------------------------------------------------------------------------------
constexpr int kMaxK = 16;

struct VariantArgs {
    const float* g[kMaxK];
    float lambda[kMaxK];
    float* p;
    float* v;
    long long nvec;     // float4 vectors
    float lr, mu;
    int* status;
};

template <int K>
__device__ __forceinline__ void combine(const VariantArgs& a, const float4 (&raw)[K], float4& pv, float4& vv) {
    float g[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int k = 0; k < K; ++k) {
        g[0] = fmaf(a.lambda[k], raw[k].x, g[0]);
        g[1] = fmaf(a.lambda[k], raw[k].y, g[1]);
        g[2] = fmaf(a.lambda[k], raw[k].z, g[2]);
        g[3] = fmaf(a.lambda[k], raw[k].w, g[3]);
    }
    vv.x = fmaf(a.mu, vv.x, g[0]); vv.y = fmaf(a.mu, vv.y, g[1]);
    vv.z = fmaf(a.mu, vv.z, g[2]); vv.w = fmaf(a.mu, vv.w, g[3]);
    pv.x = fmaf(-a.lr, vv.x, pv.x); pv.y = fmaf(-a.lr, vv.y, pv.y);
    pv.z = fmaf(-a.lr, vv.z, pv.z); pv.w = fmaf(-a.lr, vv.w, pv.w);
}

// Persistent grid: gridDim.x = SMs x resident CTAs, every CTA strides over the tiles of 256 x 2 vectors.
template <int K>
__global__ void __launch_bounds__(kBlock) persistent_kernel(const __grid_constant__ VariantArgs a) {
    agg::griddep_launch_dependents();
    agg::griddep_wait();
    constexpr int kUnroll = 2;
    const long long tile = static_cast<long long>(kBlock) * kUnroll;
    for (long long base = static_cast<long long>(blockIdx.x) * tile; base < a.nvec;
         base += static_cast<long long>(gridDim.x) * tile) {
        float4 raw[kUnroll][K], pv[kUnroll], vv[kUnroll];
        long long vi[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            vi[u] = base + u * kBlock + threadIdx.x;
            ok[u] = vi[u] < a.nvec;
            if (!ok[u]) continue;
#pragma unroll
            for (int k = 0; k < K; ++k) raw[u][k] = __ldcs(reinterpret_cast<const float4*>(a.g[k]) + vi[u]);
            pv[u] = __ldcs(reinterpret_cast<const float4*>(a.p) + vi[u]);
            vv[u] = __ldcs(reinterpret_cast<const float4*>(a.v) + vi[u]);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!ok[u]) continue;
            combine<K>(a, raw[u], pv[u], vv[u]);
            __stcs(reinterpret_cast<float4*>(a.v) + vi[u], vv[u]);
            __stcs(reinterpret_cast<float4*>(a.p) + vi[u], pv[u]);
        }
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

// Staged: one tile of TILE floats per stream and CTA.  K + 2 threads each start one cp.async.bulk into shared
// memory, all completing on one mbarrier; THREADS threads combine from shared memory, in place over the p
// and v tiles; two threads store those back with cp.async.bulk.
template <int K, int TILE, int THREADS>
__global__ void __launch_bounds__(THREADS) bulk_staged_kernel(const __grid_constant__ VariantArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int landed;
    float* s = reinterpret_cast<float*>(smem);                  // [K + 2][TILE]
    const long long e0 = static_cast<long long>(blockIdx.x) * TILE;
    const long long left = a.nvec * 4 - e0;
    const int count = static_cast<int>(left < TILE ? left : TILE);     // multiple of 4
    const uint32_t bytes = static_cast<uint32_t>(count) * 4u;
    if (threadIdx.x == 0) {
        landed = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    agg::griddep_launch_dependents();
    agg::griddep_wait();
    if (threadIdx.x == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     ::"r"(smem_u32(&bar)), "r"(bytes * (K + 2)) : "memory");
    __syncthreads();
    if (threadIdx.x < K + 2) {
        const float* src = threadIdx.x < K ? a.g[threadIdx.x] : (threadIdx.x == K ? a.p : a.v);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(s + threadIdx.x * TILE)), "l"(src + e0), "r"(bytes), "r"(smem_u32(&bar))
                     : "memory");
    }
    if (threadIdx.x == 0) {
        // the only wait of the kernel, bounded: on a time-out the CTA stores nothing and says so
        unsigned long long t0 = 0;
        int ok = 0;
        for (unsigned int spin = 0; !ok; ++spin) {
            uint32_t done;
            asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\t"
                         "selp.u32 %0, 1, 0, q;\n\t}" : "=r"(done) : "r"(smem_u32(&bar)) : "memory");
            ok = done != 0;
            if (!ok && (spin & 255u) == 255u) {
                unsigned long long now;
                asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) break;
            }
        }
        landed = ok;
        if (!ok && a.status) atomicExch(a.status, 1);
    }
    __syncthreads();
    if (!landed) return;
    for (int i = threadIdx.x * 4; i < count; i += THREADS * 4) {
        float4 raw[K];
#pragma unroll
        for (int k = 0; k < K; ++k) raw[k] = *reinterpret_cast<const float4*>(s + k * TILE + i);
        float4 pv = *reinterpret_cast<const float4*>(s + K * TILE + i);
        float4 vv = *reinterpret_cast<const float4*>(s + (K + 1) * TILE + i);
        combine<K>(a, raw, pv, vv);
        *reinterpret_cast<float4*>(s + K * TILE + i) = pv;
        *reinterpret_cast<float4*>(s + (K + 1) * TILE + i) = vv;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 2) {
        float* dst = threadIdx.x == 0 ? a.p : a.v;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"(dst + e0), "r"(smem_u32(s + (K + threadIdx.x) * TILE)), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
}

// One warp; lane 0 waits on a barrier that is never completed, with the kernels' own bounded wait.
__global__ void __launch_bounds__(32) wait_timeout_kernel(int* status, int code, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool completed = tc::mbar_wait(&bar, 0, &abort_flag, status, code, limit_ns);
        if (completed) atomicExch(status, -1);      // cannot happen: nothing arrives
    }
    __syncwarp();
}

using VariantFn = void (*)(const VariantArgs);

template <int K>
VariantFn pick_staged(int stage_floats, int* threads) {
    switch (stage_floats) {
        case 512: *threads = 128; return bulk_staged_kernel<K, 512, 128>;
        case 1024: *threads = 256; return bulk_staged_kernel<K, 1024, 256>;
        case 2048: *threads = 256; return bulk_staged_kernel<K, 2048, 256>;
        default: return nullptr;
    }
}

template <int K>
db_status launch_variant(db_bench_variant variant, int stage_floats, const VariantArgs& a, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1]{};
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.stream = stream;
    VariantFn fn = nullptr;
    if (variant == DB_BENCH_PERSISTENT) {
        fn = persistent_kernel<K>;
        int per_sm = 0;
        DB_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kBlock, 0));
        if (per_sm < 1) per_sm = 1;
        const long long tiles = (a.nvec + 2 * kBlock - 1) / (2 * kBlock);
        long long grid = static_cast<long long>(sm_count()) * per_sm;
        if (grid > tiles) grid = tiles;
        cfg.gridDim = dim3(static_cast<unsigned int>(grid));
        cfg.blockDim = dim3(kBlock);
    } else {
        int threads = 0;
        fn = pick_staged<K>(stage_floats, &threads);
        if (!fn) return DB_ERR_UNSUPPORTED;
        const size_t smem = static_cast<size_t>(K + 2) * stage_floats * sizeof(float);
        DB_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        const long long tiles = (a.nvec * 4 + stage_floats - 1) / stage_floats;
        if (tiles > 0x7fffffffLL) return DB_ERR_ARG;
        cfg.gridDim = dim3(static_cast<unsigned int>(tiles));
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = smem;
    }
    DB_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, a));
    DB_CUDA_TRY(cudaGetLastError());
    return DB_OK;
}

}  // namespace
}  // namespace dynbatch

extern "C" size_t db_bench_read_probe_sink_bytes(size_t bytes) {
    return sizeof(unsigned long long) * static_cast<size_t>(dynbatch::probe_ctas(bytes));
}

extern "C" db_status db_bench_read_probe(const void* src, size_t bytes, void* sink, void* cuda_stream) {
    using namespace dynbatch;
    if (!src || !sink) return DB_ERR_NULL;
    if (bytes == 0 || bytes % 16 || reinterpret_cast<uintptr_t>(src) % 16 || reinterpret_cast<uintptr_t>(sink) % 8)
        return DB_ERR_ARG;
    const long long ctas = probe_ctas(bytes);
    if (ctas > 0x7fffffffLL) return DB_ERR_ARG;
    read_probe_kernel<<<static_cast<unsigned int>(ctas), kBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint4*>(src), static_cast<long long>(bytes / 16), static_cast<unsigned long long*>(sink));
    DB_CUDA_TRY(cudaGetLastError());
    return DB_OK;
}

extern "C" db_status db_bench_wait_timeout(int32_t* status, int32_t code, uint64_t limit_ns, void* cuda_stream) {
    using namespace dynbatch;
    if (!status) return DB_ERR_NULL;
    if (code == 0 || limit_ns == 0 || limit_ns > tc::kWaitLimitNs || reinterpret_cast<uintptr_t>(status) % 4)
        return DB_ERR_ARG;
    wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status, code, limit_ns);
    DB_CUDA_TRY(cudaGetLastError());
    return DB_OK;
}

extern "C" db_status db_bench_aggregate_variant(db_bench_variant variant, int32_t stage_floats,
                                                const float* const* grads, const int32_t* b, int32_t K, int64_t N,
                                                float* params, float* momentum, float lr, float mu, int32_t* status,
                                                void* cuda_stream) {
    using namespace dynbatch;
    if (!grads || !b || !params || !momentum) return DB_ERR_NULL;
    if (variant != DB_BENCH_PERSISTENT && variant != DB_BENCH_BULK_STAGED) return DB_ERR_ARG;
    if (N < 0 || !std::isfinite(lr) || !std::isfinite(mu)) return DB_ERR_ARG;
    if (K != 2 && K != 4 && K != 8 && K != 16) return DB_ERR_UNSUPPORTED;
    if (N % 4 || reinterpret_cast<uintptr_t>(params) % 16 || reinterpret_cast<uintptr_t>(momentum) % 16)
        return DB_ERR_UNSUPPORTED;
    long long total = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        if (b[k] == 0) return DB_ERR_UNSUPPORTED;
        if (!grads[k]) return DB_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(grads[k]) % 16) return DB_ERR_UNSUPPORTED;
        total += b[k];
    }
    if (N == 0) return DB_OK;
    VariantArgs a{};
    for (int k = 0; k < K; ++k) {
        a.g[k] = grads[k];
        a.lambda[k] = static_cast<float>(static_cast<double>(b[k]) / static_cast<double>(total));
    }
    a.p = params;
    a.v = momentum;
    a.nvec = N / 4;
    a.lr = lr;
    a.mu = mu;
    a.status = status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    switch (K) {
        case 2: return launch_variant<2>(variant, stage_floats, a, stream);
        case 4: return launch_variant<4>(variant, stage_floats, a, stream);
        case 8: return launch_variant<8>(variant, stage_floats, a, stream);
        default: return launch_variant<16>(variant, stage_floats, a, stream);
    }
}
