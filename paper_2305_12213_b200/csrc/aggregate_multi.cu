// The fused aggregation + momentum step over a LIST of parameter tensors that do not share one arena
// (Section 3.1, Eq. 2-3; the 161 tensors of a ResNet-50 or the 199 of a BERT-base as the framework
// allocated them).  A plan, built once for a fixed set of tensors, holds in device memory one record
// per CTA: the CTA's tile of one tensor with every pointer it needs (params, momentum, the K gradient
// slices) already advanced to the tile.  Every step is then a single launch in which a CTA reads its
// record -- one round trip to memory, all of its loads independent -- and processes the tile exactly
// like the flat kernel: same order of fused multiply-adds, so results are bit-identical to it.
#include <cstdint>
#include <new>
#include <vector>

#include "agg_device.cuh"
#include "common.h"

namespace dynbatch {
namespace {

using agg::GradVec;
using agg::kBlock;
using agg::kChunk;

// Record of one CTA, 8 * (3 + K) bytes: p, v, {count, vec_ok}, then the K gradient pointers.
//   count   elements of the tile (at most kBlock * UNROLL vectors' worth)
//   vec_ok  all K + 2 pointers are 16-byte aligned: 128-bit path
constexpr int kRecHeader = 3;

struct MultiArgs {
    const long long* recs;     // records, stride kRecHeader + K words of 8 bytes
    float lambda[DB_MAX_K];    // 0 for a worker with an empty batch: its buffers are not read
    double* partials;
    double* sq_out;
    float lr, mu;
    int K;
    int total_tiles;           // records; a CTA takes TILES consecutive ones
};

template <typename GT, bool NORM>
__device__ __forceinline__ void multi_scalar(const MultiArgs& a, float* p, float* v, const long long* gp,
                                             long long j, double& sq) {
    float acc = 0.0f;
    for (int k = 0; k < a.K; ++k)
        if (a.lambda[k] != 0.0f)
            acc = fmaf(a.lambda[k], GradVec<GT>::scalar(reinterpret_cast<const void*>(__ldg(gp + k)), j), acc);
    const float vn = fmaf(a.mu, v[j], acc);
    v[j] = vn;
    p[j] = fmaf(-a.lr, vn, p[j]);
    if (NORM) sq += static_cast<double>(acc * acc);
}

// One CTA = one tile of kBlock * UNROLL vectors (kLanes elements each) of one tensor.
// KU > 0: at most KU workers, their loads fully unrolled and all issued before the first use.
// KU == 0: any K, kChunk gradient slices per round.
// TILES > 1: the CTA takes that many consecutive records; it asks for the next record while it works
// on the current one, so only the first costs a round trip of its own.
template <typename GT, int KU, int UNROLL, int TILES, bool NORM>
__global__ void __launch_bounds__(kBlock)
agg_multi_kernel(const __grid_constant__ MultiArgs a) {
    using GV = GradVec<GT>;
    using Raw = typename GV::Raw;
    constexpr int kLanes = GV::kLanes;
    constexpr int kQuads = kLanes / 4;
    constexpr int kSlots = KU > 0 ? KU : kChunk;
    agg::griddep_launch_dependents();
    agg::griddep_wait();
    const int K = a.K;
    double sq = 0.0;
#pragma unroll 1
    for (int t = 0; t < TILES; ++t) {
    const long long tile_id = static_cast<long long>(blockIdx.x) * TILES + t;
    if (tile_id >= a.total_tiles) break;
    const long long* rec = a.recs + tile_id * (kRecHeader + K);
    if (TILES > 1 && t + 1 < TILES && tile_id + 1 < a.total_tiles) {
        const char* next = reinterpret_cast<const char*>(rec + kRecHeader + K);
        if (threadIdx.x * 32 < 8 * (kRecHeader + K))
            asm volatile("prefetch.global.L1 [%0];" ::"l"(next + threadIdx.x * 32));
    }
    float* p = reinterpret_cast<float*>(__ldg(rec + 0));
    float* v = reinterpret_cast<float*>(__ldg(rec + 1));
    const long long cf = __ldg(rec + 2);
    const int count = static_cast<int>(cf & 0xffffffffLL);
    const bool vec_ok = (cf >> 32) != 0;
    const long long* gp = rec + kRecHeader;

    if (vec_ok) {
        const int full = count / kLanes;                 // whole vectors of the tile
        float4 pv[UNROLL][kQuads], vv[UNROLL][kQuads];
        float acc[UNROLL][kLanes];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            live[u] = threadIdx.x + u * kBlock < full;
#pragma unroll
            for (int l = 0; l < kLanes; ++l) acc[u][l] = 0.0f;
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (!live[u]) continue;
            const long long vi = threadIdx.x + u * kBlock;
#pragma unroll
            for (int q = 0; q < kQuads; ++q) {
                pv[u][q] = __ldcs(reinterpret_cast<const float4*>(p) + vi * kQuads + q);
                vv[u][q] = __ldcs(reinterpret_cast<const float4*>(v) + vi * kQuads + q);
            }
        }
        for (int k0 = 0; k0 < K; k0 += kSlots) {
            const void* g[kSlots];
            float lam[kSlots];
#pragma unroll
            for (int i = 0; i < kSlots; ++i) {
                const bool in = k0 + i < K;
                lam[i] = in ? a.lambda[k0 + i] : 0.0f;
                g[i] = in ? reinterpret_cast<const void*>(__ldg(gp + k0 + i)) : nullptr;
            }
            Raw raw[UNROLL][kSlots];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!live[u]) continue;
#pragma unroll
                for (int i = 0; i < kSlots; ++i)
                    if (lam[i] != 0.0f) raw[u][i] = GV::load(g[i], 0, threadIdx.x + u * kBlock);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!live[u]) continue;
#pragma unroll
                for (int i = 0; i < kSlots; ++i) {
                    if (lam[i] != 0.0f) {
                        float x[kLanes];
                        GV::widen(raw[u][i], x);
#pragma unroll
                        for (int l = 0; l < kLanes; ++l) acc[u][l] = fmaf(lam[i], x[l], acc[u][l]);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (!live[u]) continue;
            const long long vi = threadIdx.x + u * kBlock;
            float part = 0.0f;
#pragma unroll
            for (int q = 0; q < kQuads; ++q) {
                float4 vn, pn;
                vn.x = fmaf(a.mu, vv[u][q].x, acc[u][4 * q + 0]);
                vn.y = fmaf(a.mu, vv[u][q].y, acc[u][4 * q + 1]);
                vn.z = fmaf(a.mu, vv[u][q].z, acc[u][4 * q + 2]);
                vn.w = fmaf(a.mu, vv[u][q].w, acc[u][4 * q + 3]);
                pn.x = fmaf(-a.lr, vn.x, pv[u][q].x);
                pn.y = fmaf(-a.lr, vn.y, pv[u][q].y);
                pn.z = fmaf(-a.lr, vn.z, pv[u][q].z);
                pn.w = fmaf(-a.lr, vn.w, pv[u][q].w);
                __stcs(reinterpret_cast<float4*>(v) + vi * kQuads + q, vn);
                __stcs(reinterpret_cast<float4*>(p) + vi * kQuads + q, pn);
                if (NORM) {
#pragma unroll
                    for (int l = 0; l < 4; ++l) part = fmaf(acc[u][4 * q + l], acc[u][4 * q + l], part);
                }
            }
            if (NORM) sq += static_cast<double>(part);
        }
        // the tensor's last, partial vector (fewer than kLanes elements) lives in its last tile
        const int tail0 = full * kLanes;
        if (tail0 + static_cast<int>(threadIdx.x) < count)
            multi_scalar<GT, NORM>(a, p, v, gp, tail0 + threadIdx.x, sq);
    } else {
        // buffers off the 16-byte grid: element by element
#pragma unroll 1
        for (int j = threadIdx.x; j < count; j += kBlock) multi_scalar<GT, NORM>(a, p, v, gp, j, sq);
    }
    }   // tiles of this CTA
    if (NORM) agg::store_norm_partial(a.partials, sq);
}

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Launch shape by worker count, as for the flat kernel: up to 8 workers two vectors per thread with
// every load in flight at once, up to 16 one vector, beyond that kChunk slices per round.
int unroll_for(int K) { return K <= 8 ? 2 : 1; }
// measured (BERT-base shapes, K = 16, bf16): 1 record per CTA 826 us, 2: 797, 4: 1050; K = 8 (ResNet-50): 1: 182.1, 2: 184.4
int tiles_per_cta(int K) { return K > 8 && K <= 16 ? 2 : 1; }

// Tiles of one tensor: kBlock * unroll vectors of `lanes` elements each.
long long tile_elems(int lanes, int unroll) { return static_cast<long long>(kBlock) * unroll * lanes; }
long long tiles_of(long long n, long long per) { return (n + per - 1) / per; }

struct PlanLayout {
    long long total_tiles;
    size_t partials_off, recs_off, end;
};

bool plan_layout(int32_t K, int32_t T, const int64_t* sizes, db_dtype dt, PlanLayout* L) {
    const long long per = tile_elems(dt == DB_F32 ? 4 : 8, unroll_for(K));
    long long tiles = 0;
    for (int t = 0; t < T; ++t) {
        if (sizes[t] < 0) return false;
        tiles += tiles_of(sizes[t], per);
    }
    if (tiles > 0x7fffffffLL) return false;
    L->total_tiles = tiles;
    L->partials_off = 0;
    L->recs_off = L->partials_off + round256(sizeof(double) * static_cast<size_t>(tiles > 0 ? tiles : 1));
    L->end = L->recs_off + round256(8 * static_cast<size_t>(kRecHeader + K) * static_cast<size_t>(tiles > 0 ? tiles : 1));
    return true;
}

using MultiFn = void (*)(const MultiArgs);

template <typename GT, bool NORM>
MultiFn pick_multi(int K) {
    if (K <= 4) return agg_multi_kernel<GT, 4, 2, 1, NORM>;
    if (K <= 8) return agg_multi_kernel<GT, 8, 2, 1, NORM>;
    if (K <= 16) return agg_multi_kernel<GT, 16, 1, 2, NORM>;
    return agg_multi_kernel<GT, 0, 1, 1, NORM>;
}

}  // namespace
}  // namespace dynbatch

struct db_multi_plan {
    dynbatch::MultiArgs args{};
    db_dtype dtype = DB_F32;
    int32_t K = 0;
    long long total_tiles = 0;
};

extern "C" size_t db_multi_plan_device_bytes(int32_t K, db_dtype grad_dtype, const int64_t* sizes, int32_t T) {
    using namespace dynbatch;
    if (!sizes || K < 1 || K > DB_MAX_K || T < 1 || (grad_dtype != DB_F32 && grad_dtype != DB_BF16)) return 0;
    PlanLayout L;
    if (!plan_layout(K, T, sizes, grad_dtype, &L)) return 0;
    return L.end;
}

extern "C" db_status db_multi_plan_destroy(db_multi_plan* plan) {
    delete plan;
    return DB_OK;
}

extern "C" db_status db_multi_plan_create(db_multi_plan** out, const void* const* grads, db_dtype grad_dtype,
                                          int32_t K, const int64_t* sizes, int32_t T, float* const* params,
                                          float* const* momentum, void* device_table, size_t device_table_bytes,
                                          void* cuda_stream) {
    using namespace dynbatch;
    if (!out) return DB_ERR_NULL;
    *out = nullptr;
    if (!grads || !sizes || !params || !momentum || !device_table) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || T < 1) return DB_ERR_ARG;
    if (grad_dtype != DB_F32 && grad_dtype != DB_BF16) return DB_ERR_UNSUPPORTED;
    PlanLayout L;
    if (!plan_layout(K, T, sizes, grad_dtype, &L)) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(device_table) % 256 || device_table_bytes < L.end) return DB_ERR_ARG;
    const int lanes = grad_dtype == DB_F32 ? 4 : 8;
    const size_t gsize = grad_dtype == DB_F32 ? 4 : 2;
    const long long per = tile_elems(lanes, unroll_for(K));
    const size_t words = static_cast<size_t>(kRecHeader + K);

    std::vector<long long> recs(words * static_cast<size_t>(L.total_tiles));
    size_t next = 0;
    for (int t = 0; t < T; ++t) {
        const long long n = sizes[t];
        if (n > 0 && (!params[t] || !momentum[t])) return DB_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(params[t]) % 4 || reinterpret_cast<uintptr_t>(momentum[t]) % 4) return DB_ERR_ARG;
        bool vec = reinterpret_cast<uintptr_t>(params[t]) % 16 == 0 && reinterpret_cast<uintptr_t>(momentum[t]) % 16 == 0;
        for (int k = 0; k < K; ++k) {
            const void* g = grads[static_cast<size_t>(k) * T + t];
            if (n > 0 && !g) return DB_ERR_NULL;
            if (reinterpret_cast<uintptr_t>(g) % gsize) return DB_ERR_ARG;
            vec = vec && reinterpret_cast<uintptr_t>(g) % 16 == 0;
        }
        // a tile starts a whole number of 16-byte vectors into the tensor, so alignment carries over
        for (long long e0 = 0; e0 < n; e0 += per) {
            long long* r = recs.data() + words * next++;
            const long long count = n - e0 < per ? n - e0 : per;
            r[0] = static_cast<long long>(reinterpret_cast<uintptr_t>(params[t] + e0));
            r[1] = static_cast<long long>(reinterpret_cast<uintptr_t>(momentum[t] + e0));
            r[2] = count | (static_cast<long long>(vec ? 1 : 0) << 32);
            for (int k = 0; k < K; ++k)
                r[kRecHeader + k] = static_cast<long long>(
                    reinterpret_cast<uintptr_t>(static_cast<const char*>(grads[static_cast<size_t>(k) * T + t]) + e0 * gsize));
        }
    }

    db_multi_plan* plan = new (std::nothrow) db_multi_plan();
    if (!plan) return DB_ERR_ARG;
    char* base = static_cast<char*>(device_table);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t err = cudaSuccess;
    if (!recs.empty())
        err = cudaMemcpyAsync(base + L.recs_off, recs.data(), sizeof(long long) * recs.size(), cudaMemcpyHostToDevice,
                              stream);
    // the host vector goes away when this function returns: wait for the copy (plan creation is not on the hot path)
    if (err == cudaSuccess) err = cudaStreamSynchronize(stream);
    if (err != cudaSuccess) {
        delete plan;
        return record_cuda_error(err, "db_multi_plan_create");
    }
    plan->dtype = grad_dtype;
    plan->K = K;
    plan->total_tiles = L.total_tiles;
    plan->args.recs = reinterpret_cast<const long long*>(base + L.recs_off);
    plan->args.partials = reinterpret_cast<double*>(base + L.partials_off);
    plan->args.K = K;
    *out = plan;
    return DB_OK;
}

extern "C" db_status db_aggregate_update_multi(db_multi_plan* plan, const int32_t* b, float lr, float mu,
                                               double* grad_sqnorm, void* cuda_stream) {
    using namespace dynbatch;
    if (!plan || !b) return DB_ERR_NULL;
    if (!isfinite(lr) || !isfinite(mu)) return DB_ERR_ARG;
    long long total = 0;
    for (int k = 0; k < plan->K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        total += b[k];
    }
    if (total <= 0) return DB_ERR_ARG;
    if (plan->total_tiles == 0) return DB_OK;
    MultiArgs a = plan->args;
    for (int k = 0; k < plan->K; ++k)
        a.lambda[k] = static_cast<float>(static_cast<double>(b[k]) / static_cast<double>(total));
    a.lr = lr;
    a.mu = mu;
    a.sq_out = grad_sqnorm;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool norm = grad_sqnorm != nullptr;
    MultiFn fn;
    if (plan->dtype == DB_F32) fn = norm ? pick_multi<float, true>(plan->K) : pick_multi<float, false>(plan->K);
    else fn = norm ? pick_multi<__nv_bfloat16, true>(plan->K) : pick_multi<__nv_bfloat16, false>(plan->K);
    // may be scheduled while its predecessor in the stream still runs (it waits before its first access)
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1]{};
    const int per_cta = tiles_per_cta(plan->K);
    const long long ctas = (plan->total_tiles + per_cta - 1) / per_cta;
    a.total_tiles = static_cast<int>(plan->total_tiles);
    cfg.gridDim = dim3(static_cast<unsigned int>(ctas));
    cfg.blockDim = dim3(kBlock);
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    DB_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, a));
    DB_CUDA_TRY(cudaGetLastError());
    if (norm) DB_CUDA_TRY(agg::launch_norm_finalize(a.partials, ctas, a.sq_out, stream, true));
    return DB_OK;
}
