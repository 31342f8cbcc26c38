// The fused aggregation + momentum step over a LIST of parameter tensors that do not share one arena
// (Section 3.1, Eq. 2-3; the 161 tensors of a ResNet-50 or the 199 of a BERT-base as the framework
// allocated them).  A plan, built once for a fixed set of tensors, holds in device memory one descriptor
// per tensor, the K x T gradient pointers and one record per CTA (tensor, tile within the tensor); every
// step is then a single launch in which a CTA looks up its record, its tensor and the K gradient
// pointers, and processes one tile of 256 vectors exactly like the flat kernel.
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

struct TensorDesc {
    float* p;
    float* v;
    long long n;     // elements
    int vec_ok;      // all of this tensor's buffers are 16-byte aligned: 128-bit path
    int pad;
};

struct TileRecord {
    int tensor;
    int tile;        // index of the 256-vector tile inside the tensor
};

struct MultiArgs {
    const TileRecord* tiles;
    const TensorDesc* desc;
    const void* const* gptr;   // gptr[t * K + k]
    float lambda[DB_MAX_K];    // 0 for a worker with an empty batch: its buffers are not read
    double* partials;
    double* sq_out;
    float lr, mu;
    int K;
};

template <typename GT, bool NORM>
__device__ __forceinline__ void multi_scalar(const MultiArgs& a, const TensorDesc& d, const void* const* g,
                                             long long j, double& sq) {
    float acc = 0.0f;
    for (int k = 0; k < a.K; ++k)
        if (a.lambda[k] != 0.0f) acc = fmaf(a.lambda[k], GradVec<GT>::scalar(g[k], j), acc);
    const float vn = fmaf(a.mu, d.v[j], acc);
    d.v[j] = vn;
    d.p[j] = fmaf(-a.lr, vn, d.p[j]);
    if (NORM) sq += static_cast<double>(acc * acc);
}

// One CTA = one tile of kBlock vectors (kLanes elements each) of one tensor.
template <typename GT, bool NORM>
__global__ void __launch_bounds__(kBlock)
agg_multi_kernel(const __grid_constant__ MultiArgs a) {
    using GV = GradVec<GT>;
    using Raw = typename GV::Raw;
    constexpr int kLanes = GV::kLanes;
    constexpr int kQuads = kLanes / 4;
    if (NORM) agg::griddep_launch_dependents();
    const TileRecord rec = a.tiles[blockIdx.x];
    const TensorDesc d = a.desc[rec.tensor];
    const void* const* g = a.gptr + static_cast<long long>(rec.tensor) * a.K;
    const long long e0 = static_cast<long long>(rec.tile) * kBlock * kLanes;   // first element of the tile
    const long long left = d.n - e0;                                           // > 0 by construction
    double sq = 0.0;

    if (d.vec_ok) {
        const long long full = left / kLanes;            // whole vectors from e0 to the tensor's end
        const long long vi = threadIdx.x;
        if (vi < full) {
            const long long vglob = e0 / kLanes + vi;    // vector index inside the tensor
            float4 pv[kQuads], vv[kQuads];
            float acc[kLanes];
#pragma unroll
            for (int l = 0; l < kLanes; ++l) acc[l] = 0.0f;
#pragma unroll
            for (int q = 0; q < kQuads; ++q) {
                pv[q] = __ldcs(reinterpret_cast<const float4*>(d.p) + vglob * kQuads + q);
                vv[q] = __ldcs(reinterpret_cast<const float4*>(d.v) + vglob * kQuads + q);
            }
            for (int k0 = 0; k0 < a.K; k0 += kChunk) {
                Raw raw[kChunk];
#pragma unroll
                for (int i = 0; i < kChunk; ++i)
                    if (k0 + i < a.K && a.lambda[k0 + i] != 0.0f) raw[i] = GV::load(g[k0 + i], 0, vglob);
#pragma unroll
                for (int i = 0; i < kChunk; ++i) {
                    if (k0 + i < a.K && a.lambda[k0 + i] != 0.0f) {
                        float x[kLanes];
                        GV::widen(raw[i], x);
#pragma unroll
                        for (int l = 0; l < kLanes; ++l) acc[l] = fmaf(a.lambda[k0 + i], x[l], acc[l]);
                    }
                }
            }
            float part = 0.0f;
#pragma unroll
            for (int q = 0; q < kQuads; ++q) {
                float4 vn, pn;
                vn.x = fmaf(a.mu, vv[q].x, acc[4 * q + 0]);
                vn.y = fmaf(a.mu, vv[q].y, acc[4 * q + 1]);
                vn.z = fmaf(a.mu, vv[q].z, acc[4 * q + 2]);
                vn.w = fmaf(a.mu, vv[q].w, acc[4 * q + 3]);
                pn.x = fmaf(-a.lr, vn.x, pv[q].x);
                pn.y = fmaf(-a.lr, vn.y, pv[q].y);
                pn.z = fmaf(-a.lr, vn.z, pv[q].z);
                pn.w = fmaf(-a.lr, vn.w, pv[q].w);
                __stcs(reinterpret_cast<float4*>(d.v) + vglob * kQuads + q, vn);
                __stcs(reinterpret_cast<float4*>(d.p) + vglob * kQuads + q, pn);
                if (NORM) {
#pragma unroll
                    for (int l = 0; l < 4; ++l) part = fmaf(acc[4 * q + l], acc[4 * q + l], part);
                }
            }
            if (NORM) sq += static_cast<double>(part);
        }
        // the tensor's last, partial vector (fewer than kLanes elements) lives in its last tile
        if (full < kBlock) {
            const long long tail0 = e0 + full * kLanes;
            if (tail0 + threadIdx.x < d.n) multi_scalar<GT, NORM>(a, d, g, tail0 + threadIdx.x, sq);
        }
    } else {
        // buffers off the 16-byte grid: element by element, kLanes elements per thread
#pragma unroll 1
        for (int i = 0; i < kLanes; ++i) {
            const long long j = e0 + static_cast<long long>(i) * kBlock + threadIdx.x;
            if (j < d.n && j < e0 + static_cast<long long>(kBlock) * kLanes) multi_scalar<GT, NORM>(a, d, g, j, sq);
        }
    }
    if (NORM) agg::store_norm_partial(a.partials, sq);
}

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Tiles of one tensor: 256 vectors of `lanes` elements each.
long long tiles_of(long long n, int lanes) {
    const long long per = static_cast<long long>(kBlock) * lanes;
    return (n + per - 1) / per;
}

struct PlanLayout {
    long long total_tiles;
    size_t partials_off, desc_off, gptr_off, tiles_off, end;
};

bool plan_layout(int32_t K, int32_t T, const int64_t* sizes, db_dtype dt, PlanLayout* L) {
    const int lanes = dt == DB_F32 ? 4 : 8;
    long long tiles = 0;
    for (int t = 0; t < T; ++t) {
        if (sizes[t] < 0) return false;
        tiles += tiles_of(sizes[t], lanes);
    }
    if (tiles > 0x7fffffffLL) return false;
    L->total_tiles = tiles;
    L->partials_off = 0;
    L->desc_off = L->partials_off + round256(sizeof(double) * static_cast<size_t>(tiles > 0 ? tiles : 1));
    L->gptr_off = L->desc_off + round256(sizeof(TensorDesc) * static_cast<size_t>(T));
    L->tiles_off = L->gptr_off + round256(sizeof(void*) * static_cast<size_t>(T) * K);
    L->end = L->tiles_off + round256(sizeof(TileRecord) * static_cast<size_t>(tiles > 0 ? tiles : 1));
    return true;
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

    std::vector<TensorDesc> desc(T);
    std::vector<const void*> gptr(static_cast<size_t>(T) * K);
    std::vector<TileRecord> tiles(static_cast<size_t>(L.total_tiles));
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
            gptr[static_cast<size_t>(t) * K + k] = g;
        }
        desc[t] = TensorDesc{params[t], momentum[t], n, vec ? 1 : 0, 0};
        const long long nt = tiles_of(n, lanes);
        for (long long i = 0; i < nt; ++i) tiles[next++] = TileRecord{t, static_cast<int>(i)};
    }

    db_multi_plan* plan = new (std::nothrow) db_multi_plan();
    if (!plan) return DB_ERR_ARG;
    char* base = static_cast<char*>(device_table);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t err = cudaMemcpyAsync(base + L.desc_off, desc.data(), sizeof(TensorDesc) * desc.size(),
                                      cudaMemcpyHostToDevice, stream);
    if (err == cudaSuccess)
        err = cudaMemcpyAsync(base + L.gptr_off, gptr.data(), sizeof(void*) * gptr.size(), cudaMemcpyHostToDevice, stream);
    if (err == cudaSuccess && !tiles.empty())
        err = cudaMemcpyAsync(base + L.tiles_off, tiles.data(), sizeof(TileRecord) * tiles.size(),
                              cudaMemcpyHostToDevice, stream);
    // the host vectors go away when this function returns: wait for the copies (plan creation is not on the hot path)
    if (err == cudaSuccess) err = cudaStreamSynchronize(stream);
    if (err != cudaSuccess) {
        delete plan;
        return record_cuda_error(err, "db_multi_plan_create");
    }
    plan->dtype = grad_dtype;
    plan->K = K;
    plan->total_tiles = L.total_tiles;
    plan->args.tiles = reinterpret_cast<const TileRecord*>(base + L.tiles_off);
    plan->args.desc = reinterpret_cast<const TensorDesc*>(base + L.desc_off);
    plan->args.gptr = reinterpret_cast<const void* const*>(base + L.gptr_off);
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
    void (*fn)(const MultiArgs);
    if (plan->dtype == DB_F32) fn = norm ? agg_multi_kernel<float, true> : agg_multi_kernel<float, false>;
    else fn = norm ? agg_multi_kernel<__nv_bfloat16, true> : agg_multi_kernel<__nv_bfloat16, false>;
    fn<<<static_cast<unsigned int>(plan->total_tiles), kBlock, 0, stream>>>(a);
    DB_CUDA_TRY(cudaGetLastError());
    if (norm) DB_CUDA_TRY(agg::launch_norm_finalize(a.partials, plan->total_tiles, a.sq_out, stream, true));
    return DB_OK;
}
