// Device code of the fused K-way weighted gradient aggregation + optimizer update
// (Section 3.1, Eq. 2-3; momentum optimizer of Section 4's ResNet-50 workload; Adam of its MNIST workload).
// Kept apart from the host code of aggregate.cu so that the kernels' text changes only when the kernels do.
#pragma once
#include <cuda_bf16.h>

#include <cstdint>

#include "agg_device.cuh"
#include "dynbatch.h"

namespace dynbatch {
namespace {

using agg::GradVec;
using agg::kBlock;
using agg::kChunk;

struct AggArgs {
    const void* g[DB_MAX_K];  // active workers' gradient buffers
    float lambda[DB_MAX_K];   // their weights b_k / sum b
    float* p;
    float* v;                 // momentum (heavy ball) or first moment (Adam)
    float* u;                 // second moment (Adam only)
    double* partials;         // one per CTA (norm only)
    double* sq_out;
    long long n;              // elements
    long long head;           // leading elements before the first 16-byte boundary
    long long nvec;           // whole vectors after the head
    float lr, mu;             // mu: momentum coefficient, or Adam's beta1
    float beta2, eps, inv_c1, inv_c2;   // Adam: 1 / (1 - beta^t) bias corrections
    int K;
    int prefetch_ctas;        // CTAs [0, prefetch_ctas) ask the L2 for their state vectors before they wait
};

enum Optimizer { kMomentum = 0, kAdam = 1 };

// The optimizer step on one element, given the aggregated gradient g.
//   momentum: v <- mu v + g;                  p <- p - lr v
//   Adam:     m <- b1 m + (1 - b1) g;  u <- b2 u + (1 - b2) g^2;
//             p <- p - lr (m / c1) / (sqrt(u / c2) + eps)
template <int OPT>
__device__ __forceinline__ void optimizer_step(const AggArgs& a, float g, float& p, float& v, float& u) {
    if (OPT == kMomentum) {
        v = fmaf(a.mu, v, g);
        p = fmaf(-a.lr, v, p);
    } else {
        v = fmaf(a.mu, v, (1.0f - a.mu) * g);
        u = fmaf(a.beta2, u, (1.0f - a.beta2) * (g * g));
        const float denom = sqrtf(u * a.inv_c2) + a.eps;
        p = p - a.lr * (v * a.inv_c1) / denom;
    }
}

// One element, any alignment: the same FMA chain as the vector body.
template <typename GT, bool NORM, int OPT>
__device__ __forceinline__ void update_scalar(const AggArgs& a, int K, long long j, double& sq) {
    float g = 0.0f;
    for (int k = 0; k < K; ++k) g = fmaf(a.lambda[k], GradVec<GT>::scalar(a.g[k], j), g);
    float p = a.p[j], v = a.v[j], u = OPT == kAdam ? a.u[j] : 0.0f;
    optimizer_step<OPT>(a, g, p, v, u);
    a.v[j] = v;
    a.p[j] = p;
    if (OPT == kAdam) a.u[j] = u;
    if (NORM) sq += static_cast<double>(g * g);
}

// Optimizer update of the `kLanes` elements at vector index vi.
template <int kLanes, bool NORM, int OPT>
__device__ __forceinline__ void apply_update(const AggArgs& a, long long vi, const float (&g)[kLanes],
                                             float4 (&pv)[kLanes / 4], float4 (&vv)[kLanes / 4],
                                             float4 (&uv)[kLanes / 4], double& sq) {
    float4* pp = reinterpret_cast<float4*>(a.p + a.head) + vi * (kLanes / 4);
    float4* vp = reinterpret_cast<float4*>(a.v + a.head) + vi * (kLanes / 4);
    float part = 0.0f;
#pragma unroll
    for (int q = 0; q < kLanes / 4; ++q) {
        optimizer_step<OPT>(a, g[4 * q + 0], pv[q].x, vv[q].x, uv[q].x);
        optimizer_step<OPT>(a, g[4 * q + 1], pv[q].y, vv[q].y, uv[q].y);
        optimizer_step<OPT>(a, g[4 * q + 2], pv[q].z, vv[q].z, uv[q].z);
        optimizer_step<OPT>(a, g[4 * q + 3], pv[q].w, vv[q].w, uv[q].w);
        __stcs(vp + q, vv[q]);
        __stcs(pp + q, pv[q]);
        if (OPT == kAdam) __stcs(reinterpret_cast<float4*>(a.u + a.head) + vi * (kLanes / 4) + q, uv[q]);
        if (NORM) {
#pragma unroll
            for (int l = 0; l < 4; ++l) part = fmaf(g[4 * q + l], g[4 * q + l], part);
        }
    }
    if (NORM) sq += static_cast<double>(part);
}

// KT > 0: exactly KT workers, fully unrolled.  KT == 0: a.K workers, kChunk at a time.
// A CTA of BLOCK threads handles TILES consecutive tiles of BLOCK x UNROLL vectors.
template <typename GT, int KT, int BLOCK, int UNROLL, int TILES, bool NORM, int OPT>
__global__ void __launch_bounds__(BLOCK)
agg_vec_kernel(const __grid_constant__ AggArgs a) {
    using GV = GradVec<GT>;
    using Raw = typename GV::Raw;
    constexpr int kLanes = GV::kLanes;
    constexpr int kQuads = kLanes / 4;
    const int K = KT > 0 ? KT : a.K;
    double sq = 0.0;
    // Programmatic dependent launch, both ways: the kernel behind this one in the stream (the norm's fold, or
    // the next step) may be scheduled already, and this one, if it was itself scheduled early, touches
    // memory only once its predecessor has completed.  Both are no-ops for ordinary launches.
    agg::griddep_launch_dependents();
    const long long tile = static_cast<long long>(BLOCK) * UNROLL;
    // On a small grid the CTAs are resident while the predecessor still runs.  They use that time to ask the
    // L2 for their part of the state vectors (a prefetch consumes no data, so it needs no ordering against
    // whoever may still be writing them); their loads after the wait then meet the L2 instead of DRAM.  The
    // host sets prefetch_ctas to the grid size for such launches and to zero for all others.  (Not in the
    // chunked kernel, KT == 0: with this block compiled in, it ran 27 % slower at N = 2^20, K = 32.)
    if (KT > 0 && static_cast<int>(blockIdx.x) < a.prefetch_ctas) {
#pragma unroll 1
        for (int t = 0; t < TILES; ++t) {
            const long long base = (static_cast<long long>(blockIdx.x) * TILES + t) * tile;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const long long v0 = base + u * BLOCK + threadIdx.x;
                if (v0 >= a.nvec) continue;
                agg::prefetch_l2(reinterpret_cast<const float4*>(a.p + a.head) + v0 * kQuads);
                agg::prefetch_l2(reinterpret_cast<const float4*>(a.v + a.head) + v0 * kQuads);
                if (OPT == kAdam) agg::prefetch_l2(reinterpret_cast<const float4*>(a.u + a.head) + v0 * kQuads);
            }
        }
    }
    agg::griddep_wait();

#pragma unroll 1
    for (int t = 0; t < TILES; ++t) {
        const long long base = (static_cast<long long>(blockIdx.x) * TILES + t) * tile;
        if (base >= a.nvec) break;
        long long vi[UNROLL];
        bool ok[UNROLL];
        float4 pv[UNROLL][kQuads], vv[UNROLL][kQuads], uv[UNROLL][kQuads];
        float g[UNROLL][kLanes];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            vi[u] = base + u * BLOCK + threadIdx.x;
            ok[u] = vi[u] < a.nvec;
#pragma unroll
            for (int l = 0; l < kLanes; ++l) g[u][l] = 0.0f;
        }
        if (KT > 0) {
            Raw raw[UNROLL][KT > 0 ? KT : 1];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!ok[u]) continue;
#pragma unroll
                for (int k = 0; k < KT; ++k) raw[u][k] = GV::load(a.g[k], a.head, vi[u]);
#pragma unroll
                for (int q = 0; q < kQuads; ++q) {
                    pv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.p + a.head) + vi[u] * kQuads + q);
                    vv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.v + a.head) + vi[u] * kQuads + q);
                    if (OPT == kAdam)
                        uv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.u + a.head) + vi[u] * kQuads + q);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!ok[u]) continue;
#pragma unroll
                for (int k = 0; k < KT; ++k) {
                    float x[kLanes];
                    GV::widen(raw[u][k], x);
#pragma unroll
                    for (int l = 0; l < kLanes; ++l) g[u][l] = fmaf(a.lambda[k], x[l], g[u][l]);
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!ok[u]) continue;
#pragma unroll
                for (int q = 0; q < kQuads; ++q) {
                    pv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.p + a.head) + vi[u] * kQuads + q);
                    vv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.v + a.head) + vi[u] * kQuads + q);
                    if (OPT == kAdam)
                        uv[u][q] = __ldcs(reinterpret_cast<const float4*>(a.u + a.head) + vi[u] * kQuads + q);
                }
                for (int k0 = 0; k0 < K; k0 += kChunk) {
                    Raw raw[kChunk];
#pragma unroll
                    for (int i = 0; i < kChunk; ++i)
                        if (k0 + i < K) raw[i] = GV::load(a.g[k0 + i], a.head, vi[u]);
#pragma unroll
                    for (int i = 0; i < kChunk; ++i) {
                        if (k0 + i < K) {
                            float x[kLanes];
                            GV::widen(raw[i], x);
#pragma unroll
                            for (int l = 0; l < kLanes; ++l)
                                g[u][l] = fmaf(a.lambda[k0 + i], x[l], g[u][l]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (ok[u]) apply_update<kLanes, NORM, OPT>(a, vi[u], g[u], pv[u], vv[u], uv[u], sq);
    }

    // ragged ends: fewer than kLanes elements on either side of the vector body
    if (blockIdx.x == 0) {
        const long long tail0 = a.head + a.nvec * kLanes;
        if (threadIdx.x < a.head) update_scalar<GT, NORM, OPT>(a, K, threadIdx.x, sq);
        if (tail0 + threadIdx.x < a.n) update_scalar<GT, NORM, OPT>(a, K, tail0 + threadIdx.x, sq);
    }
    if (NORM) agg::store_norm_partial(a.partials, sq);
}

// Element-wise kernel for buffers whose 16-byte boundaries do not line up.
template <typename GT, bool NORM, int OPT>
__global__ void __launch_bounds__(kBlock)
agg_scalar_kernel(const __grid_constant__ AggArgs a) {
    double sq = 0.0;
    agg::griddep_launch_dependents();
    agg::griddep_wait();
    const long long step = static_cast<long long>(gridDim.x) * kBlock;
    for (long long j = static_cast<long long>(blockIdx.x) * kBlock + threadIdx.x; j < a.n; j += step)
        update_scalar<GT, NORM, OPT>(a, a.K, j, sq);
    if (NORM) agg::store_norm_partial(a.partials, sq);
}

}  // namespace
}  // namespace dynbatch
