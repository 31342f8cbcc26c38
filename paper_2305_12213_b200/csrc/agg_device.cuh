// Device helpers shared by the aggregation kernels: gradient vector access for fp32 / bf16 storage,
// the ordered block reduction, and the gradient norm's epilogue (one partial per CTA, folded by a
// one-CTA kernel that is launched behind the aggregation kernel).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace dynbatch {
namespace agg {

constexpr int kBlock = 256;      // default CTA size; kernels may run with fewer threads (a multiple of 32)
constexpr int kChunk = 8;        // gradient slices loaded per round when K is not a compile-time constant

// Raw 16-byte gradient vector and its widening to fp32 lanes.
template <typename GT> struct GradVec;

template <> struct GradVec<float> {
    static constexpr int kLanes = 4;
    using Raw = float4;
    static __device__ __forceinline__ Raw load(const void* base, long long head, long long vi) {
        return __ldcs(reinterpret_cast<const float4*>(static_cast<const float*>(base) + head) + vi);
    }
    static __device__ __forceinline__ void widen(const Raw& r, float (&x)[4]) {
        x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w;
    }
    static __device__ __forceinline__ float scalar(const void* base, long long j) {
        return __ldcs(static_cast<const float*>(base) + j);
    }
};

template <> struct GradVec<__nv_bfloat16> {
    static constexpr int kLanes = 8;
    using Raw = uint4;
    static __device__ __forceinline__ Raw load(const void* base, long long head, long long vi) {
        return __ldcs(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(base) + head) + vi);
    }
    // bf16 is the high half of a binary32: widening is a shift, exact.
    static __device__ __forceinline__ void widen(const Raw& r, float (&x)[8]) {
        x[0] = __uint_as_float(r.x << 16); x[1] = __uint_as_float(r.x & 0xffff0000u);
        x[2] = __uint_as_float(r.y << 16); x[3] = __uint_as_float(r.y & 0xffff0000u);
        x[4] = __uint_as_float(r.z << 16); x[5] = __uint_as_float(r.z & 0xffff0000u);
        x[6] = __uint_as_float(r.w << 16); x[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    static __device__ __forceinline__ float scalar(const void* base, long long j) {
        const uint16_t h = __ldcs(static_cast<const uint16_t*>(base) + j);
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};

// Block-wide sum of doubles in a fixed order (xor tree in the warp, warps in order).
__device__ __forceinline__ double block_sum(double x, double* smem) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) smem[warp] = x;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0) {
        for (int w = 0; w < static_cast<int>(blockDim.x) / 32; ++w) s += smem[w];
    }
    return s;  // valid in thread 0
}

// Programmatic dependent launch (no-ops for kernels launched without the attribute): let the next
// kernel in the stream be scheduled while this one runs / wait until the previous kernel has
// completed and its writes are visible.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Ask the L2 to fetch the line that holds `p`; nothing is read into the SM.
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Gradient norm, step 1: every CTA of an aggregation kernel leaves the sum of its squared
// aggregated gradients in partials[blockIdx.x].
__device__ __forceinline__ void store_norm_partial(double* partials, double sq) {
    __shared__ double smem[kBlock / 32];
    const double s = block_sum(sq, smem);
    if (threadIdx.x == 0) partials[blockIdx.x] = s;
}

// Gradient norm, step 2: one CTA folds the n partials in index order.  Launched right behind the
// aggregation kernel with programmatic stream serialization, so its launch latency is hidden; it
// touches the partials only after griddepcontrol.wait.  No counter, nothing to initialise, nobody spins.
static __global__ void __launch_bounds__(1024) norm_finalize_kernel(const double* __restrict__ partials, long long n,
                                                             double* __restrict__ sq_out) {
    __shared__ double smem[32];
    griddep_launch_dependents();     // the next step's kernel may be scheduled; it waits for this one itself
    griddep_wait();
    double acc = 0.0;
    for (long long i = threadIdx.x; i < n; i += blockDim.x) acc += __ldcg(partials + i);
    const double total = block_sum(acc, smem);
    if (threadIdx.x == 0) *sq_out = total;
}

// Enqueues norm_finalize_kernel behind the kernel just launched on `stream`; `overlap` lets it be scheduled
// while that kernel still runs.
static inline cudaError_t launch_norm_finalize(const double* partials, long long n, double* sq_out, cudaStream_t stream,
                                               bool overlap) {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1]{};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(n > 256 ? 1024 : 256);      // one partial per thread up to 1024 CTAs: a single round trip
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;   // without the attribute the kernel simply runs after its predecessor
    return cudaLaunchKernelEx(&cfg, norm_finalize_kernel, partials, n, sq_out);
}

}  // namespace agg
}  // namespace dynbatch
