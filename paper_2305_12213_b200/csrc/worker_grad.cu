// Ragged per-worker mean gradient of a bias-free linear-softmax classifier:
//     Z = X W,  P = softmax_rows(Z),  G = X^T (P - Y) / b_i
// the model on which Eq. 2's batch-proportional weights are checked against
// the gradient of the concatenated global batch (Section 3.1).
//
// Three launches on the caller's stream:
//   1. logits: split over the feature dimension D so that a worker with a
//      handful of rows still fills the GPU; partial sums go to the workspace;
//   2. softmax: one CTA per sample folds the partials in split order, applies
//      the max-subtracted softmax, subtracts the one-hot label, scales by 1/b_i;
//   3. gradient: G = X^T E, one 64x64 output tile per CTA, reduction depth b_i.
// Both contractions are fp32 FFMA on shared-memory tiles: at b_i <= 128 they
// sit below the tensor-core ridge (bounded by reading W and writing G).
#include <cstdint>

#include "common.h"

namespace dynbatch {
namespace {

constexpr int kTile = 64;      // output tile edge
constexpr int kDepth = 16;     // reduction slice per shared-memory stage
constexpr int kThreads = 256;  // 16 x 16 threads, 4 x 4 outputs each

// out[m, n] = sum_{k in split} A(m, k) * B[k, n]
//   A(m, k) = TRANS_A ? A[k * lda + m] : A[m * lda + k];   B row-major, ldb
//   split z covers k in [z * k_per_split, min(Kd, (z + 1) * k_per_split)) and
//   writes to out + z * split_stride.
// VEC4: lda, ldb multiples of 4 and 16-byte aligned bases (128-bit loads).
template <bool TRANS_A, bool VEC4>
__global__ void __launch_bounds__(kThreads)
tile_gemm_kernel(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                 float* __restrict__ out, int ldo, long long split_stride, int M, int N, int Kd,
                 int k_per_split) {
    __shared__ __align__(16) float As[kDepth][kTile + 4];
    __shared__ __align__(16) float Bs[kDepth][kTile];

    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
    const int k_begin = blockIdx.z * k_per_split;
    const int k_end = min(Kd, k_begin + k_per_split);
    const int tx = tid & 15, ty = tid >> 4;  // outputs: rows ty*4.., cols tx*4..

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    for (int k0 = k_begin; k0 < k_end; k0 += kDepth) {
        // ---- stage A (kTile x kDepth) transposed into As[k][m]
        if (TRANS_A) {
            const int kk = tid >> 4, mm = (tid & 15) * 4;  // 16 k-rows x 16 groups of 4 m
            const int k = k0 + kk, m = m0 + mm;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k < k_end) {
                const float* src = A + static_cast<long long>(k) * lda + m;
                if (VEC4 && m + 3 < M) {
                    t = *reinterpret_cast<const float4*>(src);
                } else {
                    if (m + 0 < M) t.x = src[0];
                    if (m + 1 < M) t.y = src[1];
                    if (m + 2 < M) t.z = src[2];
                    if (m + 3 < M) t.w = src[3];
                }
            }
            *reinterpret_cast<float4*>(&As[kk][mm]) = t;
        } else {
            const int mm = tid >> 2, kk = (tid & 3) * 4;  // 64 m-rows x 4 groups of 4 k
            const int m = m0 + mm, k = k0 + kk;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m < M) {
                const float* src = A + static_cast<long long>(m) * lda + k;
                if (VEC4 && k + 3 < k_end) {
                    t = *reinterpret_cast<const float4*>(src);
                } else {
                    if (k + 0 < k_end) t.x = src[0];
                    if (k + 1 < k_end) t.y = src[1];
                    if (k + 2 < k_end) t.z = src[2];
                    if (k + 3 < k_end) t.w = src[3];
                }
            }
            As[kk + 0][mm] = t.x;
            As[kk + 1][mm] = t.y;
            As[kk + 2][mm] = t.z;
            As[kk + 3][mm] = t.w;
        }
        // ---- stage B (kDepth x kTile)
        {
            const int kk = tid >> 4, nn = (tid & 15) * 4;
            const int k = k0 + kk, n = n0 + nn;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k < k_end) {
                const float* src = B + static_cast<long long>(k) * ldb + n;
                if (VEC4 && n + 3 < N) {
                    t = *reinterpret_cast<const float4*>(src);
                } else {
                    if (n + 0 < N) t.x = src[0];
                    if (n + 1 < N) t.y = src[1];
                    if (n + 2 < N) t.z = src[2];
                    if (n + 3 < N) t.w = src[3];
                }
            }
            *reinterpret_cast<float4*>(&Bs[kk][nn]) = t;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kDepth; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a4.x, a4.y, a4.z, a4.w};
            const float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

    float* dst = out + static_cast<long long>(blockIdx.z) * split_stride;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
        const int n = n0 + tx * 4;
        float* row = dst + static_cast<long long>(m) * ldo + n;
        if (VEC4 && (ldo & 3) == 0 && n + 3 < N) {
            *reinterpret_cast<float4*>(row) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (n + j < N) row[j] = acc[i][j];
        }
    }
}

__device__ __forceinline__ float block_reduce(float x, float* smem, bool take_max) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, x, off);
        x = take_max ? fmaxf(x, o) : x + o;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = x;
    __syncthreads();
    float r = smem[0];
    for (int w = 1; w < kThreads / 32; ++w) r = take_max ? fmaxf(r, smem[w]) : r + smem[w];
    return r;  // same value in every thread
}

// One CTA per sample i:  E[i, :] = (softmax(z_i) - onehot(y_i)) / b,  z_i = sum of the split partials.
__global__ void __launch_bounds__(kThreads)
softmax_residual_kernel(const float* __restrict__ partials, int splits, long long split_stride,
                        const int32_t* __restrict__ y, float* __restrict__ E, float* __restrict__ row_loss,
                        int b, int C) {
    __shared__ float smem[kThreads / 32];
    const int i = blockIdx.x;
    float* e = E + static_cast<long long>(i) * C;
    const float* z0 = partials + static_cast<long long>(i) * C;
    float zmax = -INFINITY;
    for (int c = threadIdx.x; c < C; c += kThreads) {
        float z = 0.0f;
        for (int s = 0; s < splits; ++s) z += z0[static_cast<long long>(s) * split_stride + c];
        e[c] = z;
        zmax = fmaxf(zmax, z);
    }
    zmax = block_reduce(zmax, smem, true);
    float den = 0.0f;
    for (int c = threadIdx.x; c < C; c += kThreads) den += expf(e[c] - zmax);
    den = block_reduce(den, smem, false);
    const int label = y[i];
    const float inv_b = 1.0f / static_cast<float>(b);
    if (threadIdx.x == 0)
        row_loss[i] = (label >= 0 && label < C) ? -((e[label] - zmax) - logf(den)) : 0.0f;
    __syncthreads();  // e[label] read above before it is overwritten below
    for (int c = threadIdx.x; c < C; c += kThreads) {
        float r = expf(e[c] - zmax) / den;
        if (c == label) r -= 1.0f;
        e[c] = r * inv_b;
    }
}

__global__ void mean_loss_kernel(const float* __restrict__ row_loss, int b, float* __restrict__ loss) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        float s = 0.0f;
        for (int i = 0; i < b; ++i) s += row_loss[i];
        *loss = s / static_cast<float>(b);
    }
}

size_t round16(size_t x) { return (x + 15) & ~static_cast<size_t>(15); }

// Splits of the feature dimension for the logits so that about two CTAs per SM exist.
int logit_splits(int b, int D, int C) {
    const long long tiles = static_cast<long long>((b + kTile - 1) / kTile) * ((C + kTile - 1) / kTile);
    const long long want = 2LL * sm_count();
    long long s = (want + tiles - 1) / tiles;
    const long long max_s = (D + 4 * kDepth - 1) / (4 * kDepth);  // at least 64 features per split
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}

struct WorkerLayout {
    int splits, k_per_split;
    size_t partial_bytes, e_bytes, loss_bytes;
};

WorkerLayout layout_for(int b, int D, int C) {
    WorkerLayout L;
    L.splits = logit_splits(b, D, C);
    int per = (D + L.splits - 1) / L.splits;
    per = (per + kDepth - 1) / kDepth * kDepth;  // whole stages, keeps 16-byte alignment of k offsets
    L.k_per_split = per;
    L.splits = (D + per - 1) / per;
    L.partial_bytes = round16(sizeof(float) * static_cast<size_t>(L.splits) * b * C);
    L.e_bytes = round16(sizeof(float) * static_cast<size_t>(b) * C);
    L.loss_bytes = round16(sizeof(float) * static_cast<size_t>(b));
    return L;
}

bool valid_shape(int b, int D, int C) { return b >= 1 && b <= 65535 && D >= 1 && C >= 1; }

}  // namespace
}  // namespace dynbatch

extern "C" size_t db_worker_grad_workspace_bytes(int32_t b_i, int32_t D, int32_t C) {
    using namespace dynbatch;
    if (!valid_shape(b_i, D, C)) return 0;
    const WorkerLayout L = layout_for(b_i, D, C);
    return L.partial_bytes + L.e_bytes + L.loss_bytes;
}

extern "C" db_status db_worker_grad(const float* X, const int32_t* y, const float* W, int32_t b_i,
                                    int32_t D, int32_t C, float* G, float* loss, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream) {
    using namespace dynbatch;
    if (!X || !y || !W || !G || !workspace) return DB_ERR_NULL;
    if (!valid_shape(b_i, D, C)) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return DB_ERR_ARG;
    const WorkerLayout L = layout_for(b_i, D, C);
    if (workspace_bytes < L.partial_bytes + L.e_bytes + L.loss_bytes) return DB_ERR_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    float* partials = static_cast<float*>(workspace);
    float* E = reinterpret_cast<float*>(static_cast<char*>(workspace) + L.partial_bytes);
    float* row_loss = reinterpret_cast<float*>(static_cast<char*>(workspace) + L.partial_bytes + L.e_bytes);
    const bool vec4 = (D % 4 == 0) && (C % 4 == 0) && reinterpret_cast<uintptr_t>(X) % 16 == 0 &&
                      reinterpret_cast<uintptr_t>(W) % 16 == 0 && reinterpret_cast<uintptr_t>(G) % 16 == 0;
    const long long bc = static_cast<long long>(b_i) * C;

    // 1. logits, split over D
    {
        dim3 grid((C + kTile - 1) / kTile, (b_i + kTile - 1) / kTile, L.splits);
        if (vec4)
            tile_gemm_kernel<false, true><<<grid, kThreads, 0, stream>>>(X, D, W, C, partials, C, bc, b_i, C, D,
                                                                         L.k_per_split);
        else
            tile_gemm_kernel<false, false><<<grid, kThreads, 0, stream>>>(X, D, W, C, partials, C, bc, b_i, C, D,
                                                                          L.k_per_split);
        DB_CUDA_TRY(cudaGetLastError());
    }
    // 2. softmax residual (P - Y) / b
    softmax_residual_kernel<<<b_i, kThreads, 0, stream>>>(partials, L.splits, bc, y, E, row_loss, b_i, C);
    DB_CUDA_TRY(cudaGetLastError());
    // 3. G = X^T E
    {
        dim3 grid((C + kTile - 1) / kTile, (D + kTile - 1) / kTile, 1);
        if (vec4)
            tile_gemm_kernel<true, true><<<grid, kThreads, 0, stream>>>(X, D, E, C, G, C, 0, D, C, b_i, b_i);
        else
            tile_gemm_kernel<true, false><<<grid, kThreads, 0, stream>>>(X, D, E, C, G, C, 0, D, C, b_i, b_i);
        DB_CUDA_TRY(cudaGetLastError());
    }
    if (loss) {
        mean_loss_kernel<<<1, 32, 0, stream>>>(row_loss, b_i, loss);
        DB_CUDA_TRY(cudaGetLastError());
    }
    return DB_OK;
}
