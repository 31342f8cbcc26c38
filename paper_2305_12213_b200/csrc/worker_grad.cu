// Ragged per-worker mean gradient of a bias-free linear-softmax classifier:
//     Z = X W,  P = softmax_rows(Z),  G = X^T (P - Y) / b_i
// the model on which Eq. 2's batch-proportional weights are checked against
// the gradient of the concatenated global batch (Section 3.1).
//
// Three launches on the caller's stream, each scheduled under its predecessor (programmatic
// dependent launch) and waiting for it before it reads its output:
//   1. logits: split over the feature dimension D so that a worker with a
//      handful of rows still fills the GPU; partial sums go to the workspace;
//      its first CTA also zeroes the status word of the call;
//   2. softmax: one CTA per sample folds the partials in split order, applies
//      the max-subtracted softmax, subtracts the one-hot label, scales by 1/b_i;
//   3. gradient: G = X^T E, reduction depth b_i; one CTA per worker also folds
//      the per-sample losses into the worker's mean loss.
// (The FFMA path keeps a memset node for its status word and loss ticket.)
// The two contractions run on the tensor cores (tcgen05, three TF32 products per
// fp32 product), fed by TMA: the logits read W and X where the caller left them
// (tc_logits.cuh; unaligned inputs go through the register-converting contraction of
// tc_gemm.cuh), and for the gradient the softmax kernel leaves E and a copy of X
// already split into TF32 halves, row-major (tc_grad.cuh).  An fp32 FFMA version on
// shared-memory tiles is kept as the accuracy reference and for very large b_i.
#include <algorithm>
#include <cstdint>

#include "common.h"
#include "tc_gemm.cuh"
#include "tc_grad.cuh"
#include "tc_logits.cuh"

namespace dynbatch {
namespace {

constexpr int kTile = 64;      // output tile edge
constexpr int kDepth = 16;     // reduction slice per shared-memory stage
constexpr int kThreads = 256;  // 16 x 16 threads, 4 x 4 outputs each
// CTA of the softmax kernel (one per sample).  Measured on the 1000-class check model, step back to back:
// 256 threads 41.7 us, 512 threads 41.0, 768 threads 42.4, 1024 threads 45.3; 128 threads (logits parked in
// memory between the passes) 44.0.
constexpr int kSoftmaxThreads = 512;

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
    for (int w = 1; w < kSoftmaxThreads / 32; ++w) r = take_max ? fmaxf(r, smem[w]) : r + smem[w];
    return r;  // same value in every thread
}

// One CTA per sample i:  E[i, :] = (softmax(z_i) - onehot(y_i)) / b,  z_i = sum of the split partials
// (split order).  The last CTA to finish also folds the per-sample losses into the mean loss; arrival
// order comes from an atomic ticket (zeroed by the caller), nobody waits.
// IN_REGS: C <= 4 * kSoftmaxThreads, every thread keeps its up to four logits in registers (one pass over memory);
// otherwise the logits are parked in E between the passes.
// Rows [off[w], off[w + 1]) belong to worker w; each worker has its own 1/b, ticket and loss slot.
struct RowGroups {
    int K;
    int off[DB_MAX_K + 1];
    int poff[DB_MAX_K + 1];   // SPLIT: the workers' first rows in the split arrays (multiples of 8)
};

// SPLIT: where the operands of the tensor-core gradient contraction go.  Row i of worker w lands in
// row poff[w] + (i - off[w]) of four row-major arrays: E split into TF32 halves (e_hi + e_lo = E up to
// 2^-22) and the same split of the sample's feature row X[i, :].  The grid then has one CTA per row of
// the split arrays; the CTAs of the up to 7 padding rows behind each worker write zeros.
struct SplitOut {
    float* e_hi;
    float* e_lo;
    long long e_pitch;     // floats per row, >= C
    const float* X;        // [rows, D] row-major
    float* x_hi;
    float* x_lo;
    long long x_pitch;     // floats per row, >= D, multiple of 4
    int D;
    int x_vec;             // D % 4 == 0 and X 16-byte aligned: 128-bit loads
};

template <bool IN_REGS, bool SPLIT>
__global__ void __launch_bounds__(kSoftmaxThreads)
softmax_residual_kernel(const float* __restrict__ partials, int splits, long long split_stride,
                        const int32_t* __restrict__ y, float* __restrict__ E, float* __restrict__ row_loss,
                        const __grid_constant__ RowGroups groups, int C, unsigned int* __restrict__ tickets,
                        float* __restrict__ losses, const __grid_constant__ SplitOut so) {
    __shared__ float smem[kSoftmaxThreads / 32];
    __shared__ float z_label;
    __shared__ bool is_last;
    tc::griddep_launch_dependents();
    int i = blockIdx.x, w = 0;
    float* eh = nullptr;
    float* el = nullptr;
    if (SPLIT) {
        const int ip = blockIdx.x;
        while (w + 1 < groups.K && ip >= groups.poff[w + 1]) ++w;
        const int r = ip - groups.poff[w];
        eh = so.e_hi + static_cast<long long>(ip) * so.e_pitch;
        el = so.e_lo + static_cast<long long>(ip) * so.e_pitch;
        float* xh = so.x_hi + static_cast<long long>(ip) * so.x_pitch;
        float* xl = so.x_lo + static_cast<long long>(ip) * so.x_pitch;
        // the columns between C (D) and the pitch are copied with the rest of their 32-column chunk: zeros
        for (int c = C + threadIdx.x; c < so.e_pitch; c += kSoftmaxThreads) { eh[c] = 0.0f; el[c] = 0.0f; }
        for (int d = so.D + threadIdx.x; d < so.x_pitch; d += kSoftmaxThreads) { xh[d] = 0.0f; xl[d] = 0.0f; }
        if (r >= groups.off[w + 1] - groups.off[w]) {
            // padding row: zeros in all four arrays (the workspace may hold anything, NaN included)
            for (int c = threadIdx.x; c < C; c += kSoftmaxThreads) { eh[c] = 0.0f; el[c] = 0.0f; }
            for (int d = threadIdx.x; d < so.D; d += kSoftmaxThreads) { xh[d] = 0.0f; xl[d] = 0.0f; }
            return;
        }
        i = groups.off[w] + r;
        // the feature row is an input of the whole call, not of the logits kernel: split it while that runs
        const float* xr = so.X + static_cast<long long>(i) * so.D;
        if (so.x_vec) {
            for (int d = threadIdx.x * 4; d < so.D; d += 4 * kSoftmaxThreads) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(xr + d));
                float4 h, l;
                tc::split_tf32(v.x, h.x, l.x);
                tc::split_tf32(v.y, h.y, l.y);
                tc::split_tf32(v.z, h.z, l.z);
                tc::split_tf32(v.w, h.w, l.w);
                *reinterpret_cast<float4*>(xh + d) = h;
                *reinterpret_cast<float4*>(xl + d) = l;
            }
        } else {
            for (int d = threadIdx.x; d < so.D; d += kSoftmaxThreads) tc::split_tf32(__ldg(xr + d), xh[d], xl[d]);
        }
    } else {
        while (w + 1 < groups.K && i >= groups.off[w + 1]) ++w;
    }
    const int row0 = groups.off[w], b = groups.off[w + 1] - row0;
    unsigned int* ticket = tickets + w;
    float* loss = losses ? losses + w : nullptr;
    float* e = E + static_cast<long long>(i) * C;
    const float* z0 = partials + static_cast<long long>(i) * C;
    const int label = y[i];
    const float inv_b = 1.0f / static_cast<float>(b);
    float zmax = -INFINITY;
    float z[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (threadIdx.x == 0) z_label = 0.0f;
    tc::griddep_wait();      // the logits kernel has finished and its partial sums are visible
    // four classes per thread and eight splits per round: 32 independent loads in flight, adds in split order
    for (int cb = 0; cb < C; cb += 4 * kSoftmaxThreads) {
#pragma unroll
        for (int j = 0; j < 4; ++j) z[j] = 0.0f;
        for (int s0 = 0; s0 < splits; s0 += 8) {
            float t[4][8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = cb + j * kSoftmaxThreads + threadIdx.x;
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    t[j][u] = (c < C && s0 + u < splits)
                                  ? __ldg(z0 + static_cast<long long>(s0 + u) * split_stride + c) : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (s0 + u < splits) z[j] += t[j][u];
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = cb + j * kSoftmaxThreads + threadIdx.x;
            if (c < C) {
                if (!IN_REGS) e[c] = z[j];
                zmax = fmaxf(zmax, z[j]);
            }
        }
    }
    zmax = block_reduce(zmax, smem, true);
    float den = 0.0f;
    if (IN_REGS) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = j * kSoftmaxThreads + threadIdx.x;
            if (c < C) {
                z[j] = expf(z[j] - zmax);       // numerator of the softmax
                den += z[j];
                if (c == label) z_label = z[j];
            }
        }
    } else {
        for (int c = threadIdx.x; c < C; c += kSoftmaxThreads) {
            const float p = expf(e[c] - zmax);
            den += p;
            if (c == label) z_label = p;
        }
    }
    den = block_reduce(den, smem, false);       // its barriers also publish z_label
    if (threadIdx.x == 0)
        row_loss[i] = (label >= 0 && label < C) ? -logf(z_label / den) : 0.0f;
    if (IN_REGS) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = j * kSoftmaxThreads + threadIdx.x;
            if (c < C) {
                float r = z[j] / den;
                if (c == label) r -= 1.0f;
                r *= inv_b;
                if (SPLIT) tc::split_tf32(r, eh[c], el[c]);
                else e[c] = r;
            }
        }
    } else {
        for (int c = threadIdx.x; c < C; c += kSoftmaxThreads) {
            float r = expf(e[c] - zmax) / den;
            if (c == label) r -= 1.0f;
            r *= inv_b;
            if (SPLIT) tc::split_tf32(r, eh[c], el[c]);
            else e[c] = r;
        }
    }
    if (loss == nullptr) return;
    if (threadIdx.x == 0) {
        __threadfence();
        is_last = atomicAdd(ticket, 1u) == static_cast<unsigned int>(b) - 1u;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    float part = 0.0f;
    for (int r = threadIdx.x; r < b; r += kSoftmaxThreads) part += __ldcg(row_loss + row0 + r);
    const float total = block_reduce(part, smem, false);
    if (threadIdx.x == 0) *loss = total * inv_b;
}

// Launch configuration of a kernel that may start while its predecessor in the stream still runs
// (it calls griddepcontrol.wait before reading the predecessor's output).
struct OverlappedLaunch {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1]{};
    OverlappedLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool overlap) {
        cfg.gridDim = grid;
        cfg.blockDim = block;
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = overlap ? 1 : 0;
    }
};

// `split` non-null: one CTA per row of the split arrays (groups.poff[groups.K] of them), else one per sample.
db_status launch_softmax(const float* partials, int splits, long long split_stride, const int32_t* y, float* E,
                         float* row_loss, const RowGroups& groups, int rows, int C, unsigned int* tickets,
                         float* losses, cudaStream_t stream, bool overlap, const SplitOut* split = nullptr) {
    const bool in_regs = C <= 4 * kSoftmaxThreads;
    OverlappedLaunch L(dim3(split ? groups.poff[groups.K] : rows), dim3(kSoftmaxThreads), 0, stream, overlap);
    const SplitOut so = split ? *split : SplitOut{};
    auto fn = split ? (in_regs ? softmax_residual_kernel<true, true> : softmax_residual_kernel<false, true>)
                    : (in_regs ? softmax_residual_kernel<true, false> : softmax_residual_kernel<false, false>);
    DB_CUDA_TRY(cudaLaunchKernelEx(&L.cfg, fn, partials, splits, split_stride, y, E, row_loss, groups, C, tickets,
                                   losses, so));
    return DB_OK;
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

constexpr int kMaxTensorCoreBatch = 4096;  // longer reductions over the batch go to FFMA
constexpr size_t kStatusBytes = 16;        // device status word of the tensor-core kernels

// Workspace of the FFMA path (one worker).
struct WorkerLayout {
    int splits, k_per_split;
    size_t partial_bytes, e_bytes, loss_bytes;
    size_t total() const { return kStatusBytes + partial_bytes + e_bytes + loss_bytes; }
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

using TcKernel = void (*)(const tc::GemmArgs);

template <int N_TILE, int MODE_A>
TcKernel pick_tc_b(int mode_b) {
    switch (mode_b) {
        case tc::kLoadKVec: return tc::tf32x3_gemm_kernel<N_TILE, MODE_A, tc::kLoadKVec>;
        case tc::kLoadRowVec: return tc::tf32x3_gemm_kernel<N_TILE, MODE_A, tc::kLoadRowVec>;
        default: return tc::tf32x3_gemm_kernel<N_TILE, MODE_A, tc::kLoadScalar>;
    }
}

template <int N_TILE>
TcKernel pick_tc(int mode_a, int mode_b) {
    switch (mode_a) {
        case tc::kLoadKVec: return pick_tc_b<N_TILE, tc::kLoadKVec>(mode_b);
        case tc::kLoadRowVec: return pick_tc_b<N_TILE, tc::kLoadRowVec>(mode_b);
        default: return pick_tc_b<N_TILE, tc::kLoadScalar>(mode_b);
    }
}

// Widest loader the operand's strides and alignment allow.
int load_mode(const float* p, long long row_stride, long long k_stride) {
    const bool base16 = reinterpret_cast<uintptr_t>(p) % 16 == 0;
    if (k_stride == 1 && row_stride % 4 == 0 && base16) return tc::kLoadKVec;
    if (row_stride == 1 && k_stride % 4 == 0 && base16) return tc::kLoadRowVec;
    return tc::kLoadScalar;
}

// out(m, n) = sum_k A(m, k) B(n, k) on the tensor cores; a.k_per_split must be a multiple of 32.
db_status launch_tc_gemm(tc::GemmArgs a, int n_tile, cudaStream_t stream, bool overlap = false) {
    if (n_tile != 32 && n_tile != 64) n_tile = 128;
    const int mode_a = load_mode(a.A, a.a_row, a.a_k), mode_b = load_mode(a.B, a.b_row, a.b_k);
    // one main accumulator per four reduction blocks (chains of 16 additions), within 512 columns
    const int blocks = a.k_per_split / tc::kBlockK;
    int n_acc = (blocks + 3) / 4;
    if (n_acc > 512 / n_tile - 1) n_acc = 512 / n_tile - 1;
    a.n_acc = n_acc < 1 ? 1 : n_acc;
    TcKernel fn = nullptr;
    int smem;
    switch (n_tile) {
        case 32: fn = pick_tc<32>(mode_a, mode_b); smem = tc::SmemLayout<32>::kBytes; break;
        case 64: fn = pick_tc<64>(mode_a, mode_b); smem = tc::SmemLayout<64>::kBytes; break;
        default: fn = pick_tc<128>(mode_a, mode_b); smem = tc::SmemLayout<128>::kBytes; break;
    }
    DB_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int splits = a.k_per_split > 0 ? (a.K + a.k_per_split - 1) / a.k_per_split : 1;
    dim3 grid((a.N + n_tile - 1) / n_tile, (a.M + tc::kTileM - 1) / tc::kTileM, splits < 1 ? 1 : splits);
    OverlappedLaunch L(grid, dim3(tc::kThreads), smem, stream, overlap);
    DB_CUDA_TRY(cudaLaunchKernelEx(&L.cfg, fn, a));
    DB_CUDA_TRY(cudaGetLastError());
    return DB_OK;
}

bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

// defined below, beside the grouped entry point
db_status launch_logits_tma(const float* X, long long x_pitch, const float* W, long long w_pitch, float* partials,
                            long long o_split, long long o_n, int rows, int D, int C, int k_per_split, int n_tile,
                            int* status, bool first_of_call, cudaStream_t stream);
size_t grouped_workspace_total(long long rows, int K, int D, int C);
db_status worker_grad_tensor(const float* X, const int32_t* y, const float* W, const int32_t* offsets, int K, int D,
                             int C, float* const* G, float* losses, void* workspace, cudaStream_t stream);

}  // namespace
}  // namespace dynbatch

extern "C" db_status db_contract_f32(const float* A, int64_t a_row, int64_t a_k, const float* B, int64_t b_row,
                                     int64_t b_k, float* out, int64_t o_m, int64_t o_n, int32_t M, int32_t N,
                                     int32_t K, int32_t* status, void* cuda_stream) {
    using namespace dynbatch;
    if (!A || !B || !out || !status) return DB_ERR_NULL;
    if (M < 1 || N < 1 || K < 0) return DB_ERR_ARG;
    if (a_row < 0 || a_k < 0 || b_row < 0 || b_k < 0 || o_m < 1 || o_n < 1) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(A) % 4 || reinterpret_cast<uintptr_t>(B) % 4 ||
        reinterpret_cast<uintptr_t>(out) % 4 || reinterpret_cast<uintptr_t>(status) % 4)
        return DB_ERR_ARG;
    const int n_tile = N <= 32 ? 32 : (N <= 64 ? 64 : 128);
    const int k_round = K > 0 ? (K + tc::kBlockK - 1) / tc::kBlockK * tc::kBlockK : tc::kBlockK;
    // A contiguous along m, B along k, out along m: the layout of the logits, operands by TMA
    if (K > 0 && a_row == 1 && a_k % 4 == 0 && aligned16(A) && b_k == 1 && b_row % 4 == 0 && aligned16(B) && o_m == 1)
        return launch_logits_tma(B, b_row, A, a_k, out, 0, o_n, N, K, M, k_round, n_tile, status, false,
                                 static_cast<cudaStream_t>(cuda_stream));
    tc::GemmArgs a{};
    a.A = A; a.a_row = a_row; a.a_k = a_k;
    a.B = B; a.b_row = b_row; a.b_k = b_k;
    a.out = out; a.o_m = o_m; a.o_n = o_n; a.o_split = 0;
    a.M = M; a.N = N; a.K = K;
    a.k_per_split = k_round;
    a.status = status;
    return launch_tc_gemm(a, n_tile, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" size_t db_worker_grad_workspace_bytes(int32_t b_i, int32_t D, int32_t C) {
    using namespace dynbatch;
    if (!valid_shape(b_i, D, C)) return 0;
    const size_t f = layout_for(b_i, D, C).total();
    if (b_i > kMaxTensorCoreBatch) return f;
    const size_t t = grouped_workspace_total(b_i, 1, D, C);
    return t > f ? t : f;
}

extern "C" db_status db_worker_grad_ex(const float* X, const int32_t* y, const float* W, int32_t b_i,
                                       int32_t D, int32_t C, float* G, float* loss, void* workspace,
                                       size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    using namespace dynbatch;
    if (!X || !y || !W || !G || !workspace) return DB_ERR_NULL;
    if (!valid_shape(b_i, D, C)) return DB_ERR_ARG;
    if (flags & ~static_cast<uint32_t>(DB_WORKER_GRAD_FFMA)) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return DB_ERR_ARG;
    if (workspace_bytes < db_worker_grad_workspace_bytes(b_i, D, C)) return DB_ERR_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!(flags & DB_WORKER_GRAD_FFMA) && b_i <= kMaxTensorCoreBatch) {
        // the tensor-core path is the grouped one with a single worker
        const int32_t offsets[2] = {0, b_i};
        float* const out[1] = {G};
        return worker_grad_tensor(X, y, W, offsets, 1, D, C, out, loss, workspace, stream);
    }
    const WorkerLayout L = layout_for(b_i, D, C);

    char* base = static_cast<char*>(workspace);
    int* status = reinterpret_cast<int*>(base);
    float* partials = reinterpret_cast<float*>(base + kStatusBytes);
    float* E = reinterpret_cast<float*>(base + kStatusBytes + L.partial_bytes);
    float* row_loss = reinterpret_cast<float*>(base + kStatusBytes + L.partial_bytes + L.e_bytes);
    const long long bc = static_cast<long long>(b_i) * C;
    DB_CUDA_TRY(cudaMemsetAsync(status, 0, kStatusBytes, stream));

    // 1. logits, split over D
    {
        const bool vec4 = (D % 4 == 0) && (C % 4 == 0) && aligned16(X) && aligned16(W);
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
    RowGroups one{};
    one.K = 1;
    one.off[0] = 0;
    one.off[1] = b_i;
    {
        const db_status st = launch_softmax(partials, L.splits, bc, y, E, row_loss, one, b_i, C,
                                            reinterpret_cast<unsigned int*>(status) + 1, loss, stream, false);
        if (st != DB_OK) return st;
    }
    // 3. G = X^T E
    {
        const bool vec4 = (D % 4 == 0) && (C % 4 == 0) && aligned16(X) && aligned16(G);
        dim3 grid((C + kTile - 1) / kTile, (D + kTile - 1) / kTile, 1);
        if (vec4)
            tile_gemm_kernel<true, true><<<grid, kThreads, 0, stream>>>(X, D, E, C, G, C, 0, D, C, b_i, b_i);
        else
            tile_gemm_kernel<true, false><<<grid, kThreads, 0, stream>>>(X, D, E, C, G, C, 0, D, C, b_i, b_i);
        DB_CUDA_TRY(cudaGetLastError());
    }
    return DB_OK;
}

namespace dynbatch {
namespace {

struct GroupedLayout {
    int splits, k_per_split, n_tile;
    long long rows_p;            // rows of the split arrays: every worker padded to a multiple of 8 (upper bound)
    long long x_pitch, e_pitch;  // floats per row of the split arrays (multiples of 32: 128-byte rows)
    size_t header_bytes, partial_bytes, e_bytes, loss_bytes, xs_bytes, es_bytes;
    size_t total() const {
        return header_bytes + partial_bytes + e_bytes + loss_bytes + 2 * xs_bytes + 2 * es_bytes;
    }
};

long long round_up(long long x, long long m) { return (x + m - 1) / m * m; }

// All workers' rows go through one logits contraction (they share W); split over D for about one CTA per SM.
GroupedLayout grouped_layout(long long rows, int K, int D, int C) {
    GroupedLayout L;
    L.n_tile = rows <= 32 ? 32 : (rows <= 64 ? 64 : 128);
    const long long tiles = static_cast<long long>((C + tc::kTileM - 1) / tc::kTileM) * ((rows + L.n_tile - 1) / L.n_tile);
    long long s = sm_count() / tiles;
    const int kblocks = (D + tc::kBlockK - 1) / tc::kBlockK;
    if (s > kblocks) s = kblocks;
    if (s < 1) s = 1;
    const int per_blocks = static_cast<int>((kblocks + s - 1) / s);
    L.k_per_split = per_blocks * tc::kBlockK;
    L.splits = (D + L.k_per_split - 1) / L.k_per_split;
    L.rows_p = round_up(rows + 7LL * K, 8);
    L.x_pitch = round_up(D, 32);
    L.e_pitch = round_up(C, 32);
    L.header_bytes = round16(kStatusBytes + sizeof(unsigned int) * static_cast<size_t>(K));
    L.partial_bytes = round16(sizeof(float) * static_cast<size_t>(L.splits) * rows * C);
    L.e_bytes = round16(sizeof(float) * static_cast<size_t>(rows) * C);
    L.loss_bytes = round16(sizeof(float) * static_cast<size_t>(rows));
    L.xs_bytes = sizeof(float) * static_cast<size_t>(L.rows_p) * L.x_pitch;
    L.es_bytes = sizeof(float) * static_cast<size_t>(L.rows_p) * L.e_pitch;
    return L;
}

size_t grouped_workspace_total(long long rows, int K, int D, int C) { return grouped_layout(rows, K, D, C).total(); }

bool valid_group_shape(long long rows, int K, int D, int C) {
    return K >= 1 && K <= DB_MAX_K && rows >= K && rows <= (1 << 22) && D >= 1 && C >= 1;
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library needs no link against the driver.
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) !=
                cudaSuccess || q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor map of a row-major fp32 array [rows, cols] with `pitch` floats per row, read in boxes of
// box_rows rows x 32 columns; elements outside [rows, cols] read as zero.  Operands that are contiguous
// along the output index need the 128-byte swizzle of 32-byte pieces (the only one the tensor core takes
// for 32-bit operands in that orientation), operands contiguous along the reduction the ordinary one.
db_status make_operand_map(CUtensorMap* map, const float* base, long long rows, long long cols, long long pitch,
                           int box_rows, bool output_index_major) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) {
        record_message("cuTensorMapEncodeTiled is not available from this driver");
        return DB_ERR_CUDA;
    }
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch) * sizeof(float)};
    const cuuint32_t box[2] = {32, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t elem[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
                           CU_TENSOR_MAP_INTERLEAVE_NONE,
                           output_index_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        record_message("cuTensorMapEncodeTiled rejected an operand layout of the worker gradient");
        return DB_ERR_CUDA;
    }
    return DB_OK;
}

// Tensor map of a row-major fp32 array [rows, pitch] (pitch a multiple of 32 floats) seen as
// [pitch / 32 chunks][rows][32 floats]: the chunk stride (128 bytes) is smaller than the row stride, which
// the encoder accepts.  A box of {32, box_rows, box_chunks} lands in shared memory chunk-major, each
// chunk a [box_rows x 128 bytes] block with the 128-byte swizzle of 32-byte pieces; rows beyond `rows`
// read as zero.  Every column of the pitch must hold finite data or belong to an output that is never
// stored.
db_status make_chunked_map(CUtensorMap* map, const float* base, long long rows, long long pitch, int box_rows,
                           int box_chunks) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) {
        record_message("cuTensorMapEncodeTiled is not available from this driver");
        return DB_ERR_CUDA;
    }
    const cuuint64_t dims[3] = {32, static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(pitch / 32)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch) * sizeof(float), 128};
    const cuuint32_t box[3] = {32, static_cast<cuuint32_t>(box_rows), static_cast<cuuint32_t>(box_chunks)};
    const cuuint32_t elem[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, elem,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        record_message("cuTensorMapEncodeTiled rejected the chunked layout of a gradient operand");
        return DB_ERR_CUDA;
    }
    return DB_OK;
}

// out(n, c) = sum_d X(n, d) W(d, c) with both operands copied by TMA from where the caller left them
// (the logits; also db_contract_f32 for operands laid out that way).  Needs 16-byte aligned W and X and
// row pitches that are multiples of 4 floats; out(n, c) lands at out[split * o_split + n * o_n + c].
db_status launch_logits_tma(const float* X, long long x_pitch, const float* W, long long w_pitch, float* partials,
                            long long o_split, long long o_n, int rows, int D, int C, int k_per_split, int n_tile,
                            int* status, bool first_of_call, cudaStream_t stream) {
    tcl::LogitArgs a{};
    db_status st;
    if ((st = make_operand_map(&a.w, W, D, C, w_pitch, tcl::kBlockK, true)) != DB_OK) return st;
    if ((st = make_operand_map(&a.x, X, rows, D, x_pitch, n_tile, false)) != DB_OK) return st;
    a.o_n = o_n;
    a.out = partials; a.o_split = o_split; a.rows = rows; a.D = D; a.C = C; a.k_per_split = k_per_split;
    a.status = status;
    a.clear_status = first_of_call ? 1 : 0;
    // one main accumulator per four reduction blocks (chains of 16 additions), within 512 columns
    const int blocks = k_per_split / tcl::kBlockK;
    a.n_acc = std::min(std::max((blocks + 3) / 4, 1), 512 / n_tile - 1);
    const int splits = (D + k_per_split - 1) / k_per_split;
    dim3 grid((rows + n_tile - 1) / n_tile, (C + tcl::kTileM - 1) / tcl::kTileM, splits);
    void (*fn)(const tcl::LogitArgs) = nullptr;
    int smem = 0;
    switch (n_tile) {
        case 32: fn = tcl::logits_tma_kernel<32>; smem = tcl::Smem<32>::kBytes; break;
        case 64: fn = tcl::logits_tma_kernel<64>; smem = tcl::Smem<64>::kBytes; break;
        default: fn = tcl::logits_tma_kernel<128>; smem = tcl::Smem<128>::kBytes; break;
    }
    DB_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    // as the first kernel of a worker-gradient call it may be scheduled under whatever precedes the call
    OverlappedLaunch OL(grid, dim3(tcl::kThreads), smem, stream, first_of_call);
    DB_CUDA_TRY(cudaLaunchKernelEx(&OL.cfg, fn, a));
    DB_CUDA_TRY(cudaGetLastError());
    return DB_OK;
}

// The tensor-core path for K >= 1 workers; arguments already validated.
db_status worker_grad_tensor(const float* X, const int32_t* y, const float* W, const int32_t* offsets, int K, int D,
                             int C, float* const* G, float* losses, void* workspace, cudaStream_t stream) {
    const long long rows = offsets[K];
    const GroupedLayout L = grouped_layout(rows, K, D, C);
    char* base = static_cast<char*>(workspace);
    int* status = reinterpret_cast<int*>(base);
    char* cur = base + L.header_bytes;
    float* partials = reinterpret_cast<float*>(cur); cur += L.partial_bytes;
    float* E = reinterpret_cast<float*>(cur); cur += L.e_bytes;
    float* row_loss = reinterpret_cast<float*>(cur); cur += L.loss_bytes;
    float* x_hi = reinterpret_cast<float*>(cur); cur += L.xs_bytes;
    float* x_lo = reinterpret_cast<float*>(cur); cur += L.xs_bytes;
    float* e_hi = reinterpret_cast<float*>(cur); cur += L.es_bytes;
    float* e_lo = reinterpret_cast<float*>(cur);
    const long long rc = rows * C;

    RowGroups rg{};
    rg.K = K;
    for (int w = 0; w <= K; ++w) rg.off[w] = offsets[w];
    rg.poff[0] = 0;
    for (int w = 0; w < K; ++w) rg.poff[w + 1] = rg.poff[w] + static_cast<int>(round_up(offsets[w + 1] - offsets[w], 8));
    const long long rows_p = rg.poff[K];

    // Tile width of the gradient kernel: 128 classes while three main accumulators keep the chains short.
    int max_rows = 0;
    for (int w = 0; w < K; ++w) max_rows = std::max(max_rows, rg.poff[w + 1] - rg.poff[w]);
    const bool wide = max_rows <= tcg::kWideTileMaxRows;
    const int tile_n = wide ? 128 : 64;
    const int max_acc = wide ? tcg::Shape<128>::kMaxAcc : tcg::Shape<64>::kMaxAcc;
    const int grad_smem = wide ? tcg::Shape<128>::kSmemBytes : tcg::Shape<64>::kSmemBytes;
    void (*grad_fn)(const tcg::GradArgs) = wide ? tcg::grad_tma_kernel<128> : tcg::grad_tma_kernel<64>;

    tcg::GradArgs ga{};
    db_status st;
    if ((st = make_chunked_map(&ga.x_hi, x_hi, rows_p, L.x_pitch, tcg::kRowsPerStage, tcg::kAChunks)) != DB_OK) return st;
    if ((st = make_chunked_map(&ga.x_lo, x_lo, rows_p, L.x_pitch, tcg::kRowsPerStage, tcg::kAChunks)) != DB_OK) return st;
    if ((st = make_chunked_map(&ga.e_hi, e_hi, rows_p, L.e_pitch, tcg::kRowsPerStage, tile_n / tcg::kChunk)) != DB_OK) return st;
    if ((st = make_chunked_map(&ga.e_lo, e_lo, rows_p, L.e_pitch, tcg::kRowsPerStage, tile_n / tcg::kChunk)) != DB_OK) return st;
    // one main accumulator per four 32-sample blocks (chains of 16 additions), within the 512 columns
    const int max_blocks = (max_rows + tcg::kAccRows - 1) / tcg::kAccRows;
    ga.n_acc = std::min(std::max((max_blocks + 3) / 4, 1), max_acc);

    // largest batches first: their CTAs run longest and should not form the tail of the grid
    int order[DB_MAX_K];
    for (int w = 0; w < K; ++w) order[w] = w;
    std::stable_sort(order, order + K, [&](int u, int v) {
        return offsets[u + 1] - offsets[u] > offsets[v + 1] - offsets[v];
    });
    for (int z = 0; z < K; ++z) {
        const int w = order[z];
        ga.out[z] = G[w];
        ga.row0[z] = rg.poff[w];
        ga.steps[z] = (rg.poff[w + 1] - rg.poff[w]) / tcg::kStepRows;
    }
    // the tiles leave by TMA when every G_w allows it (16-byte aligned, rows a multiple of 16 bytes)
    ga.tma_store = C % 4 == 0;
    for (int z = 0; z < K && ga.tma_store; ++z) ga.tma_store = aligned16(ga.out[z]);
    for (int z = 0; z < K && ga.tma_store; ++z)
        if ((st = make_operand_map(&ga.out_map[z], ga.out[z], D, C, C, tcg::kTileM, false)) != DB_OK) return st;

    // Nothing has been enqueued up to here.  The status word is zeroed by the first CTA of the logits
    // kernel and the mean losses are folded by the gradient kernel, so the call is three launches and
    // nothing else.
    // 1. logits of every row, transposed orientation, split over D; operands by TMA where their
    //    alignment allows it, else through the register-converting contraction
    if (aligned16(W) && aligned16(X) && C % 4 == 0 && D % 4 == 0) {
        st = launch_logits_tma(X, D, W, C, partials, rc, C, static_cast<int>(rows), D, C, L.k_per_split, L.n_tile,
                               status, true, stream);
        if (st != DB_OK) return st;
    } else {
        tc::GemmArgs a{};
        a.A = W; a.a_row = 1; a.a_k = C;          // A(m = class, k = feature) = W[k, m]
        a.B = X; a.b_row = D; a.b_k = 1;          // B(n = sample, k = feature) = X[n, k]
        a.out = partials; a.o_m = 1; a.o_n = C; a.o_split = rc;   // Z[n, m], one slab per split
        a.M = C; a.N = static_cast<int>(rows); a.K = D; a.k_per_split = L.k_per_split; a.status = status;
        a.clear_status = 1;
        st = launch_tc_gemm(a, L.n_tile, stream);
        if (st != DB_OK) return st;
    }
    // 2. softmax residual with each worker's own 1/b, left split into TF32 halves beside the split X
    {
        SplitOut so{};
        so.e_hi = e_hi; so.e_lo = e_lo; so.e_pitch = L.e_pitch;
        so.X = X; so.x_hi = x_hi; so.x_lo = x_lo; so.x_pitch = L.x_pitch; so.D = D;
        so.x_vec = (D % 4 == 0) && aligned16(X);
        st = launch_softmax(partials, L.splits, rc, y, E, row_loss, rg, static_cast<int>(rows), C, nullptr, nullptr,
                            stream, true, &so);
        if (st != DB_OK) return st;
    }
    // 3. one gradient per worker: G_w = X_w^T E_w, reduction over that worker's rows only
    {
        ga.D = D; ga.C = C; ga.status = status;
        ga.row_loss = losses ? row_loss : nullptr;
        for (int z = 0; z < K && losses; ++z) {
            const int w = order[z];
            ga.loss_out[z] = losses + w;
            ga.loss_row0[z] = offsets[w];
            ga.loss_rows[z] = offsets[w + 1] - offsets[w];
        }
        DB_CUDA_TRY(cudaFuncSetAttribute(grad_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, grad_smem));
        dim3 grid((C + tile_n - 1) / tile_n, (D + tcg::kTileM - 1) / tcg::kTileM, K);
        OverlappedLaunch OL(grid, dim3(tcg::kThreads), grad_smem, stream, true);
        DB_CUDA_TRY(cudaLaunchKernelEx(&OL.cfg, grad_fn, ga));
        DB_CUDA_TRY(cudaGetLastError());
    }
    return DB_OK;
}

}  // namespace
}  // namespace dynbatch

extern "C" size_t db_worker_grad_grouped_workspace_bytes(int32_t total_rows, int32_t K, int32_t D, int32_t C) {
    using namespace dynbatch;
    if (!valid_group_shape(total_rows, K, D, C)) return 0;
    return grouped_layout(total_rows, K, D, C).total();
}

extern "C" db_status db_worker_grad_grouped(const float* X, const int32_t* y, const float* W,
                                            const int32_t* offsets, int32_t K, int32_t D, int32_t C,
                                            float* const* G, float* losses, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream) {
    using namespace dynbatch;
    if (!X || !y || !W || !offsets || !G || !workspace) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || D < 1 || C < 1) return DB_ERR_ARG;
    if (offsets[0] != 0) return DB_ERR_ARG;
    for (int w = 0; w < K; ++w) {
        const long long bw = static_cast<long long>(offsets[w + 1]) - offsets[w];
        if (bw < 1) return DB_ERR_ARG;                         // every worker holds at least one sample
        if (bw > kMaxTensorCoreBatch) return DB_ERR_UNSUPPORTED;
        if (!G[w]) return DB_ERR_NULL;
    }
    const long long rows = offsets[K];
    if (!valid_group_shape(rows, K, D, C)) return DB_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return DB_ERR_ARG;
    if (workspace_bytes < grouped_layout(rows, K, D, C).total()) return DB_ERR_ARG;
    return worker_grad_tensor(X, y, W, offsets, K, D, C, G, losses, workspace, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" db_status db_worker_grad(const float* X, const int32_t* y, const float* W, int32_t b_i,
                                    int32_t D, int32_t C, float* G, float* loss, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream) {
    return db_worker_grad_ex(X, y, W, b_i, D, C, G, loss, workspace, workspace_bytes, 0, cuda_stream);
}
