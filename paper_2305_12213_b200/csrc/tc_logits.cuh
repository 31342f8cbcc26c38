// The logits of the linear-softmax model on the tensor cores, fed by TMA (sm_100a):
//     Z(n, c) = sum_d X(n, d) * W(d, c)         computed transposed, 128 classes x N_TILE samples per CTA,
// the feature dimension split over blockIdx.z; split z writes its partial sums to out + z * o_split.
//
// Both operands are read where the caller left them, as plain fp32:
//   - W ([D, C] row-major) has the reduction index d as its row, so a class tile is contiguous along
//     the OUTPUT index: tcgen05.mma takes it in that orientation (see tc_grad.cuh for the layout rules
//     of 32-bit operands), from TMA boxes of 32 features x 32 classes;
//   - X ([rows, D] row-major) is contiguous along the reduction: the ordinary orientation, one TMA box
//     of N_TILE samples x 32 features with the 128-byte swizzle.
// The tensor core reads only the upper 19 bits of a 32-bit TF32 operand (measured: raw fp32 gives
// results bit-identical to x & 0xFFFFE000), so a copied tile already is its own hi half; eight warps
// add the lo half, lo = tf32(x - hi), element-wise into a second tile with the same layout, and the
// usual three products per fp32 product follow (lo*hi + hi*lo into one accumulator, hi*hi round-robin
// into the others: tc_gemm.cuh explains why).
//
// 320 threads: warps 0-7 derive the lo halves and later drain the accumulators, warp 8 owns tensor
// memory and (one lane) issues the products, warp 9 issues the copies: five lanes, one box each, in
// the same instruction (measured: a further box costs about half as much that way as from the same
// thread, and an iteration of the copy loop costs 0.3 us before its first box).  Before the CTA
// waits for its predecessor, its threads ask the L2 to prefetch every box of its share of W and X, one
// box each, so that the ring of three stages meets L2 latencies, not DRAM's (issued in a row by the
// copying warp these requests delayed its first copy by 1.6 us; issued after the wait instead of
// before it the step behind a running predecessor took 0.85 us longer).
// Every wait is bounded as in tc_gemm.cuh.
#pragma once
#include <cuda.h>

#include "tc_gemm.cuh"

namespace dynbatch {
namespace tcl {

constexpr int kTileM = 128;            // classes per CTA = tensor-memory lanes
constexpr int kBlockK = 32;            // features per stage
constexpr int kStages = 3;
constexpr int kSplitWarps = 8;
constexpr int kSplitThreads = kSplitWarps * 32;
constexpr int kThreads = kSplitThreads + 64;
constexpr int kAChunks = kTileM / 32;                      // 32-class column chunks of the W tile
constexpr int kAChunkBytes = kBlockK * 128;                // one [32 features x 32 classes] box
constexpr int kABytes = kAChunks * kAChunkBytes;           // 16 KB: the W tile of a stage (hi); lo follows

template <int N_TILE>
struct Smem {
    static constexpr int kBBytes = N_TILE * 128;           // the X tile of a stage (hi); lo follows
    static constexpr int kStage = 2 * kABytes + 2 * kBBytes;
    static constexpr int kCopy = kABytes + kBBytes;        // what the TMA delivers per stage
    static constexpr int kBytes = kStages * kStage + 1024; // + slack for 1024-byte alignment
};

struct LogitArgs {
    CUtensorMap w;                 // [D, C] fp32, boxes of 32 rows x 32 columns, 128-byte swizzle of 32-byte pieces
    CUtensorMap x;                 // [rows, D] fp32, boxes of N_TILE rows x 32 columns, 128-byte swizzle
    float* out;                    // Z(n, c) at out[split * o_split + n * o_n + c]
    long long o_split, o_n;
    int rows, D, C;
    int k_per_split;               // multiple of 32
    int n_acc;                     // main accumulators, (n_acc + 1) * N_TILE <= 512
    int* status;
    int clear_status;              // non-zero: the first CTA zeroes *status before any wait can set it
};

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tc::smem_u32(bar)), "r"(bytes)
                 : "memory");
}
// One box of a 2-D tensor map into shared memory; x counts elements of the contiguous dimension and
// must be a multiple of 4 (16 bytes).  Coordinates outside the tensor read as zero.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(tc::smem_u32(bar)) : "memory");
}
// Ask the L2 to fetch a box; nothing waits for it.
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y) : "memory");
}

// W tile: output-index-major, 128-byte swizzle of 32-byte pieces (layout type 1), 4 reduction rows per
// 512-byte group, the next 32 classes kAChunkBytes further.
__device__ __forceinline__ uint64_t smem_desc_w(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(kAChunkBytes >> 4) << 16;
    d |= static_cast<uint64_t>(512 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(1) << 61;
    return d;
}
// fp32 accumulator, TF32 operands, A output-index-major (bit 15), B reduction-major, M x N tile.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (static_cast<uint32_t>(N >> 3) << 17) |
           (static_cast<uint32_t>(M >> 4) << 24);
}

// grid: (ceil(rows / N_TILE), ceil(C / 128), splits of D)
template <int N_TILE>
__global__ void __launch_bounds__(kThreads, 1)
logits_tma_kernel(const __grid_constant__ LogitArgs g) {
    using L = Smem<N_TILE>;
    static_assert(N_TILE == 32 || N_TILE == 64 || N_TILE == 128, "accumulator columns: power of two >= 32");
    static_assert(L::kCopy / 16 % kSplitThreads == 0, "whole 16-byte pieces per splitting thread");
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];     // a stage's copies have landed
    __shared__ __align__(8) uint64_t split_bar[kStages];    // its lo halves are in place
    __shared__ __align__(8) uint64_t empty_bar[kStages];    // the products reading it have finished
    __shared__ __align__(8) uint64_t done_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    unsigned char* ring = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * N_TILE, m0 = blockIdx.y * kTileM;
    const int k_begin = blockIdx.z * g.k_per_split;
    const int k_end = min(g.D, k_begin + g.k_per_split);
    const int nkb = (k_end - k_begin + kBlockK - 1) / kBlockK;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(&full_bar[s], 1);
            tc::mbar_init(&split_bar[s], kSplitWarps);
            tc::mbar_init(&empty_bar[s], 1);
        }
        tc::mbar_init(&done_bar, 1);
        tc::fence_barrier_init();
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&g.w)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&g.x)) : "memory");
    }
    const uint32_t tmem_cols = tc::tmem_columns((g.n_acc + 1) * N_TILE);
    if (warp == kSplitWarps) tc::tmem_alloc(&tmem_base_slot, tmem_cols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // The successor (the softmax kernel) splits X into the workspace before its own wait.  It may be
    // scheduled only once every kernel before this one has finished -- an earlier call's gradient kernel
    // may still be reading those arrays -- so the trigger comes after the wait, not before it.
    // Before the wait, while the predecessor may still run: ask the L2 for every box of W and X this CTA will
    // copy, one box per thread (a TMA instruction costs its thread 0.2 - 0.4 us, measured, so they are issued side
    // by side rather than in a row by the copying warp).  A prefetch consumes no data and needs no ordering
    // against whoever may still be writing W; the three-stage ring then meets L2 latency instead of DRAM's.
    if (tid < nkb * kAChunks)
        tma_prefetch_2d(&g.w, m0 + (tid % kAChunks) * 32, k_begin + (tid / kAChunks) * kBlockK);
    else if (tid < nkb * kAChunks + nkb && tid < kSplitThreads)
        tma_prefetch_2d(&g.x, k_begin + (tid - nkb * kAChunks) * kBlockK, n0);
    tc::griddep_wait();
    tc::griddep_launch_dependents();
    // a time-out needs seconds, this store comes microseconds after the launch: no wait can have given up yet
    if (g.clear_status && tid == 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) *g.status = 0;

    if (warp == kSplitWarps + 1) {
        // ------------------------------------------------------------ TMA copies: lanes 0-3 a W chunk each, lane 4 X
        const bool is_w = lane < kAChunks;
        const CUtensorMap* map = is_w ? &g.w : &g.x;
        const uint32_t box_off = is_w ? lane * kAChunkBytes : 2 * kABytes;
        int issued = 0;
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kStages;
            int ok = 1;
            if (lane == 0) {
                if (kb >= kStages)
                    ok = tc::mbar_wait(&empty_bar[s], ((kb / kStages) - 1) & 1, &abort_flag, g.status, 4);
                if (abort_flag) ok = 0;
                if (ok) mbar_expect_tx(&full_bar[s], L::kCopy);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const int k0 = k_begin + kb * kBlockK;
            if (lane <= kAChunks) {
                const uint32_t dst = tc::smem_u32(ring + s * L::kStage) + box_off;
                if (is_w) tma_load_2d(dst, map, m0 + lane * 32, k0, &full_bar[s]);      // {class, feature}
                else tma_load_2d(dst, map, k0, n0, &full_bar[s]);                        // {feature, sample}
            }
            __syncwarp();
            issued = kb + 1;
        }
        if (lane == 0) {
            // the copies issued last write into this CTA's shared memory until they land: see them
            // complete (bounded) before this thread lets the CTA exit, whatever the other roles do
            for (int kb = max(0, issued - kStages); kb < issued; ++kb) {
                const unsigned long long t0 = tc::global_ns();
                while (!tc::mbar_try_wait(&full_bar[kb % kStages], (kb / kStages) & 1) &&
                       tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            }
        }
    } else if (warp == kSplitWarps) {
        // ------------------------------------------------------------ tensor-core issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kTileM, N_TILE);
            const uint32_t acc_cross = tmem_base + g.n_acc * N_TILE;
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int s = kb % kStages;
                alive = tc::mbar_wait(&split_bar[s], (kb / kStages) & 1, &abort_flag, g.status, 2);
                if (!alive) break;
                tc::tc_fence_after();
                const uint32_t st = tc::smem_u32(ring + s * L::kStage);
                const uint64_t a_hi = smem_desc_w(st), a_lo = smem_desc_w(st + kABytes);
                const uint64_t b_hi = tc::smem_desc_k_sw128(st + 2 * kABytes);
                const uint64_t b_lo = tc::smem_desc_k_sw128(st + 2 * kABytes + L::kBBytes);
                const uint32_t acc_main = tmem_base + (kb % g.n_acc) * N_TILE;
#pragma unroll
                for (int ks = 0; ks < kBlockK / 8; ++ks) {
                    const uint64_t a_adv = static_cast<uint64_t>((ks * 8 * 128) >> 4);   // 8 feature rows of 128 bytes
                    const uint64_t b_adv = static_cast<uint64_t>((ks * 8 * 4) >> 4);     // 8 features = 32 bytes along the row
                    tc::mma_tf32(acc_cross, a_lo + a_adv, b_hi + b_adv, idesc, (kb | ks) != 0);
                    tc::mma_tf32(acc_cross, a_hi + a_adv, b_lo + b_adv, idesc, 1);
                    tc::mma_tf32(acc_main, a_hi + a_adv, b_hi + b_adv, idesc, (kb >= g.n_acc) || ks != 0);
                }
                tc::mma_commit(&empty_bar[s]);
            }
            tc::mma_commit(&done_bar);
            if (!alive) {
                const unsigned long long t0 = tc::global_ns();
                while (!tc::mbar_try_wait(&done_bar, 0) && tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            }
            tc::tc_fence_before();
        }
    } else {
        // ------------------------------------------------------------ lo halves, then the epilogue
        bool alive = true;
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kStages;
            // the decision is made the same for the whole warp: what follows has warp-wide operations
            alive = __all_sync(0xffffffffu, tc::mbar_wait(&full_bar[s], (kb / kStages) & 1, &abort_flag, g.status, 8));
            if (!alive) break;
            unsigned char* st = ring + s * L::kStage;
            // element-wise, so neither swizzle matters: a lo tile mirrors its hi tile's layout
            constexpr int kPer = L::kCopy / 16 / kSplitThreads;
            float4 v[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int i = tid + j * kSplitThreads;
                v[j] = *reinterpret_cast<const float4*>(
                    i < kABytes / 16 ? st + i * 16 : st + 2 * kABytes + (i - kABytes / 16) * 16);
            }
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int i = tid + j * kSplitThreads;
                unsigned char* dst = i < kABytes / 16 ? st + kABytes + i * 16
                                                      : st + 2 * kABytes + L::kBBytes + (i - kABytes / 16) * 16;
                float4 lo;     // hi is what the tensor core sees of v: the value without its 13 low mantissa bits
                lo.x = tc::round_tf32(v[j].x - __uint_as_float(__float_as_uint(v[j].x) & 0xFFFFE000u));
                lo.y = tc::round_tf32(v[j].y - __uint_as_float(__float_as_uint(v[j].y) & 0xFFFFE000u));
                lo.z = tc::round_tf32(v[j].z - __uint_as_float(__float_as_uint(v[j].z) & 0xFFFFE000u));
                lo.w = tc::round_tf32(v[j].w - __uint_as_float(__float_as_uint(v[j].w) & 0xFFFFE000u));
                *reinterpret_cast<float4*>(dst) = lo;
            }
            tc::fence_proxy_async_smem();        // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&split_bar[s]);
        }
        if (alive && nkb > 0) alive = tc::mbar_wait(&done_bar, 0, &abort_flag, g.status, 3);
        alive = __all_sync(0xffffffffu, alive);      // tcgen05.ld below is a warp-wide instruction
        tc::tc_fence_after();
        if (alive) {
            // warp w may read tensor-memory lanes 32 (w mod 4) .. +31; the two warps that share a lane
            // quarter take alternate 32-column chunks.  Lanes are consecutive classes: coalesced stores.
            const int quarter = warp & 3;
            const int m = m0 + quarter * 32 + lane;
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            float* obase = g.out + static_cast<long long>(blockIdx.z) * g.o_split + m;
            const int used = min(g.n_acc, nkb);
#pragma unroll 1
            for (int c0 = (warp >> 2) * 32; c0 < N_TILE; c0 += 32 * (kSplitWarps / 4)) {
                uint32_t r[32];
                if (nkb > 0) {
                    uint32_t x[32];
                    __syncwarp();
                    tc::tmem_load32(lane_base + g.n_acc * N_TILE + c0, r);
                    for (int a = used - 1; a >= 0; --a) {
                        tc::tmem_load32(lane_base + a * N_TILE + c0, x);
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(x[j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                const int n_first = n0 + c0;
                if (m >= g.C || n_first >= g.rows) continue;
                float* col = obase + static_cast<long long>(n_first) * g.o_n;
                const int n_left = g.rows - n_first;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < n_left) *col = __uint_as_float(r[j]);
                    col += g.o_n;
                }
            }
        }
        tc::tc_fence_before();
    }
    __syncthreads();
    if (warp == kSplitWarps) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace tcl
}  // namespace dynbatch
