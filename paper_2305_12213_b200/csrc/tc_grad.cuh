// The ragged gradient contraction on the tensor cores, fed by TMA (sm_100a):
//     G_w(d, c) = sum_{r in worker w} X(r, d) * E(r, c)          for every worker w in one launch
// X ([rows, D]) and E ([rows, C]) are row-major with the reduction index r as the row, so both
// operands are contiguous along their OUTPUT index.  tcgen05.mma reads such "MN-major" tiles
// directly, which removes the transposition through registers that the general contraction in
// tc_gemm.cuh has to do; what is left of the operand preparation, the split of every fp32 value
// into two TF32 halves, is done once by the kernel that produces E (and copies X), not once per
// output tile.  A CTA of this kernel therefore only
//   - copies boxes of 16 rows of the four split arrays (X_hi, X_lo, E_hi, E_lo) into shared memory
//     with cp.async.bulk.tensor (128-byte swizzle of 32-byte pieces, completion on an mbarrier),
//   - issues three tcgen05.mma.kind::tf32 per 8 rows (lo*hi + hi*lo into one accumulator in tensor
//     memory, hi*hi round-robin into the others, see tc_gemm.cuh for why), and
//   - drains the accumulators and writes its 128 x TILE_N tile of G: through shared memory in the
//     box layout of a TMA store when G is 16-byte aligned with rows of a multiple of 16 bytes, else
//     as whole rows with ordinary stores.
// In the split arrays every worker's rows start at a multiple of 8 and are padded with zero rows to
// a multiple of 8, the reduction depth of one TF32 product.
//
// The tile is 128 x 128 where the accumulator chains allow it (batches up to 1024 rows: three main
// accumulators; two thirds of the operand traffic of 128 x 64 tiles and 1.4 us less on the step of the
// 256-sample check model), else 128 x 64 with up to seven accumulators.
//
// 320 threads: warp 0 (one lane) issues the TMA copies, warp 1 owns the tensor-memory allocation
// and (one lane) issues the products, warps 2-9 are the epilogue (two per tensor-memory lane quarter,
// half of the tile's columns each: 0.35 us less on the step than four warps; sending each 32-column box off as
// soon as it is staged, instead of the whole tile at once, gained nothing).  Three shared-memory stages of
// 16 samples; two (wide tile) or three CTAs fit on an SM and their phases (copy, products, epilogue)
// overlap.  Measured with a time stamp per phase, a CTA is a chain of latencies rather than a stream:
// 1 us from the predecessor's end to the first copy instruction, 1 - 2 us until the first stage has
// landed, about 0.5 us per stage after that, and 2 us to drain and store a tile.  Leaving out, in turn,
// the copies, the products or the stores shortened the step by 1 - 3 us each; none of them is the
// bound.  A persistent one-CTA-per-SM form with the roles fully decoupled (five stages, two
// accumulator sets, staging tile of its own, items dealt to the least-loaded CTA), one with four
// copying warps and one that copied X and E as plain fp32 and derived the lo halves in shared memory
// (half the L2 traffic) all took as long or longer, and are not kept.  Every wait is bounded (see
// tc_gemm.cuh); on a time-out the copy thread waits, again bounded, for the copies it has in flight
// before the CTA returns.
#pragma once
#include <cuda.h>

#include "tc_gemm.cuh"

namespace dynbatch {
namespace tcg {

constexpr int kTileM = 128;            // features per CTA = tensor-memory lanes
constexpr int kChunk = 32;             // fp32 per 128-byte swizzled row
constexpr int kStepRows = 8;           // reduction depth of one TF32 product
constexpr int kRowsPerStage = 16;      // samples per stage: two products' worth
constexpr int kAccRows = 32;           // consecutive samples whose hi*hi products share an accumulator turn
constexpr int kStages = 3;
constexpr int kChunkBytes = kRowsPerStage * 128;            // one [16 x 32] block of a stage
constexpr int kAChunks = kTileM / kChunk;
constexpr int kABytes = kAChunks * kChunkBytes;             // X_hi (or X_lo) part of a stage
constexpr int kEpilogueWarps = 8;      // two per tensor-memory lane quarter, half of the tile's columns each
constexpr int kEpilogueThreads = kEpilogueWarps * 32;
constexpr int kThreads = 64 + kEpilogueThreads;

// Sizes that follow from the tile width (classes per CTA = accumulator columns).
template <int TILE_N>
struct Shape {
    static constexpr int kBChunks = TILE_N / kChunk;
    static constexpr int kBBytes = kBChunks * kChunkBytes;              // E_hi (or E_lo) part of a stage
    static constexpr int kStageBytes = 2 * kABytes + 2 * kBBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024;     // + slack for 1024-byte alignment
    static constexpr int kMaxAcc = 512 / TILE_N - 1;                    // main accumulators beside the cross-term one
    static constexpr int kStagePitch = TILE_N + 4;                      // floats per row of the output staging tile
    static_assert(kTileM * kStagePitch * 4 <= kStages * kStageBytes, "output staging fits in the operand stages");
    static_assert(kTileM * TILE_N * 4 <= kStages * kStageBytes, "so does the tile in the TMA store's box layout");
};
constexpr int kWideTileMaxRows = 1024;  // 128-column tiles have three main accumulators: chains of <= 1024 / 3 rows

struct GradArgs {
    // The split arrays seen as [32-column chunk][row][32 floats] (the chunk stride, 128 bytes, is smaller than
    // the row stride), 128-byte swizzle of 32-byte pieces: one box of {32, 16 rows, n chunks} fills the
    // chunk-major tile of a stage with a single copy instruction.
    CUtensorMap x_hi, x_lo;        // [padded rows, D], boxes of 4 chunks
    CUtensorMap e_hi, e_lo;        // [padded rows, C], boxes of TILE_N / 32 chunks
    // slot z (blockIdx.z): the workers by falling row count, so that the longest CTAs start first
    float* out[DB_MAX_K];          // G of the worker in slot z, [D, C] row-major
    int tma_store;                 // every G is 16-byte aligned and C % 4 == 0: out_map[] is valid, tiles leave by TMA
    CUtensorMap out_map[DB_MAX_K]; // G as [D, C], boxes of 128 rows x 32 columns, 128-byte swizzle
    int row0[DB_MAX_K];            // first row of the worker in the split arrays (multiple of 8)
    int steps[DB_MAX_K];           // its padded row count / 8
    int D, C;
    int n_acc;                     // main accumulators in use, 1..kMaxAcc
    int* status;
    // mean loss of the worker in slot z = (sum of row_loss[loss_row0[z] .. + loss_rows[z])) / loss_rows[z],
    // written to loss_out[z] by the CTA with blockIdx.x == blockIdx.y == 0; row_loss == nullptr: not wanted
    const float* row_loss;
    float* loss_out[DB_MAX_K];
    int loss_row0[DB_MAX_K];
    int loss_rows[DB_MAX_K];
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

// One box of a 3-D tensor map; x (elements of the contiguous dimension) must be a multiple of 4.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(tc::smem_u32(bar)) : "memory");
}

// One box from shared memory to a 2-D tensor map (rows and columns outside the tensor are not written),
// as part of the thread's current bulk group.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until the bulk groups of this thread have finished READING shared memory.
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Shared-memory matrix descriptor of an operand stored output-index-major.  For 32-bit elements the
// tensor core accepts this orientation only with the 128-byte swizzle that permutes 32-byte pieces
// (layout type 1; the TMA mode of the same name writes it): 32 consecutive output indices form a
// 128-byte row, 4 reduction rows a 512-byte swizzle group.  The next 32 output indices start
// kChunkBytes further (leading byte offset), the next 4 reduction rows 512 bytes further (stride
// byte offset); one product consumes two such groups.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(kChunkBytes >> 4) << 16;
    d |= static_cast<uint64_t>(512 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(1) << 61;
    return d;
}
// fp32 accumulator, TF32 operands, both output-index-major (bits 15 and 16), M x N tile.
__host__ __device__ constexpr uint32_t instr_desc_tf32_mn(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
           (static_cast<uint32_t>(M >> 4) << 24);
}

// Barrier 1 over the epilogue threads that also ANDs a predicate: the same answer in every thread.
__device__ __forceinline__ bool epilogue_all(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out) : "r"(static_cast<uint32_t>(pred)), "n"(kEpilogueThreads) : "memory");
    return out != 0;
}

// Ask for a tensor map to be fetched into the descriptor cache before its first use.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// grid: (ceil(C / TILE_N), ceil(D / 128), workers)
template <int TILE_N>
__global__ void __launch_bounds__(kThreads)
grad_tma_kernel(const __grid_constant__ GradArgs g) {
    using S = Shape<TILE_N>;
    constexpr int kStageBytes = S::kStageBytes, kBBytes = S::kBBytes, kStagePitch = S::kStagePitch;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];     // a stage's copies have landed
    __shared__ __align__(8) uint64_t empty_bar[kStages];    // the products reading it have finished
    __shared__ __align__(8) uint64_t done_bar;              // all products have finished
    __shared__ __align__(8) uint64_t drain_bar;             // after a time-out: what had been issued has finished
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    unsigned char* tiles = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int z = blockIdx.z;
    // read from the parameter block before the wait for the previous kernel, not after it
    const int steps = g.steps[z], first_row = g.row0[z];
    const int loads = (steps * kStepRows + kRowsPerStage - 1) / kRowsPerStage;
    const int m0 = blockIdx.y * kTileM, n0 = blockIdx.x * TILE_N;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(&full_bar[s], 1);
            tc::mbar_init(&empty_bar[s], 1);
        }
        tc::mbar_init(&done_bar, 1);
        tc::mbar_init(&drain_bar, 1);
        tc::fence_barrier_init();
        prefetch_tensormap(&g.x_hi);
        prefetch_tensormap(&g.x_lo);
        prefetch_tensormap(&g.e_hi);
        prefetch_tensormap(&g.e_lo);
    }
    const uint32_t tmem_cols = tc::tmem_columns((g.n_acc + 1) * TILE_N);
    if (warp == 1) tc::tmem_alloc(&tmem_base_slot, tmem_cols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // everything above overlaps the kernel that writes the split operands
    tc::griddep_launch_dependents();
    tc::griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA copies
        if (lane == 0) {
            int issued = 0;
            for (int l = 0; l < loads; ++l) {
                const int s = l % kStages;
                if (l >= kStages &&
                    !tc::mbar_wait(&empty_bar[s], ((l / kStages) - 1) & 1, &abort_flag, g.status, 4))
                    break;
                if (abort_flag) break;
                mbar_expect_tx(&full_bar[s], kStageBytes);
                const uint32_t dst = tc::smem_u32(tiles + s * kStageBytes);
                const int row = first_row + l * kRowsPerStage;
                tma_load_3d(dst, &g.x_hi, 0, row, m0 / kChunk, &full_bar[s]);
                tma_load_3d(dst + kABytes, &g.x_lo, 0, row, m0 / kChunk, &full_bar[s]);
                tma_load_3d(dst + 2 * kABytes, &g.e_hi, 0, row, n0 / kChunk, &full_bar[s]);
                tma_load_3d(dst + 2 * kABytes + kBBytes, &g.e_lo, 0, row, n0 / kChunk, &full_bar[s]);
                issued = l + 1;
            }
            // the copies issued last write into this CTA's shared memory until they land: see them
            // complete (bounded) before this thread lets the CTA exit, whatever the other roles do
            for (int l = max(0, issued - kStages); l < issued; ++l) {
                const unsigned long long t0 = tc::global_ns();
                while (!tc::mbar_try_wait(&full_bar[l % kStages], (l / kStages) & 1) &&
                       tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            }
        }
        // the worker's mean loss: its per-sample losses were written by the kernel before this one
        if (g.row_loss != nullptr && g.loss_out[z] != nullptr && blockIdx.x == 0 && blockIdx.y == 0) {
            __syncwarp();
            const float* rl = g.row_loss + g.loss_row0[z];
            float part = 0.0f;
            for (int r = lane; r < g.loss_rows[z]; r += 32) part += __ldcg(rl + r);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
            if (lane == 0) *g.loss_out[z] = part / static_cast<float>(g.loss_rows[z]);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ tensor-core issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_tf32_mn(kTileM, TILE_N);
            const uint32_t acc_cross = tmem_base + g.n_acc * TILE_N;
            bool alive = true;
            for (int l = 0; l < loads && alive; ++l) {
                const int s = l % kStages;
                alive = tc::mbar_wait(&full_bar[s], (l / kStages) & 1, &abort_flag, g.status, 5);
                if (!alive) break;
                tc::tc_fence_after();
                const uint32_t st = tc::smem_u32(tiles + s * kStageBytes);
                const int blk = l * kRowsPerStage / kAccRows;          // which 32-sample block
                const bool blk_start = (l * kRowsPerStage) % kAccRows == 0;
                const uint32_t acc_main = tmem_base + (blk % g.n_acc) * TILE_N;
                const int here = min(kRowsPerStage / kStepRows, steps - l * (kRowsPerStage / kStepRows));
                for (int q = 0; q < here; ++q) {
                    const uint32_t off = q * 1024;      // 8 rows of 128 bytes
                    const uint64_t a_hi = smem_desc_mn_sw128(st + off);
                    const uint64_t a_lo = smem_desc_mn_sw128(st + kABytes + off);
                    const uint64_t b_hi = smem_desc_mn_sw128(st + 2 * kABytes + off);
                    const uint64_t b_lo = smem_desc_mn_sw128(st + 2 * kABytes + kBBytes + off);
                    tc::mma_tf32(acc_cross, a_lo, b_hi, idesc, (l | q) != 0);
                    tc::mma_tf32(acc_cross, a_hi, b_lo, idesc, 1);
                    tc::mma_tf32(acc_main, a_hi, b_hi, idesc, blk >= g.n_acc || !blk_start || q != 0);
                }
                tc::mma_commit(&empty_bar[s]);
            }
            if (alive) tc::mma_commit(&done_bar);
            if (!alive) {
                // a wait gave up somewhere in the CTA: see, bounded, what had been issued finish before the
                // tensor memory is freed
                tc::mma_commit(&drain_bar);
                const unsigned long long t0 = tc::global_ns();
                while (!tc::mbar_try_wait(&drain_bar, 0) && tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            }
            tc::tc_fence_before();
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int et = tid - 64;                     // 0..255
        const int quarter = warp & 3;                // the tensor-memory lanes this warp may read
        const int col_half = (warp - 2) >> 2;        // which half of the tile's columns it drains
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const int row = quarter * 32 + lane;
        float* srow = reinterpret_cast<float*>(tiles) + row * kStagePitch;
        // the decision is made the same for all eight warps (a barrier that ANDs their predicates): what
        // follows has warp-wide instructions and a barrier among them
        if (epilogue_all(tc::mbar_wait(&done_bar, 0, &abort_flag, g.status, 6))) {
            tc::tc_fence_after();
            const int used = min(g.n_acc, (steps * kStepRows + kAccRows - 1) / kAccRows);
#pragma unroll 1
            for (int c0 = col_half * (TILE_N / 2); c0 < (col_half + 1) * (TILE_N / 2); c0 += 32) {
                uint32_t r[32], x[32];
                __syncwarp();
                tc::tmem_load32(lane_base + g.n_acc * TILE_N + c0, r);
                for (int a = used - 1; a >= 0; --a) {
                    tc::tmem_load32(lane_base + a * TILE_N + c0, x);
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(x[j]));
                }
                if (g.tma_store) {
                    // the box layout of the store: [32-column block][128 rows][128 bytes], 16-byte pieces
                    // permuted by the row's low three bits (which also keeps these stores conflict-free)
                    unsigned char* box = tiles + (c0 / 32) * (kTileM * 128) + row * 128;
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(box + (((j >> 2) ^ (row & 7)) << 4)) =
                            make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                        __uint_as_float(r[j + 3]));
                } else {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(srow + c0 + j) =
                            make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                        __uint_as_float(r[j + 3]));
                }
            }
            if (g.tma_store) tc::fence_proxy_async_smem();    // the TMA engine reads what these threads wrote
            tc::tc_fence_before();                            // the accumulators have been read
            asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
            if (g.tma_store) {
                if (et == 0) {
#pragma unroll
                    for (int h = 0; h < TILE_N / 32; ++h)
                        if (n0 + h * 32 < g.C)
                            tma_store_2d(&g.out_map[z], n0 + h * 32, m0, tc::smem_u32(tiles + h * (kTileM * 128)));
                    bulk_commit();
                    bulk_wait_read();      // shared memory must stay until the engine has read the tile
                }
            } else {
                // whole rows of the tile, TILE_N / 4 threads per row
                const float* stage = reinterpret_cast<const float*>(tiles);
                float* obase = g.out[z];
                const int rows = min(kTileM, g.D - m0), cols = min(TILE_N, g.C - n0);
                constexpr int kVecPerRow = TILE_N / 4;
                constexpr int kRowsPerPass = kEpilogueThreads / kVecPerRow;
                const int vcol = (et % kVecPerRow) * 4, rsub = et / kVecPerRow;
                const bool vec_ok = (g.C % 4 == 0) && (reinterpret_cast<uintptr_t>(obase) % 16 == 0);
                for (int r0 = 0; r0 < rows; r0 += kRowsPerPass) {
                    const int rr = r0 + rsub;
                    if (rr >= rows || vcol >= cols) continue;
                    const float4 val = *reinterpret_cast<const float4*>(stage + rr * kStagePitch + vcol);
                    float* dst = obase + static_cast<long long>(m0 + rr) * g.C + n0 + vcol;
                    if (vec_ok && vcol + 4 <= cols) {
                        *reinterpret_cast<float4*>(dst) = val;
                    } else {
                        dst[0] = val.x;
                        if (vcol + 1 < cols) dst[1] = val.y;
                        if (vcol + 2 < cols) dst[2] = val.z;
                        if (vcol + 3 < cols) dst[3] = val.w;
                    }
                }
            }
        }
        tc::tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace tcg
}  // namespace dynbatch
