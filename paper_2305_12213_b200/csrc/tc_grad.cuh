// The ragged gradient contraction on the tensor cores, fed by TMA (sm_100a):
//     G_w(d, c) = sum_{r in worker w} X(r, d) * E(r, c)          for every worker w in one launch
// X ([rows, D]) and E ([rows, C]) are row-major with the reduction index r as the row, so both
// operands are contiguous along their OUTPUT index.  tcgen05.mma reads such "MN-major" tiles
// directly, which removes the transposition through registers that the general contraction in
// tc_gemm.cuh has to do; what is left of the operand preparation, the split of every fp32 value
// into two TF32 halves, is done once by the kernel that produces E (and copies X), not once per
// output tile.  In the split arrays every worker's rows start at a multiple of 8 and are padded with
// zero rows to a multiple of 8, the reduction depth of one TF32 product.
//
// One persistent CTA per SM works through a list of items, an item being one 128 x TILE_N tile of one
// worker's G.  Three roles run decoupled, so that the operand stream from the L2 never stops for a
// tile boundary (measured on B200: a CTA's copy loop draws about 64 bytes per clock, the SM's L2 port,
// while the per-tile phases around it -- first copy, accumulator drain, store -- cost 2 us each when
// they are not overlapped):
//   warps 0-3 (one lane each) copy boxes of 16 rows of the four split arrays (X_hi, X_lo, E_hi, E_lo)
//                      into a ring of shared-memory stages with cp.async.bulk.tensor (128-byte swizzle
//                      of 32-byte pieces, completion on an mbarrier), running ahead across items; stage
//                      i is filled by warp i mod 4, because one thread's copy loop takes about 0.5 us
//                      per stage (measured), twice what the L2 port needs to deliver it;
//   warp 4 (one lane)  issues three tcgen05.mma.kind::tf32 per 8 rows (lo*hi + hi*lo into one
//                      accumulator in tensor memory, hi*hi round-robin into the others, see
//                      tc_gemm.cuh for why) into one of SETS accumulator sets and hands the set over
//                      with tcgen05.commit;
//   warps 5-12         drain a finished set, hand it back, and write the tile: through a staging tile
//                      in shared memory of its own, in the box layout of a TMA store when G is 16-byte
//                      aligned with rows of a multiple of 16 bytes, else as whole rows with ordinary
//                      stores.
// The items of a CTA come from a table in the kernel parameters that the host fills by dealing the
// items, most rows first, each to the CTA with the least work so far; problems with more items than the
// table holds take them round-robin.  Every wait is bounded (see tc_gemm.cuh); on a time-out the roles
// stop, the copy thread waits, again bounded, for the copies it has in flight and the issuing thread
// for its products before tensor memory is freed.
#pragma once
#include <cuda.h>

#include "tc_gemm.cuh"

namespace dynbatch {
namespace tcg {

constexpr int kTileM = 128;            // features per tile = tensor-memory lanes
constexpr int kChunk = 32;             // fp32 per 128-byte swizzled row
constexpr int kStepRows = 8;           // reduction depth of one TF32 product
constexpr int kRowsPerStage = 16;      // samples per stage: two products' worth
constexpr int kAccRows = 32;           // consecutive samples whose hi*hi products share an accumulator turn
constexpr int kChunkBytes = kRowsPerStage * 128;            // one [16 x 32] block of a stage
constexpr int kAChunks = kTileM / kChunk;
constexpr int kABytes = kAChunks * kChunkBytes;             // X_hi (or X_lo) part of a stage
constexpr int kEpilogueWarps = 8;      // two per tensor-memory lane quarter, half of the tile's columns each
constexpr int kEpilogueThreads = kEpilogueWarps * 32;
constexpr int kCopyWarps = 4;          // one lane each; stage i is filled by warp i mod 4
constexpr int kIssueWarp = kCopyWarps; // owns tensor memory, one lane issues the products
constexpr int kFirstEpilogueWarp = kCopyWarps + 1;
constexpr int kThreads = (kCopyWarps + 1) * 32 + kEpilogueThreads;
constexpr int kMaxCtas = 160;          // rows of the item table (CTAs of the persistent grid)
constexpr int kMaxItemsPerCta = 16;    // its columns

// Sizes that follow from the tile width (classes per tile = accumulator columns) and the number of
// accumulator sets.
template <int TILE_N, int SETS>
struct Shape {
    static constexpr int kBChunks = TILE_N / kChunk;
    static constexpr int kBBytes = kBChunks * kChunkBytes;              // E_hi (or E_lo) part of a stage
    static constexpr int kStageBytes = 2 * kABytes + 2 * kBBytes;
    static constexpr int kStagingBytes = kTileM * TILE_N * 4;           // the tile in the TMA store's box layout
    static constexpr int kStages = TILE_N == 128 ? 5 : 6;
    static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;   // + slack for 1024-byte alignment
    static constexpr int kMaxAcc = 512 / (SETS * TILE_N) - 1;           // main accumulators of a set, beside the cross-term one
    static_assert(kSmemBytes <= 227 * 1024 - 1024, "one CTA per SM, with room for the barriers");
    static_assert(kMaxAcc >= 1, "a set holds a main and a cross-term accumulator");
};

struct GradArgs {
    // The split arrays seen as [32-column chunk][row][32 floats] (the chunk stride, 128 bytes, is smaller than
    // the row stride), 128-byte swizzle of 32-byte pieces: one box of {32, 16 rows, n chunks} fills the
    // chunk-major tile of a stage with a single copy instruction.
    CUtensorMap x_hi, x_lo;        // [padded rows, D], boxes of 4 chunks
    CUtensorMap e_hi, e_lo;        // [padded rows, C], boxes of TILE_N / 32 chunks
    // Items: item i is tile (i % tiles) of the worker in slot i / tiles; slots are ordered by falling row count.
    int tiles_x, tiles;            // tiles along C; tiles per worker
    int n_items;
    int use_table;                 // item_table / item_count are valid, else CTA j takes items j, j + gridDim.x, ...
    unsigned short item_table[kMaxCtas][kMaxItemsPerCta];
    unsigned char item_count[kMaxCtas];
    float* out[DB_MAX_K];          // G of the worker in slot z, [D, C] row-major
    int tma_store;                 // every G is 16-byte aligned and C % 4 == 0: out_map[] is valid, tiles leave by TMA
    CUtensorMap out_map[DB_MAX_K]; // G as [D, C], boxes of 128 rows x 32 columns, 128-byte swizzle
    int row0[DB_MAX_K];            // first row of the worker in the split arrays (multiple of 8)
    int steps[DB_MAX_K];           // its padded row count / 8
    int K;                         // slots
    int D, C;
    int n_acc;                     // main accumulators in use per set, 1..kMaxAcc
    int* status;
    // mean loss of the worker in slot z = (sum of row_loss[loss_row0[z] .. + loss_rows[z])) / loss_rows[z], written
    // to loss_out[z] by CTA z % gridDim.x; row_loss == nullptr: not wanted
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
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// The k-th item of this CTA, or -1 past its last.
__device__ __forceinline__ int item_of(const GradArgs& g, int k) {
    if (g.use_table) return k < g.item_count[blockIdx.x] ? g.item_table[blockIdx.x][k] : -1;
    const long long i = static_cast<long long>(blockIdx.x) + static_cast<long long>(k) * gridDim.x;
    return i < g.n_items ? static_cast<int>(i) : -1;
}

// grid: one CTA per SM (fewer when there are fewer items)
template <int TILE_N, int SETS>
__global__ void __launch_bounds__(kThreads, 1)
grad_tma_kernel(const __grid_constant__ GradArgs g) {
    using S = Shape<TILE_N, SETS>;
    constexpr int kStages = S::kStages, kStageBytes = S::kStageBytes, kBBytes = S::kBBytes;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];     // a stage's copies have landed
    __shared__ __align__(8) uint64_t empty_bar[kStages];    // the products reading it have finished
    __shared__ __align__(8) uint64_t acc_full_bar[SETS];    // all products of an item have finished
    __shared__ __align__(8) uint64_t acc_empty_bar[SETS];   // its sums have been read out of tensor memory
    __shared__ __align__(8) uint64_t drain_bar;             // after a time-out: what had been issued has finished
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    unsigned char* tiles = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* staging = tiles + kStages * kStageBytes;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(&full_bar[s], 1);
            tc::mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < SETS; ++a) {
            tc::mbar_init(&acc_full_bar[a], 1);
            tc::mbar_init(&acc_empty_bar[a], 1);
        }
        tc::mbar_init(&drain_bar, 1);
        tc::fence_barrier_init();
        prefetch_tensormap(&g.x_hi);
        prefetch_tensormap(&g.x_lo);
        prefetch_tensormap(&g.e_hi);
        prefetch_tensormap(&g.e_lo);
    }
    const int set_cols = (g.n_acc + 1) * TILE_N;
    const uint32_t tmem_cols = tc::tmem_columns(SETS * set_cols);
    if (warp == kIssueWarp) tc::tmem_alloc(&tmem_base_slot, tmem_cols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // everything above overlaps the kernel that writes the split operands
    tc::griddep_launch_dependents();
    tc::griddep_wait();

    if (warp < kCopyWarps) {
        // ------------------------------------------------------------ TMA copies
        if (lane == 0) {
            int stage_i = 0;            // stages met so far, over all items; this warp fills those with stage_i % 4 == warp
            bool alive = true;
            for (int k = 0; alive; ++k) {
                const int item = item_of(g, k);
                if (item < 0) break;
                const int z = item / g.tiles, t = item % g.tiles;
                const int m0 = (t / g.tiles_x) * kTileM, n0 = (t % g.tiles_x) * TILE_N;
                const int loads = (g.steps[z] * kStepRows + kRowsPerStage - 1) / kRowsPerStage;
                for (int l = 0; l < loads; ++l, ++stage_i) {
                    if (stage_i % kCopyWarps != warp) continue;
                    const int s = stage_i % kStages;
                    if (stage_i >= kStages)
                        alive = tc::mbar_wait(&empty_bar[s], ((stage_i / kStages) - 1) & 1, &abort_flag, g.status, 4);
                    if (abort_flag) alive = false;
                    if (!alive) break;
                    mbar_expect_tx(&full_bar[s], kStageBytes);
                    const uint32_t dst = tc::smem_u32(tiles + s * kStageBytes);
                    const int row = g.row0[z] + l * kRowsPerStage;
                    tma_load_3d(dst, &g.x_hi, 0, row, m0 / kChunk, &full_bar[s]);
                    tma_load_3d(dst + kABytes, &g.x_lo, 0, row, m0 / kChunk, &full_bar[s]);
                    tma_load_3d(dst + 2 * kABytes, &g.e_hi, 0, row, n0 / kChunk, &full_bar[s]);
                    tma_load_3d(dst + 2 * kABytes + kBBytes, &g.e_lo, 0, row, n0 / kChunk, &full_bar[s]);
                }
            }
            // The copies this thread issued last write into this CTA's shared memory until they land: see them
            // complete (bounded) before this thread lets the CTA exit, whatever the other roles do.  After a
            // time-out stage_i stands at the stage that was not issued.
            for (int i = max(0, stage_i - kStages); i < stage_i; ++i) {
                if (i % kCopyWarps != warp) continue;
                const unsigned long long t0 = tc::global_ns();
                while (!tc::mbar_try_wait(&full_bar[i % kStages], (i / kStages) & 1) &&
                       tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            }
        }
        // mean losses: the per-sample losses were written by the kernel before this one
        if (warp == 0 && g.row_loss != nullptr) {
            __syncwarp();
            for (int z = blockIdx.x; z < g.K; z += gridDim.x) {
                if (g.loss_out[z] == nullptr) continue;
                const float* rl = g.row_loss + g.loss_row0[z];
                float part = 0.0f;
                for (int r = lane; r < g.loss_rows[z]; r += 32) part += __ldcg(rl + r);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                if (lane == 0) *g.loss_out[z] = part / static_cast<float>(g.loss_rows[z]);
            }
        }
    } else if (warp == kIssueWarp) {
        // ------------------------------------------------------------ tensor-core issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_tf32_mn(kTileM, TILE_N);
            bool alive = true;
            int used_stages = 0;        // stages consumed so far, over all items
            for (int k = 0; alive; ++k) {
                const int item = item_of(g, k);
                if (item < 0) break;
                const int a = k % SETS;
                // the set still holds the sums of the item SETS back until the epilogue has read them
                if (k >= SETS) {
                    alive = tc::mbar_wait(&acc_empty_bar[a], ((k / SETS) - 1) & 1, &abort_flag, g.status, 9);
                    if (!alive) break;
                    tc::tc_fence_after();
                }
                const uint32_t set_base = tmem_base + a * set_cols;
                const uint32_t acc_cross = set_base + g.n_acc * TILE_N;
                const int steps = g.steps[item / g.tiles];
                const int loads = (steps * kStepRows + kRowsPerStage - 1) / kRowsPerStage;
                for (int l = 0; l < loads; ++l) {
                    const int s = used_stages % kStages;
                    alive = tc::mbar_wait(&full_bar[s], (used_stages / kStages) & 1, &abort_flag, g.status, 5);
                    if (!alive) break;
                    tc::tc_fence_after();
                    const uint32_t st = tc::smem_u32(tiles + s * kStageBytes);
                    const int blk = l * kRowsPerStage / kAccRows;          // which 32-sample block
                    const bool blk_start = (l * kRowsPerStage) % kAccRows == 0;
                    const uint32_t acc_main = set_base + (blk % g.n_acc) * TILE_N;
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
                    ++used_stages;
                }
                if (alive) tc::mma_commit(&acc_full_bar[a]);
            }
            // see, bounded, what has been issued finish before the tensor memory is freed
            tc::mma_commit(&drain_bar);
            const unsigned long long t0 = tc::global_ns();
            while (!tc::mbar_try_wait(&drain_bar, 0) && tc::global_ns() - t0 < tc::kWaitLimitNs) {}
            tc::tc_fence_before();
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int et = tid - kFirstEpilogueWarp * 32;            // 0..255
        const int quarter = warp & 3;                            // the tensor-memory lanes this warp may read
        const int col_half = (warp - kFirstEpilogueWarp) >> 2;   // which half of the tile's columns it drains
        const int row = quarter * 32 + lane;
        for (int k = 0;; ++k) {
            const int item = item_of(g, k);
            if (item < 0) break;
            const int a = k % SETS;
            const int z = item / g.tiles, t = item % g.tiles;
            const int m0 = (t / g.tiles_x) * kTileM, n0 = (t % g.tiles_x) * TILE_N;
            // the verdict is made the same for all eight warps (a barrier that ANDs their predicates): what
            // follows has warp-wide instructions and barriers among them
            if (!epilogue_all(tc::mbar_wait(&acc_full_bar[a], (k / SETS) & 1, &abort_flag, g.status, 6))) break;
            tc::tc_fence_after();
            const uint32_t lane_base = tmem_base + a * set_cols + (static_cast<uint32_t>(quarter * 32) << 16);
            const int steps = g.steps[z];
            const int used = min(g.n_acc, (steps * kStepRows + kAccRows - 1) / kAccRows);
#pragma unroll 1
            for (int c0 = col_half * (TILE_N / 2); c0 < (col_half + 1) * (TILE_N / 2); c0 += 32) {
                uint32_t r[32], x[32];
                __syncwarp();
                tc::tmem_load32(lane_base + g.n_acc * TILE_N + c0, r);
                for (int acc = used - 1; acc >= 0; --acc) {
                    tc::tmem_load32(lane_base + acc * TILE_N + c0, x);
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(x[j]));
                }
                // the box layout of a TMA store, used for both ways out: [32-column block][128 rows][128 bytes],
                // 16-byte pieces permuted by the row's low three bits (which also keeps these stores conflict-free)
                unsigned char* box = staging + (c0 / 32) * (kTileM * 128) + row * 128;
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(box + (((j >> 2) ^ (row & 7)) << 4)) =
                        make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                    __uint_as_float(r[j + 3]));
            }
            tc::fence_proxy_async_smem();                     // the TMA engine may read what these threads wrote
            tc::tc_fence_before();                            // the accumulators have been read
            epilogue_sync();
            if (et == 0) tc::mbar_arrive(&acc_empty_bar[a]);  // the set may take the item SETS ahead
            if (g.tma_store) {
                if (et == 0) {
#pragma unroll
                    for (int h = 0; h < TILE_N / 32; ++h)
                        if (n0 + h * 32 < g.C)
                            tma_store_2d(&g.out_map[z], n0 + h * 32, m0, tc::smem_u32(staging + h * (kTileM * 128)));
                    bulk_commit();
                    bulk_wait_read();      // the staging tile must stay until the engine has read it
                }
            } else {
                // whole rows of the tile, TILE_N / 4 threads per row
                float* obase = g.out[z];
                const int rows = min(kTileM, g.D - m0), cols = min(TILE_N, g.C - n0);
                constexpr int kVecPerRow = TILE_N / 4;
                constexpr int kRowsPerPass = kEpilogueThreads / kVecPerRow;
                const int vcol = (et % kVecPerRow) * 4, rsub = et / kVecPerRow;
                const bool vec_ok = (g.C % 4 == 0) && (reinterpret_cast<uintptr_t>(obase) % 16 == 0);
                for (int r0 = 0; r0 < rows; r0 += kRowsPerPass) {
                    const int rr = r0 + rsub;
                    if (rr >= rows || vcol >= cols) continue;
                    const float4 val = *reinterpret_cast<const float4*>(
                        staging + (vcol / 32) * (kTileM * 128) + rr * 128 + ((((vcol % 32) >> 2) ^ (rr & 7)) << 4));
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
            epilogue_sync();               // the staging tile is free for the next item
        }
        tc::tc_fence_before();
    }
    __syncthreads();
    if (warp == kIssueWarp) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace tcg
}  // namespace dynbatch
