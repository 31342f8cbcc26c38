// fp32-accurate GEMM on the 5th-generation tensor cores (tcgen05, sm_100a):
//     out(m, n) = sum_k A(m, k) * B(n, k)           A, B, out fp32 in global memory
// Each fp32 operand is split on the fly into two TF32 numbers, x = hi + lo with
// hi = tf32(x), lo = tf32(x - hi), and three tensor-core products are accumulated
// in fp32 in tensor memory: lo*hi + hi*lo + hi*hi (the dropped lo*lo term is 2^-22
// relative).  This is what the ragged softmax gradient needs: its two contractions
// are dense, but the result must match an fp64 oracle to 1e-5, which a single TF32
// or bf16 product (2^-11 / 2^-8) cannot do.
//
// Structure of one CTA (288 threads), one 128 x N_TILE output tile, reduction in
// blocks of 32:
//   warps 0-7  read A and B straight from global memory with whatever strides the
//              caller gives (either operand may be reduction-contiguous or
//              row-contiguous), split hi/lo in registers and store the four operand
//              tiles into shared memory in the tensor core's reduction-major 128-byte
//              swizzled layout; a TMA copy cannot be used because the data has to be
//              transformed (and often transposed) between global and shared memory.
//              Afterwards they drain the accumulator (tcgen05.ld) and write the tile.
//   warp 8     owns the tensor memory allocation; its lane 0 issues the tcgen05.mma
//              instructions and signals stage reuse / completion with tcgen05.commit.
// Two shared-memory stages, full/empty mbarriers.  Every wait is bounded: on a
// time-out the kernel records a code in *status, stops issuing work, waits (bounded)
// for its own tensor-core operations, frees its tensor memory and returns.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "dynbatch.h"

namespace dynbatch {
namespace tc {

constexpr int kTileM = 128;        // rows of the output tile = TMEM lanes
constexpr int kBlockK = 32;        // fp32 elements per 128-byte swizzled row
constexpr int kStages = 2;
constexpr int kLoaderWarps = 8;    // two per scheduler: one hides the other's latencies
constexpr int kLoaderThreads = kLoaderWarps * 32;
constexpr int kThreads = kLoaderThreads + 32;   // + the warp that owns tensor memory and issues the products
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

struct GemmArgs {
    const float* A; long long a_row, a_k;   // A(m, k) = A[m * a_row + k * a_k]
    const float* B; long long b_row, b_k;   // B(n, k) = B[n * b_row + k * b_k]
    float* out; long long o_m, o_n;         // out(m, n) at out[m * o_m + n * o_n] (+ split * o_split)
    long long o_split;
    int M, N, K;
    int k_per_split;                        // multiple of kBlockK; split z covers [z*kps, min(K, (z+1)*kps))
    int n_acc;                              // main accumulators used round-robin, (n_acc + 1) * N_TILE <= 512
    int* status;                            // device word, set non-zero if a wait gave up
    int clear_status;                       // non-zero: the first CTA zeroes *status before any wait can set it
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Waits for the barrier phase; gives up after limit_ns or when another thread already did.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int code, unsigned long long limit_ns = kWaitLimitNs) {
    unsigned long long t0 = 0;
    for (unsigned int spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spin & 255u) == 255u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) {
                *abort_flag = 1;
                if (status) atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}
// Programmatic dependent launch: let the next kernel in the stream start its prologue while this one
// runs, and wait for the previous kernel's results before touching them.  Both are no-ops for a
// kernel launched without the attribute.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
    const uint32_t zero = 0;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(zero) : "memory");
}
// Arrives on the mbarrier once every tcgen05 operation issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Tensor-memory allocations are powers of two between 32 and 512 columns.
__host__ __device__ constexpr uint32_t tmem_columns(int needed) {
    uint32_t c = 32;
    while (c < static_cast<uint32_t>(needed)) c <<= 1;
    return c;
}

// Shared-memory matrix descriptor of a reduction-major tile with 128-byte rows and the
// 128-byte swizzle: 8-row groups are 1024 bytes apart; version 1; layout type 2.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);       // start address
    d |= static_cast<uint64_t>(1) << 16;                        // leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                        // descriptor version
    d |= static_cast<uint64_t>(2) << 61;                        // 128-byte swizzle
    return d;
}
// Instruction descriptor: fp32 accumulator, TF32 A and B, both reduction-major, M x N tile.
__host__ __device__ constexpr uint32_t instr_desc_tf32(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
           (static_cast<uint32_t>(M >> 4) << 24);
}

// Nearest TF32 (10 explicit mantissa bits), ties away from zero, by integer arithmetic on the bits:
// add half a TF32 unit in the last place, clear the 13 low bits.
__device__ __forceinline__ float round_tf32(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}
// x = hi + lo up to 2^-22 |x|, both halves representable in TF32 (x - hi is exact in fp32).
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
    hi = round_tf32(x);
    lo = round_tf32(x - hi);
}

// Byte offset of element (row, k) in a [rows x 32] fp32 tile with 128-byte rows and the
// 128-byte swizzle (16-byte chunk index XOR row mod 8); the tile base is 1024-byte aligned.
__device__ __forceinline__ uint32_t swz(int row, int k) {
    return static_cast<uint32_t>(row * 128 + ((((k >> 2) ^ (row & 7)) << 4) | ((k & 3) << 2)));
}

// How one operand tile (ROWS x 32 fp32) travels from global memory to shared memory.
// element (r, kk) = src[r * row_stride + kk * k_stride], zero outside r < rows_valid, kk < k_valid.
enum LoadMode {
    kLoadKVec = 0,    // k_stride == 1: one float4 along k per thread and step (rows 16-byte aligned)
    kLoadRowVec = 1,  // row_stride == 1: one float4 along the rows per thread and step (k columns 16-byte aligned)
    kLoadScalar = 2   // anything else: single elements
};

// Registers of one thread's share of a tile: ROWS * 32 / kLoaderThreads values.
template <int ROWS> struct TileRegs { float v[ROWS * kBlockK / kLoaderThreads]; };

// Phase 1: issue every global load of the tile (nothing depends on another load).
template <int ROWS, int MODE>
__device__ __forceinline__ void tile_load(TileRegs<ROWS>& t, const float* __restrict__ src, long long row_stride,
                                          long long k_stride, int rows_valid, int k_valid, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    if (MODE == kLoadKVec) {
        const int kk = (tid & 7) * 4;
#pragma unroll
        for (int i = 0; i < ROWS / (kLoaderThreads / 8); ++i) {
            const int r = (tid >> 3) + i * (kLoaderThreads / 8);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < rows_valid) {
                const float* p = src + static_cast<long long>(r) * row_stride + kk;
                if (kk + 3 < k_valid) {
                    x = __ldg(reinterpret_cast<const float4*>(p));
                } else {
                    if (kk + 0 < k_valid) x.x = __ldg(p + 0);
                    if (kk + 1 < k_valid) x.y = __ldg(p + 1);
                    if (kk + 2 < k_valid) x.z = __ldg(p + 2);
                }
            }
            t.v[4 * i + 0] = x.x; t.v[4 * i + 1] = x.y; t.v[4 * i + 2] = x.z; t.v[4 * i + 3] = x.w;
        }
    } else if (MODE == kLoadRowVec) {
        // a warp step covers 8 rows x 16 k: lane -> (4 rows starting at 4 * (lane & 1), k = lane >> 1);
        // the four scalar stores of a step then hit 32 different banks
        const int kl = lane >> 1, rsub = (lane & 1) * 4;
#pragma unroll
        for (int i = 0; i < ROWS / (4 * kLoaderWarps); ++i) {
            const int step = warp + i * kLoaderWarps;      // (ROWS / 8) row groups x 2 k halves
            const int r = (step >> 1) * 8 + rsub, kk = (step & 1) * 16 + kl;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (kk < k_valid && r < rows_valid) {
                const float* p = src + r + static_cast<long long>(kk) * k_stride;
                if (r + 3 < rows_valid) {
                    x = __ldg(reinterpret_cast<const float4*>(p));
                } else {
                    x.x = __ldg(p);
                    if (r + 1 < rows_valid) x.y = __ldg(p + 1);
                    if (r + 2 < rows_valid) x.z = __ldg(p + 2);
                }
            }
            t.v[4 * i + 0] = x.x; t.v[4 * i + 1] = x.y; t.v[4 * i + 2] = x.z; t.v[4 * i + 3] = x.w;
        }
    } else {
        // 8 rows x 4 k patches per warp step
        const int rl = lane & 7, kl = lane >> 3;
#pragma unroll
        for (int i = 0; i < ROWS / kLoaderWarps; ++i) {
            const int pidx = warp + i * kLoaderWarps;
            const int r = (pidx >> 3) * 8 + rl, kk = (pidx & 7) * 4 + kl;
            float x = 0.f;
            if (r < rows_valid && kk < k_valid)
                x = __ldg(src + static_cast<long long>(r) * row_stride + static_cast<long long>(kk) * k_stride);
            t.v[i] = x;
        }
    }
}

// Phase 2: split into TF32 halves and store into the swizzled hi / lo tiles.  `lo_delta` is the byte
// distance from the hi tile to the lo tile.  A thread's elements sit at a fixed swizzled offset plus a
// compile-time multiple of whole 8-row groups, so every store is [register + immediate].
template <int ROWS, int MODE>
__device__ __forceinline__ void tile_store(const TileRegs<ROWS>& t, unsigned char* hi_tile, int lo_delta, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    if (MODE == kLoadKVec) {
        // rows (tid >> 3) + 32 i: the row's position in its 8-row group never changes
        unsigned char* base = hi_tile + swz(tid >> 3, (tid & 7) * 4);
#pragma unroll
        for (int i = 0; i < ROWS / (kLoaderThreads / 8); ++i) {
            float4 h, l;
            split_tf32(t.v[4 * i + 0], h.x, l.x);
            split_tf32(t.v[4 * i + 1], h.y, l.y);
            split_tf32(t.v[4 * i + 2], h.z, l.z);
            split_tf32(t.v[4 * i + 3], h.w, l.w);
            unsigned char* dst = base + i * (kLoaderThreads / 8) * 128;
            *reinterpret_cast<float4*>(dst) = h;
            *reinterpret_cast<float4*>(dst + lo_delta) = l;
        }
    } else if (MODE == kLoadRowVec) {
        // step = warp + 8 i: k half (warp & 1) and the row's position in its group are fixed per thread
        const int kk = (warp & 1) * 16 + (lane >> 1), r0 = (warp >> 1) * 8 + (lane & 1) * 4;
        unsigned char* base[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) base[j] = hi_tile + swz(r0 + j, kk);
#pragma unroll
        for (int i = 0; i < ROWS / (4 * kLoaderWarps); ++i) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float h, l;
                split_tf32(t.v[4 * i + j], h, l);
                unsigned char* dst = base[j] + i * (kLoaderWarps / 2) * 8 * 128;
                *reinterpret_cast<float*>(dst) = h;
                *reinterpret_cast<float*>(dst + lo_delta) = l;
            }
        }
    } else {
        // patch = warp + 8 i: k group (warp & 7 ... ) fixed, row group advances by one per step
        const int rl = lane & 7, kk = (warp & 7) * 4 + (lane >> 3);
        unsigned char* base = hi_tile + swz(rl, kk);
#pragma unroll
        for (int i = 0; i < ROWS / kLoaderWarps; ++i) {
            float h, l;
            split_tf32(t.v[i], h, l);
            unsigned char* dst = base + i * 8 * 128;       // (warp + 8 i) >> 3 = i row groups of 8
            *reinterpret_cast<float*>(dst) = h;
            *reinterpret_cast<float*>(dst + lo_delta) = l;
        }
    }
}

template <int N_TILE>
struct SmemLayout {
    static constexpr int kATile = kTileM * 128;             // bytes of one A tile (hi or lo)
    static constexpr int kBTile = N_TILE * 128;
    static constexpr int kStage = 2 * kATile + 2 * kBTile;  // A_hi, A_lo, B_hi, B_lo
    static constexpr int kBytes = kStages * kStage + 1024;  // + slack for 1024-byte alignment
};

// Tensor memory: g.n_acc main accumulators of N_TILE columns each take the hi*hi products of the
// reduction blocks round-robin (block kb goes to accumulator kb mod n_acc); one more accumulator
// takes both cross terms.  The tensor core truncates when it adds into an fp32 accumulator, a bias
// that grows with the length of the chain (measured 7e-9 * K relative), so the chain is cut into
// n_acc shorter ones that the epilogue adds with ordinary rounded fp32 additions.  The cross terms
// are 2^-11 of the main one: the rounding of their own chain is invisible.
template <int N_TILE, int MODE_A, int MODE_B>
__device__ __forceinline__ void tf32x3_gemm_body(const GemmArgs& g, const int split) {
    using L = SmemLayout<N_TILE>;
    constexpr int kStagePitch = N_TILE + 4;   // floats per row of the output staging tile (16-byte rows, no bank conflicts)
    static_assert(kTileM * kStagePitch * 4 <= kStages * L::kStage, "output staging fits in the operand stages");
    static_assert(N_TILE == 32 || N_TILE == 64 || N_TILE == 128, "accumulator columns: power of two >= 32");
    static_assert(kLoaderWarps == 8, "the tile_load / tile_store lane maps assume eight loader warps");
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ __align__(8) uint64_t done_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    unsigned char* tiles = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.y * kTileM, n0 = blockIdx.x * N_TILE;
    const int k_begin = split * g.k_per_split;
    const int k_end = min(g.K, k_begin + g.k_per_split);
    const int nkb = (k_end - k_begin + kBlockK - 1) / kBlockK;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], kLoaderThreads);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&done_bar, 1);
        fence_barrier_init();
    }
    const uint32_t tmem_cols = tmem_columns((g.n_acc + 1) * N_TILE);
    if (warp == kLoaderWarps) tmem_alloc(&tmem_base_slot, tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // Everything above overlaps the previous kernel; its outputs are read only from here on.  The
    // successor is released after the wait: as the logits kernel of a worker-gradient call it is followed
    // by a kernel that writes the workspace before waiting, which must not start while an earlier call's
    // kernels still read it.
    griddep_wait();
    griddep_launch_dependents();
    // a time-out needs seconds, this store comes microseconds after the launch: no wait can have given up yet
    if (g.clear_status && tid == 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) *g.status = 0;

    if (warp < kLoaderWarps) {
        // ------------------------------------------------------------ producers
        const float* Abase = g.A + static_cast<long long>(m0) * g.a_row;
        const float* Bbase = g.B + static_cast<long long>(n0) * g.b_row;
        const int a_rows = min(kTileM, g.M - m0), b_rows = min(N_TILE, g.N - n0);
        TileRegs<kTileM> ra, ra_next;
        TileRegs<N_TILE> rb, rb_next;
        if (nkb > 0) {
            const int k_valid = min(kBlockK, k_end - k_begin);
            tile_load<kTileM, MODE_A>(ra, Abase + static_cast<long long>(k_begin) * g.a_k, g.a_row, g.a_k, a_rows,
                                      k_valid, tid);
            tile_load<N_TILE, MODE_B>(rb, Bbase + static_cast<long long>(k_begin) * g.b_k, g.b_row, g.b_k, b_rows,
                                      k_valid, tid);
        }
        bool alive = true;
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kStages;
            if (kb + 1 < nkb) {
                // the next block's loads fly while this block is converted, stored and multiplied
                const int k0 = k_begin + (kb + 1) * kBlockK;
                const int k_valid = min(kBlockK, k_end - k0);
                tile_load<kTileM, MODE_A>(ra_next, Abase + static_cast<long long>(k0) * g.a_k, g.a_row, g.a_k,
                                          a_rows, k_valid, tid);
                tile_load<N_TILE, MODE_B>(rb_next, Bbase + static_cast<long long>(k0) * g.b_k, g.b_row, g.b_k,
                                          b_rows, k_valid, tid);
            }
            if (kb >= kStages)
                alive = mbar_wait(&empty_bar[s], ((kb / kStages) - 1) & 1, &abort_flag, g.status, 1);
            if (!alive) break;
            unsigned char* st = tiles + s * L::kStage;
            tile_store<kTileM, MODE_A>(ra, st, L::kATile, tid);
            tile_store<N_TILE, MODE_B>(rb, st + 2 * L::kATile, L::kBTile, tid);
            fence_proxy_async_smem();   // make the generic-proxy stores visible to the tensor core
            mbar_arrive(&full_bar[s]);
            ra = ra_next;
            rb = rb_next;
        }
        // ------------------------------------------------------------ epilogue
        if (alive && nkb > 0) alive = mbar_wait(&done_bar, 0, &abort_flag, g.status, 3);
        alive = __all_sync(0xffffffffu, alive);      // tcgen05.ld below is a warp-wide instruction
        tc_fence_after();
        if (alive) {
            // warp w may read tensor-memory lanes 32 (w mod 4) .. +31; the two warps that share a lane
            // quarter take alternate 32-column chunks
            const int quarter = warp & 3;
            const int m = m0 + quarter * 32 + lane;         // this thread's accumulator lane = output row
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            float* obase = g.out + static_cast<long long>(split) * g.o_split + static_cast<long long>(m) * g.o_m;
            const int used = min(g.n_acc, nkb);
#pragma unroll 1
            for (int c0 = (warp >> 2) * 32; c0 < N_TILE; c0 += 32 * (kLoaderWarps / 4)) {
                uint32_t r[32];
                if (nkb > 0) {
                    uint32_t x[32];
                    __syncwarp();
                    tmem_load32(lane_base + g.n_acc * N_TILE + c0, r);          // cross terms
                    for (int a = used - 1; a >= 0; --a) {
                        tmem_load32(lane_base + a * N_TILE + c0, x);
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(x[j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                const int n_first = n0 + c0;
                if (g.o_n != 1 && (m >= g.M || n_first >= g.N)) continue;
                if (g.o_n == 1) {
                    // rows are contiguous along n: park the chunk in shared memory (the operand stages
                    // are free once the last product has completed) and write whole rows below
                    float* srow = reinterpret_cast<float*>(tiles) + (quarter * 32 + lane) * kStagePitch + c0;
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(srow + j) =
                            make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                        __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                } else {
                    // lanes are consecutive m: coalesced when o_m == 1
                    float* col = obase + static_cast<long long>(n_first) * g.o_n;
                    const int n_left = g.N - n_first;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < n_left) *col = __uint_as_float(r[j]);
                        col += g.o_n;
                    }
                }
            }
        }
        if (g.o_n == 1) {
            // all eight epilogue warps meet (named barrier 1; the issuing warp is not part of it)
            asm volatile("bar.sync 1, %0;" ::"n"(kLoaderThreads) : "memory");
            if (alive) {
                const float* stage = reinterpret_cast<const float*>(tiles);
                float* obase = g.out + static_cast<long long>(split) * g.o_split;
                const int rows = min(kTileM, g.M - m0), cols = min(N_TILE, g.N - n0);
                constexpr int kVecPerRow = N_TILE / 4;                 // float4 per tile row
                constexpr int kRowsPerPass = kLoaderThreads / kVecPerRow;
                const int vcol = (tid % kVecPerRow) * 4, rsub = tid / kVecPerRow;
                const bool vec_ok = (g.o_m % 4 == 0) && (reinterpret_cast<uintptr_t>(obase + n0) % 16 == 0);
                for (int r0 = 0; r0 < rows; r0 += kRowsPerPass) {
                    const int rr = r0 + rsub;
                    if (rr >= rows || vcol >= cols) continue;
                    const float4 val = *reinterpret_cast<const float4*>(stage + rr * kStagePitch + vcol);
                    float* dst = obase + static_cast<long long>(m0 + rr) * g.o_m + n0 + vcol;
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
        tc_fence_before();
    } else if (lane == 0) {
        // ------------------------------------------------------------ tensor-core issuer
        constexpr uint32_t idesc = instr_desc_tf32(kTileM, N_TILE);
        const uint32_t acc_cross = tmem_base + g.n_acc * N_TILE;
        bool alive = true;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            const int s = kb % kStages;
            alive = mbar_wait(&full_bar[s], (kb / kStages) & 1, &abort_flag, g.status, 2);
            if (!alive) break;
            tc_fence_after();
            const uint32_t st = smem_u32(tiles + s * L::kStage);
            const uint64_t a_hi = smem_desc_k_sw128(st), a_lo = smem_desc_k_sw128(st + L::kATile);
            const uint64_t b_hi = smem_desc_k_sw128(st + 2 * L::kATile);
            const uint64_t b_lo = smem_desc_k_sw128(st + 2 * L::kATile + L::kBTile);
            const uint32_t acc_main = tmem_base + (kb % g.n_acc) * N_TILE;
#pragma unroll
            for (int ks = 0; ks < kBlockK / 8; ++ks) {
                const uint64_t adv = static_cast<uint64_t>((ks * 8 * 4) >> 4);   // 32 bytes per 8 TF32
                mma_tf32(acc_cross, a_lo + adv, b_hi + adv, idesc, (kb | ks) != 0);
                mma_tf32(acc_cross, a_hi + adv, b_lo + adv, idesc, 1);
                mma_tf32(acc_main, a_hi + adv, b_hi + adv, idesc, (kb >= g.n_acc) || ks != 0);
            }
            mma_commit(&empty_bar[s]);   // the stage may be refilled once these products have been read
        }
        mma_commit(&done_bar);
        if (!alive) {
            // give the operations already issued a bounded time to finish before the memory goes away
            unsigned long long t0 = global_ns();
            while (!mbar_try_wait(&done_bar, 0) && global_ns() - t0 < kWaitLimitNs) {}
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == kLoaderWarps) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// blockIdx.z = split of the reduction.
template <int N_TILE, int MODE_A, int MODE_B>
__global__ void __launch_bounds__(kThreads)
tf32x3_gemm_kernel(const __grid_constant__ GemmArgs g) {
    tf32x3_gemm_body<N_TILE, MODE_A, MODE_B>(g, blockIdx.z);
}

}  // namespace tc
}  // namespace dynbatch
