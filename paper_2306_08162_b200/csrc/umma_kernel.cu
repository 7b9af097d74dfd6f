// Tensor-core kernel of the quantized-linear + LoRA layer for sm_100a: TMA-staged packed codes and group parameters,
// register-level unpack + dequantisation to bf16 in shared memory, tcgen05 MMA with fp32 accumulators in tensor
// memory, LoRA update fused as one extra MMA per tile, bf16 epilogue.
//
// One kernel template serves both directions (Figure 1 of the paper):
//   forward        Out[m, n] = sum_k X[m, k]  W[n, k] + s sum_j H[m, j] B[n, j]      contraction over k
//   backward-input Out[m, k] = sum_n dY[m, n] W[n, k] + s sum_j G[m, j] A[j, k]      contraction over n
// The backward direction is the paper's fused "transpose + unpack + matmul" (Section 3.1): nothing is transposed in
// memory.  The packed word still yields consecutive-k codes; they are written as one 16-byte chunk of a shared-memory
// operand whose *non-contraction* dimension is contiguous, and the MMA descriptor's major-ness bit does the rest.
//
// Orientation: the dequantised weight tile is the MMA's A operand (128 rows), the activation tile is the B operand
// (up to 256 token rows), so every dequantised weight is reused by up to 256 tokens inside one CTA.  The accumulator
// D[weight row, token] lives in tensor memory (two buffers of 256 columns, so the epilogue of one tile overlaps the
// main loop of the next).
//
// Warp roles (480 threads): warp 0 = TMA producer of activation tiles, warp 1 = MMA issuer (+ tensor-memory
// allocation), warp 2 = TMA producer of packed codes + group parameters (its ring runs ahead of the activation ring),
// warps 3-6 = epilogue (+ LoRA operand staging), warps 7-14 = unpack/dequant (two groups taking alternate stages).
// Every mbarrier wait is bounded; on a timeout the kernel records a status word, drains and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "device_state.h"
#include "launch.h"
#include "lora_down.cuh"

namespace qlora {

__device__ unsigned int g_device_status = 0;   // sticky; bit 0: an mbarrier wait timed out

// The producer clusters of a launch signal its tile CTAs through a pair of counters in the CALLER's workspace (the layer
// calls carve two words out of it): [0] producer CTAs that have published their rows, [1] tile CTAs that have seen the
// full count.  A one-warp kernel ahead of the launch sets the pair to zero (in stream order, with programmatic dependent
// launch, so the main kernel's set-up still overlaps its predecessor); the last tile CTA zeroes it again.

namespace {

constexpr int kThreads = 480;
constexpr int kDequantWarp0 = 7, kGroupWarps = 4;   // two dequant groups of four warps
constexpr int kEpiWarp0 = 3, kEpiWarps = 4;
constexpr int kSyncWords = 64;                       // counters in the workspace: [0], [1] producer clusters, [2 ..] one per split tile
constexpr size_t kSplitTileBytes = 2 * 2 * 8 * 8 * 128 * 16;   // exchange area of one split tile: 2 halves x 2 CTAs x 8 chunks x 4 KiB
constexpr int kWRows = 128;          // weight rows (MMA M) per tile: n in forward, k in backward
constexpr int kStepC = 64;           // contraction elements per pipeline stage
constexpr int kWStageBytes = kWRows * kStepC * 2;   // 16 KiB of bf16 per stage
constexpr int kAccStride = 256;      // tensor-memory columns per accumulator buffer
constexpr uint32_t kSpinLimit = 1u << 26;
constexpr int kWaitLimitUs = 250000;   // default limit of a wait, a launch parameter: far beyond any healthy wait (microseconds), short for a hang

struct Params {
    int M, N, K, bits, g, r, r_pad;
    int C;               // output columns (N forward, K backward)
    int BT;              // token rows per tile (MMA N): 32, 64, 128 or 256
    int n_tok_tiles, n_tiles, steps;
    int split;           // CTAs per cluster sharing one tile, each taking `steps` consecutive steps of the contraction (1 = no cluster)
    int S, P;            // stages of the activation/weight ring and of the packed ring
    int packed_cols;     // 128 forward, 64 backward
    int packed_rows;     // int32 rows per stage
    int scale_rows;      // group rows per stage
    uint32_t words_bytes, scale_bytes, packed_slot_bytes, x_stage_bytes;
    uint32_t off_x, off_w, off_p, off_lora_a, off_lora_p, off_bar;   // offsets from the 1024-aligned smem base
    float s;
    const float* Pmat;               // H (forward) or G (backward), fp32 [M, r]
    const __nv_bfloat16* L;          // B [N, r] (forward) or A [r, K] (backward)
    __nv_bfloat16* Out;
    // producer clusters (n_prod > 0, as in the CTA-pair kernel): the first n_prod clusters of the grid compute
    // P = In * Ldown into Pout (== Pmat) beside the tiles and publish it through counter pair `slot`
    int n_prod, T, lds_stages;
    unsigned int* sync;   // the counter pair (n_prod > 0)
    int wait_limit_us;    // every wait inside the kernel gives up after this long
    const __nv_bfloat16* In;         // [M, T]
    const __nv_bfloat16* Ldown;      // A [r, K] (forward) or B [N, r] (backward)
    float* Pout;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after abort_flag[1] microseconds of wall time (the launch's limit, set beside the flag when the
// kernel starts) or kSpinLimit polls.  Returns false when the kernel is
// aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    uint64_t t0 = 0;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u) {
            if (*abort_flag) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > (uint64_t)abort_flag[1] * 1000ull) break;
        }
    }
    *abort_flag = 1;
    atomicOr(&g_device_status, 1u);
    return false;
}
// Whole-warp wait: lane 0 polls (so a waiting warp costs one lane's issue slots), the outcome is broadcast, and every
// lane then observes the completed phase itself before touching the data the barrier guards.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int lane) {
    if (__all_sync(0xFFFFFFFFu, mbar_try_wait(bar, parity) != 0u)) return true;   // already complete: one instruction per lane
    uint32_t ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1u : 0u;
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    if (ok) (void)mbar_try_wait(bar, parity);
    return ok != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- thread-block cluster helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
    return v;
}


// Bounded wait until a counter in global memory reaches `target` (written by other CTAs of the same launch).
__device__ __forceinline__ bool wait_counter(const unsigned* ctr, unsigned target, volatile int* abort_flag) {
    uint64_t t0 = 0;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v >= target) return true;
        __nanosleep(256);
        if ((i & 63u) == 63u) {
            if (*abort_flag) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > (uint64_t)abort_flag[1] * 1000ull) break;
        }
    }
    *abort_flag = 1;
    atomicOr(&g_device_status, 1u);
    return false;
}

#include "lora_down_stream.cuh"

// Shared-memory matrix descriptor (version 1).  Offsets in bytes; layout 0 = no swizzle, 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n_mma; majors: 0 = contraction-contiguous, 1 = other.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n_mma, uint32_t a_mn_major, uint32_t b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major << 15) | (b_mn_major << 16) | ((n_mma >> 3) << 17) |
           ((128u >> 4) << 24);
}

// Ring position: slot index plus the phase bit of the current lap (no division in the hot loops).
struct Ring {
    uint32_t slot = 0, phase = 0;
    __device__ __forceinline__ void advance(uint32_t n) { if (++slot == n) { slot = 0; phase ^= 1u; } }
};

template <int BITS, bool TRANSPOSED>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_q,
                 const __grid_constant__ CUtensorMap tm_scales, const __grid_constant__ CUtensorMap tm_zeros,
                 const Params p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s[2];   // [0] set when a wait gave up, [1] the launch's wait limit in microseconds
    volatile int* abort_flag = abort_flag_s;
    pdl_launch_dependents();

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem0 - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t S = (uint32_t)p.S, P = (uint32_t)p.P;

    // barrier addresses
    const uint32_t bar_full_x = smem0 + p.off_bar;          // [S]  stage full: activation tile landed (TMA) and weight tile
    const uint32_t bar_full_w = bar_full_x;                 //      written by one dequant group (one wait for the MMA issuer)
    const uint32_t bar_empty = bar_full_x + 8 * S;          // [S]  MMAs reading the stage have completed
    const uint32_t bar_full_p = bar_empty + 8 * S;          // [P]  packed words + group parameters landed (TMA)
    const uint32_t bar_empty_p = bar_full_p + 8 * P;        // [P]  the dequant group has read them into registers
    const uint32_t bar_acc_full = bar_empty_p + 8 * P;      // [2]  accumulator buffer complete
    const uint32_t bar_acc_empty = bar_acc_full + 16;       // [2]  accumulator buffer drained by the epilogue
    const uint32_t bar_lora_full = bar_acc_empty + 16;      // [1]  LoRA operand tiles staged

    if (threadIdx.x == 0) {
        abort_flag_s[0] = 0; abort_flag_s[1] = p.wait_limit_us;
        for (uint32_t i = 0; i < S; ++i) {
            mbar_init(bar_full_x + 8 * i, 1 + kGroupWarps);
            mbar_init(bar_empty + 8 * i, 1);
        }
        for (uint32_t i = 0; i < P; ++i) {
            mbar_init(bar_full_p + 8 * i, 1);
            mbar_init(bar_empty_p + 8 * i, kGroupWarps);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, kEpiWarps);
        }
        mbar_init(bar_lora_full, kEpiWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // whole warp: allocate all 512 tensor-memory columns (one CTA per SM owns them)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // Set-up done.  The frozen weights are read-only for every call of the library, so their producer starts at once; the
    // roles that touch what the preceding work in the stream may have produced (activations, P) or may still be reading
    // (the output) call pdl_wait() first.

    // Few tokens give few tiles: the contraction of a tile is then split over a cluster of p.split CTAs (rank i takes steps
    // i * p.steps ...), each accumulates its part in tensor memory, and the parts are added through distributed shared
    // memory at the end.  One tile per cluster in that mode.
    const int rank = p.split > 1 ? (int)cluster_ctarank() : 0;
    const int first_tile = (int)blockIdx.x / p.split - p.n_prod, tile_stride = (int)gridDim.x / p.split - p.n_prod;
    const int step0 = rank * p.steps;

    if (first_tile < 0) {
        // ------------------------------------------------------------------ producer cluster: LoRA down-projection on SMs
        // the tiles leave idle (one CTA per row block or more; lowest block indices, so they wait for nobody)
        const int n_ctas = p.n_prod * p.split;
        pdl_wait();
        if (p.r <= 8) lora_down_stream<!TRANSPOSED, 1>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, n_ctas, smem_gen, p.lds_stages, abort_flag);
        else          lora_down_stream<!TRANSPOSED, 2>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, n_ctas, smem_gen, p.lds_stages, abort_flag);
        __threadfence();       // every thread's rows of P are visible device-wide before the CTA is counted
        __syncthreads();
        if (threadIdx.x == 0) atomicAdd(&p.sync[0], 1u);
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: activation tiles
        if (lane == 0) {
            pdl_wait();
            Ring ring;
            for (int tile = first_tile; tile < p.n_tiles; tile += tile_stride) {
                const int m0 = (tile % p.n_tok_tiles) * p.BT;
                for (int step = 0; step < p.steps; ++step) {
                    if (!mbar_wait(bar_empty + 8 * ring.slot, ring.phase ^ 1u, abort_flag)) goto done;
                    const uint32_t bar = bar_full_x + 8 * ring.slot;
                    mbar_expect_tx(bar, p.x_stage_bytes);
                    tma_load_2d(smem0 + p.off_x + ring.slot * p.x_stage_bytes, &tm_act, bar, (step0 + step) * kStepC, m0);
                    ring.advance(S);
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ TMA producer: packed codes, scales, zeros
        if (lane == 0) {
            Ring ring;
            const uint32_t tx_bytes = p.words_bytes + 2 * p.scale_bytes;
            for (int tile = first_tile; tile < p.n_tiles; tile += tile_stride) {
                const int w0 = (tile / p.n_tok_tiles) * kWRows;
                // forward: weight rows n = w0.., contraction k = c0..;  backward: weight rows k = w0.., contraction n = c0..
                const int g_row = TRANSPOSED ? w0 / p.g : 0;
                for (int step = 0; step < p.steps; ++step) {
                    if (!mbar_wait(bar_empty_p + 8 * ring.slot, ring.phase ^ 1u, abort_flag)) goto done;
                    const uint32_t dst = smem0 + p.off_p + ring.slot * p.packed_slot_bytes;
                    const uint32_t bar = bar_full_p + 8 * ring.slot;
                    mbar_expect_tx(bar, tx_bytes);
                    const int c0 = (step0 + step) * kStepC;
                    if (!TRANSPOSED) {
                        const int gr = c0 / p.g;
                        tma_load_2d(dst, &tm_q, bar, w0, c0 * BITS / 32);
                        tma_load_2d(dst + p.words_bytes, &tm_scales, bar, w0, gr);
                        tma_load_2d(dst + p.words_bytes + p.scale_bytes, &tm_zeros, bar, w0, gr);
                    } else {
                        tma_load_2d(dst, &tm_q, bar, c0, w0 * BITS / 32);
                        tma_load_2d(dst + p.words_bytes, &tm_scales, bar, c0, g_row);
                        tma_load_2d(dst + p.words_bytes + p.scale_bytes, &tm_zeros, bar, c0, g_row);
                    }
                    ring.advance(P);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            const uint32_t idesc = instr_desc((uint32_t)p.BT, TRANSPOSED ? 1u : 0u, 0u);
            const uint32_t idesc_lora = instr_desc((uint32_t)p.BT, 0u, 0u);
            // Descriptors of slot 0; the start-address field (16-byte units) is advanced per slot and per 16-wide MMA step.
            // activation tile: contraction-contiguous rows of 128 B, 128-byte swizzle, 8-row groups 1024 B apart.
            // weight tile: forward = the same layout (rows n); backward = rows are the contraction (n) with 64 k contiguous:
            //   MN-major, 64-element atoms 8192 B apart (LBO), 8-row contraction groups 1024 B apart (SBO).
            const uint64_t b_desc0 = smem_desc(smem0 + p.off_x, 16, 1024, 2);
            const uint64_t a_desc0 = TRANSPOSED ? smem_desc(smem0 + p.off_w, 8192, 1024, 2) : smem_desc(smem0 + p.off_w, 16, 1024, 2);
            constexpr uint32_t a_k16 = TRANSPOSED ? (2048u >> 4) : (32u >> 4);
            const uint32_t x_step = p.x_stage_bytes >> 4;
            Ring ring;
            uint32_t tile_it = 0;
            for (int tile = first_tile; tile < p.n_tiles; tile += tile_stride, ++tile_it) {
                const uint32_t buf = tile_it & 1u;
                const uint32_t d_tmem = tmem_base + buf * kAccStride;
                if (!mbar_wait(bar_acc_empty + 8 * buf, ((tile_it >> 1) & 1u) ^ 1u, abort_flag)) goto done;
                tc_fence_after();
                uint32_t acc = 0;
                for (int step = 0; step < p.steps; ++step) {
                    if (!mbar_wait(bar_full_x + 8 * ring.slot, ring.phase, abort_flag)) goto done;
                    tc_fence_after();
                    const uint64_t b_desc = b_desc0 + ring.slot * x_step;
                    const uint64_t a_desc = a_desc0 + ring.slot * (uint32_t)(kWStageBytes >> 4);
#pragma unroll
                    for (int k16 = 0; k16 < kStepC / 16; ++k16) {
                        tc_mma(d_tmem, a_desc + k16 * a_k16, b_desc + k16 * 2, idesc, acc);
                        acc = 1;
                    }
                    tc_commit(bar_empty + 8 * ring.slot);
                    ring.advance(S);
                }
                if (p.r > 0 && rank == 0) {   // the LoRA update goes into one rank's part only
                    if (!mbar_wait(bar_lora_full, tile_it & 1u, abort_flag)) goto done;
                    tc_fence_after();
                    for (int jb = 0; jb < p.r_pad / 16; ++jb) {
                        // un-swizzled operands: 8-row x 16-byte core matrices 128 B apart (SBO), contraction halves LBO apart
                        const uint64_t a_desc = smem_desc(smem0 + p.off_lora_a + jb * 2 * (kWRows * 16), kWRows * 16, 128, 0);
                        const uint64_t b_desc = smem_desc(smem0 + p.off_lora_p + jb * 2 * (p.BT * 16), p.BT * 16, 128, 0);
                        tc_mma(d_tmem, a_desc, b_desc, idesc_lora, 1u);
                    }
                }
                tc_commit(bar_acc_full + 8 * buf);
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kDequantWarp0) {
        // ------------------------------------------------------------------ epilogue (+ LoRA operand staging)
        const int q = warp & 3;                      // tensor-memory lane quarter this warp may read
        const int et = threadIdx.x - kEpiWarp0 * 32; // 0..127
        pdl_wait();
        uint32_t tile_it = 0;
        for (int tile = first_tile; tile < p.n_tiles; tile += tile_stride, ++tile_it) {
            const int wt = tile / p.n_tok_tiles, tt = tile % p.n_tok_tiles;
            const int w0 = wt * kWRows, m0 = tt * p.BT;
            const uint32_t buf = tile_it & 1u;
            if (p.n_prod > 0 && tile_it == 0 && rank == 0) {
                // P is being computed by this launch's producer clusters: one thread waits for all of their CTAs, is counted
                // as done with the counter, and the last such CTA of the launch zeroes the pair for the next one.
                if (et == 0 && wait_counter(&p.sync[0], (unsigned)(p.n_prod * p.split), abort_flag)) {
                    const unsigned n_cons = gridDim.x / (unsigned)p.split - (unsigned)p.n_prod;   // one waiting CTA per tile cluster
                    if (atomicAdd(&p.sync[1], 1u) == n_cons - 1u) {
                        atomicExch(&p.sync[0], 0u);
                        atomicExch(&p.sync[1], 0u);
                    }
                }
                asm volatile("bar.sync 2, %0;" ::"r"(kEpiWarps * 32) : "memory");
                if (*abort_flag) break;
            }
            if (p.r > 0 && rank == 0) {   // (the LoRA update goes into rank 0's part only)
                // (the previous tile's LoRA MMA has completed: its accumulator-full barrier was observed below)
                uint8_t* la = smem_gen + p.off_lora_a;
                uint8_t* lp = smem_gen + p.off_lora_p;
                const int row = et, wrow = w0 + row;
                for (int jc = 0; jc < p.r_pad / 8; ++jc) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (jc * 8 < p.r && wrow < p.C) {
                        if (!TRANSPOSED) {
                            v = __ldg(reinterpret_cast<const uint4*>(p.L + (size_t)wrow * p.r + jc * 8));      // B[n, j..j+7]
                        } else {
                            uint32_t e[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                e[j] = __bfloat16_as_ushort(__ldg(p.L + (size_t)(jc * 8 + j) * p.K + wrow));     // A[j, k]
                            v = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
                        }
                    }
                    *reinterpret_cast<uint4*>(la + jc * (kWRows * 16) + (row >> 3) * 128 + (row & 7) * 16) = v;
                }
                for (int row_t = et; row_t < p.BT; row_t += 128) {
                    const int m = m0 + row_t;
                    for (int jc = 0; jc < p.r_pad / 8; ++jc) {
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (jc * 8 < p.r && m < p.M) {
                            // (not the read-only path: P may have been written by this launch's producer clusters)
                            const float4 a = __ldcg(reinterpret_cast<const float4*>(p.Pmat + (size_t)m * p.r + jc * 8));
                            const float4 b = __ldcg(reinterpret_cast<const float4*>(p.Pmat + (size_t)m * p.r + jc * 8 + 4));
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(p.s * a.x, p.s * a.y), h1 = __floats2bfloat162_rn(p.s * a.z, p.s * a.w);
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(p.s * b.x, p.s * b.y), h3 = __floats2bfloat162_rn(p.s * b.z, p.s * b.w);
                            v = make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                                           *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
                        }
                        *reinterpret_cast<uint4*>(lp + jc * (p.BT * 16) + (row_t >> 3) * 128 + (row_t & 7) * 16) = v;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_lora_full);
            }
            if (!warp_wait(bar_acc_full + 8 * buf, (tile_it >> 1) & 1u, abort_flag, lane)) break;
            tc_fence_after();
            const int c = w0 + q * 32 + lane;                 // output column owned by this thread
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kAccStride;
            if (p.split > 1) {
                // this rank's part of the tile, fp32 [token][128 weight rows], over the (now idle) operand ring
                float* part = reinterpret_cast<float*>(smem_gen);
#pragma unroll 1
                for (int cb = 0; cb < p.BT; cb += 16) {
                    uint32_t v[16];
                    tc_ld16(taddr + cb, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) part[(cb + j) * kWRows + q * 32 + lane] = __uint_as_float(v[j]);
                }
                tc_fence_before();
                break;
            }
#pragma unroll 1
            for (int cb = 0; cb < p.BT; cb += 16) {
                uint32_t v[16];
                tc_ld16(taddr + cb, v);
                tc_wait_ld();
                if (c < p.C) {
                    __nv_bfloat16* optr = p.Out + (size_t)(m0 + cb) * p.C + c;
                    const int rows_left = p.M - (m0 + cb);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (j < rows_left) *optr = __float2bfloat16_rn(__uint_as_float(v[j]));
                        optr += p.C;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
        }
    } else if (warp >= kDequantWarp0) {
        // ------------------------------------------------------------------ unpack + dequant
        // Two groups of four warps take alternate pipeline stages, so each group has two stage times for its serial chain
        // (wait, shared-memory loads, arithmetic, wait, stores, fence, arrive).  Inside a group a thread owns one column of
        // the packed tile and two blocks of 32 consecutive-k codes.
        const int group = (warp - kDequantWarp0) / kGroupWarps;    // 0 or 1
        const int gt = threadIdx.x - (kDequantWarp0 + group * kGroupWarps) * 32;   // 0..127 inside the group
        const int col = gt % p.packed_cols;                       // column of the packed tile (n in both directions)
        const int kb0 = gt / p.packed_cols;                       // forward: 0; backward: 0..1
        const int kb_stride = TRANSPOSED ? 2 : 1;                 // the thread's two code blocks are kb0 and kb0 + kb_stride
        const uint32_t row_base = (uint32_t)(col >> 3) * 1024u + (uint32_t)(col & 7) * 128u;   // row `col` of a swizzled tile
        const uint32_t sw = (uint32_t)(col & 7);
        uint32_t w_off[2], chunk0[2], srow[2];
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            const int kb = kb0 + b * kb_stride;                   // 32-code block along k: 0..1 forward, 0..3 backward
            w_off[b] = row_base + (TRANSPOSED ? (uint32_t)(kb >> 1) * 8192u : 0u);
            chunk0[b] = (uint32_t)((TRANSPOSED ? (kb & 1) : kb) * 4);
            srow[b] = TRANSPOSED ? (uint32_t)(((kb * 32) / p.g) % p.scale_rows) : 0u;
        }
        const uint32_t pcols = (uint32_t)p.packed_cols;
        const int my_tiles = first_tile < p.n_tiles ? (p.n_tiles - first_tile + tile_stride - 1) / tile_stride : 0;
        const int total = my_tiles * p.steps;
        Ring ring_w, ring_p;
        if (group == 1) { ring_w.advance(S); ring_p.advance(P); }
        for (int it = group; it < total; it += 2) {
            if (!warp_wait(bar_full_p + 8 * ring_p.slot, ring_p.phase, abort_flag, lane)) break;
            const uint8_t* pk = smem_gen + p.off_p + ring_p.slot * p.packed_slot_bytes;
            const uint32_t* pw = reinterpret_cast<const uint32_t*>(pk);
            const __half* ps = reinterpret_cast<const __half*>(pk + p.words_bytes);
            const __half* pz = reinterpret_cast<const __half*>(pk + p.words_bytes + p.scale_bytes);
            uint32_t w[2][BITS];
            __half sc[2], zp[2];
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const uint32_t kb = (uint32_t)(kb0 + b * kb_stride);
#pragma unroll
                for (int i = 0; i < BITS; ++i) w[b][i] = pw[(kb * BITS + i) * pcols + col];
                sc[b] = ps[srow[b] * pcols + col];
                zp[b] = pz[srow[b] * pcols + col];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty_p + 8 * ring_p.slot);

            uint32_t out[2][16];
#pragma unroll
            for (int b = 0; b < 2; ++b) dequant32<BITS>(w[b], group_params(sc[b], zp[b]), out[b]);

            if (!warp_wait(bar_empty + 8 * ring_w.slot, ring_w.phase ^ 1u, abort_flag, lane)) break;
            uint8_t* ws = smem_gen + p.off_w + ring_w.slot * kWStageBytes;
#pragma unroll
            for (int b = 0; b < 2; ++b)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<uint4*>(ws + w_off[b] + (((chunk0[b] + c) ^ sw) << 4)) =
                        make_uint4(out[b][4 * c], out[b][4 * c + 1], out[b][4 * c + 2], out[b][4 * c + 3]);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full_w + 8 * ring_w.slot);
            ring_w.advance(S); ring_w.advance(S);
            ring_p.advance(P); ring_p.advance(P);
        }
    }

done:
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // give copies that may still be in flight time to land before the CTA's memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (p.split > 1) {
        // Add the ranks' parts in rank order (fixed order: deterministic); rank i finishes tokens i * BT / split ...
        __syncwarp();
        cluster_sync_all();
        pdl_wait();            // every thread stores part of the output below
        if (!*abort_flag && first_tile >= 0 && first_tile < p.n_tiles) {
            const int wt = first_tile / p.n_tok_tiles, tt = first_tile % p.n_tok_tiles;
            const int w0 = wt * kWRows, m0 = tt * p.BT;
            const int tok_per_rank = p.BT / p.split;
            const uint32_t part_addr = smem0;
            uint32_t peer[4];
            for (int rk = 0; rk < 4; ++rk) peer[rk] = map_to_cta(part_addr, (uint32_t)(rk < p.split ? rk : 0));
            for (int e = threadIdx.x; e < tok_per_rank * (kWRows / 4); e += kThreads) {   // four weight rows (output columns) at a time
                const int t = rank * tok_per_rank + e / (kWRows / 4), cw = (e % (kWRows / 4)) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int rk = 0; rk < p.split; ++rk) {
                    const float4 x = ld_cluster_f32x4(peer[rk] + (uint32_t)((t * kWRows + cw) * 4));
                    v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
                }
                if (m0 + t < p.M && w0 + cw < p.C) {     // C is a multiple of 8: four columns are all-in or all-out
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                    *reinterpret_cast<uint2*>(p.Out + (size_t)(m0 + t) * p.C + w0 + cw) =
                        make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
                }
            }
        }
        __syncwarp();
        cluster_sync_all();   // nobody leaves while a peer may still read its part
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            f = nullptr;
        return (EncodeTiledFn)f;
    }();
    return fn;
}

bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner, uint64_t outer,
                 uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle sw) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Sets a launch's counter pair to zero.  It is launched like the layer kernels (programmatic stream serialization): it
// lets its successor start at once and writes only after its own predecessor -- whose last tile CTAs may still be
// using the pair -- has completed; the kernel behind it touches the pair only after griddepcontrol.wait, i.e. after this
// grid has completed.
__global__ void sync_zero_kernel(unsigned int* sync) {
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x < kSyncWords) sync[threadIdx.x] = 0u;
}

int zero_sync_pair(unsigned int* sync, cudaStream_t st) {
    return launch_pdl(sync_zero_kernel, dim3(1), dim3(kSyncWords), 0, st, 1, sync) == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// Ldown != NULL: P = In * Ldown is still to be computed.  Where the tile clusters leave room for more clusters on the GPU
// (cudaOccupancyMaxActiveClusters: 33 clusters of 4 fit on 148 SMs, 74 of 2), producer clusters in front of the grid do
// it beside the tiles; else a down-projection launch goes ahead of the kernel.
template <int BITS, bool TRANSPOSED>
int launch_impl(const CUtensorMap& ta, const CUtensorMap& tq, const CUtensorMap& ts, const CUtensorMap& tz, const Params& p_in,
                size_t smem_bytes, int grid, cudaStream_t st, const void* Ldown, unsigned int* sync) {
    static SmemLimit limit;
    static std::mutex mu;
    static int max_clusters_dev[kMaxDevices][5] = {};   // per device, by cluster width
    auto kern = umma_gemm_kernel<BITS, TRANSPOSED>;
    if (!limit.raise(kern, 232448 - 1024)) return QLORA_ERR_CUDA;
    Params p = p_in;
    p.n_prod = 0; p.sync = nullptr; p.wait_limit_us = kWaitLimitUs;
    if (Ldown != nullptr && p.r > 0) {
        std::lock_guard<std::mutex> lock(mu);
        const int dev = device_ordinal();
        int* max_clusters = max_clusters_dev[dev < 0 ? 0 : dev];
        if (max_clusters[p.split] == 0) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(sm_count() / p.split * p.split));
            cfg.blockDim = dim3(kThreads);
            cfg.dynamicSmemBytes = 232448 - 1024;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = (unsigned)p.split; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = -1; }
            max_clusters[p.split] = n;
        }
        const int n_blocks = (p.M + 15) / 16;
        const int idle = max_clusters[p.split] - grid / p.split;
        int n_prod = (n_blocks + p.split - 1) / p.split;           // one row block per producer CTA when there is room
        if (n_prod > idle) n_prod = idle;
        const bool fits = p.r <= 16 && n_prod > 0 && n_prod * p.split * 2 >= n_blocks && p.lds_stages >= LDS_MIN_STAGES;
        if (fits && sync != nullptr) {
            p.n_prod = n_prod;
            p.sync = sync;
            grid += n_prod * p.split;
            const int rc = zero_sync_pair(sync, st);
            if (rc != QLORA_OK) return rc;
        } else {
            const int rc = launch_lora_down(p.M, p.T, p.r, !TRANSPOSED, p.In, p.Ldown, p.Pout, st);
            if (rc != QLORA_OK) return rc;
        }
    }
    // one cluster of p.split CTAs per tile when the contraction is split
    return launch_pdl(kern, dim3((unsigned)grid), dim3(kThreads), smem_bytes, st, (unsigned)p.split, ta, tq, ts, tz, p) == cudaSuccess
               ? QLORA_OK : QLORA_ERR_CUDA;
}

#include "umma_pair.cuh"

}  // namespace

int launch_lora_down_stream(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st) {
    return launch_lora_down_stream_impl(M, T, r, l_is_A, In, L, P, st);
}

bool umma_supported(const qlora_desc& d, int M) {
    if (M < 1) return false;
    if (d.K % 64 != 0 || d.N % 64 != 0) return false;              // contraction steps of 64 in both directions
    if (!(d.group_size == 64 || d.group_size % 128 == 0)) return false;
    if (d.r > 64) return false;
    return true;
}

// Tiles of a partly filled last wave that are split two ways along the contraction (0: none).  Worth it when at most
// half a wave is left over, so that every left-over tile finds two pairs, and the halves are still long enough.
static int pair_split_tiles(int n_tiles, int steps, int pairs) {
    if (n_tiles <= pairs || steps < 16) return 0;
    const int rem = n_tiles % pairs;
    if (rem == 0 || 2 * rem > pairs || 2 + rem > kSyncWords) return 0;
    return rem;
}

// Workspace the CTA-pair kernel may use to exchange the halves of split tiles, forward or backward (0 when M is too small
// for that kernel or nothing is split).
size_t umma_split_scratch_bytes(const qlora_desc& d, int M) {
    if (M <= 256 || !umma_supported(d, M)) return 0;
    const int pairs = sm_count() / 2;
    const int tok_tiles = (M + 4 * kPairTok - 1) / (4 * kPairTok);
    const int rem_f = pair_split_tiles(tok_tiles * ((d.N + 2 * kPairW - 1) / (2 * kPairW)), d.K / kStepC, pairs);
    const int rem_b = pair_split_tiles(tok_tiles * ((d.K + 2 * kPairW - 1) / (2 * kPairW)), d.N / kStepC, pairs);
    return (size_t)(rem_f > rem_b ? rem_f : rem_b) * kSplitTileBytes;
}

// Workspace with which a backward call of this shape can compute dB on its producer clusters: one [N, r] fp32 part per
// producer CTA (0: the CTA-pair kernel would not take dB on).
size_t umma_db_part_bytes(const qlora_desc& d, int M) {
    return (size_t)2 * umma_db_on_producers(d, M) * (size_t)d.N * d.r * sizeof(float);
}

// CTA-pair kernel: 512 tokens x 256 weight rows per pair of SMs (see prefer_pair_kernel for when it is used).
static int launch_umma_pair(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q, const void* scales,
                            const void* zeros, const void* L, float* Pmat, void* Out, cudaStream_t st, const void* Ldown,
                            unsigned int* sync, void* split_buf, size_t split_bytes, DbFuse* db, bool plan_only = false) {
    // plan_only: nothing is launched and no pointer is looked at; the return value is the number of producer pairs when a
    // backward call with every optional workspace area would form dB on them, else 0
    PairParams p{};
    p.M = M; p.N = d.N; p.K = d.K; p.bits = d.bits; p.g = d.group_size; p.r = d.r; p.r_pad = (d.r + 15) / 16 * 16;
    p.C = transposed ? d.K : d.N;
    const int T = transposed ? d.N : d.K;
    p.n_tok_tiles = (M + 4 * kPairTok - 1) / (4 * kPairTok);
    const int n_w_tiles = (p.C + 2 * kPairW - 1) / (2 * kPairW);
    p.n_tiles = p.n_tok_tiles * n_w_tiles;
    p.steps = T / kStepC;
    p.packed_cols = transposed ? 64 : 128;
    p.packed_rows = (transposed ? 128 : 64) * d.bits / 32;
    p.scale_rows = transposed ? (d.group_size >= 128 ? 1 : 128 / d.group_size) : 1;
    p.words_bytes = (uint32_t)(p.packed_rows * p.packed_cols * 4);
    p.scale_bytes = (uint32_t)(p.scale_rows * p.packed_cols * 2);
    p.packed_slot_bytes = (p.words_bytes + 2 * p.scale_bytes + 127u) / 128u * 128u;
    p.s = d.r > 0 ? d.alpha / (float)d.r : 0.f;
    p.Pmat = Pmat; p.L = (const __nv_bfloat16*)L; p.Out = (__nv_bfloat16*)Out;

    uint32_t lora_l = (uint32_t)(kPairW * p.r_pad * 2), lora_p = (uint32_t)(2 * kPairTok * p.r_pad * 2);
    if (lora_l + lora_p < 8192) lora_p = 8192 - lora_l;   // the area doubles as the epilogue's staging slices (4 warps x 2 KiB)
    const uint32_t budget = 232448 - 1024 /*alignment slack*/ - 2048 /*static, barriers, padding*/;
    p.P = 4;
    const uint32_t fixed = lora_l + lora_p + p.P * p.packed_slot_bytes + 512;
    const uint32_t per_stage = kPairXStage + kWStageBytes;
    int S = (int)((budget - fixed) / per_stage);
    if (S > 8) S = 8;
    if (S < 2) return QLORA_ERR_UNSUPPORTED;
    p.S = S;
    p.off_x = 0;
    p.off_w = p.off_x + S * kPairXStage;
    p.off_p = p.off_w + S * kWStageBytes;
    p.off_lora_l = p.off_p + p.P * p.packed_slot_bytes;
    p.off_lora_p = p.off_lora_l + lora_l;
    p.off_bar = (p.off_lora_p + lora_p + 127u) / 128u * 128u;
    const size_t smem_bytes = (size_t)p.off_bar + 512 + 1024;

    const int pairs = sm_count() / 2;
    p.n_prod = 0; p.T = T; p.sync = nullptr; p.wait_limit_us = kWaitLimitUs;
    p.In = (const __nv_bfloat16*)In; p.Ldown = (const __nv_bfloat16*)Ldown; p.Pout = Pmat;
    p.lds_stages = (int)((p.off_bar - LDS_BAR_BYTES) / LDS_STAGE_BYTES);
    if (p.lds_stages > 6) p.lds_stages = 6;
    // P = In * Ldown still to be computed (Ldown given): on SM pairs the tiles leave idle when those can take all row
    // blocks (they are then done well before the tiles' contractions are), else by a launch ahead of this one.  Both sum
    // in the same order.  producers(last) = how many pairs would do it when the last wave has `last` items (0: none can).
    const bool want_p = (Ldown != nullptr || plan_only) && d.r > 0;
    if (plan_only) { sync = reinterpret_cast<unsigned int*>(sizeof(unsigned int)); split_buf = sync; split_bytes = ~(size_t)0; }   // (never dereferenced)
    const int n_blocks = (M + 15) / 16;
    auto producers = [&](int last) {
        // pairs with less to do: no tile at all, or one item fewer than the rest when the last wave is partly filled
        const int idle = p.n_tiles < pairs ? pairs - p.n_tiles : (last ? pairs - last : 0);
        int n_prod = (n_blocks + 3) / 4;                     // four row blocks per producer CTA pair when there is room
        if (n_prod > idle) n_prod = idle;
        const bool fits = want_p && sync != nullptr && d.r <= 16 && n_prod > 0 && n_prod * 2 * LDS_MAXB >= n_blocks &&
                          p.lds_stages >= LDS_MIN_STAGES;
        return fits ? n_prod : 0;
    };
    // A partly filled last wave (more tiles than pairs, at most half a wave left over): each left-over tile goes to two
    // pairs, half of the contraction each, which exchange halves of the result through the workspace -- unless that
    // takes away the idle pairs that would otherwise have computed P beside the tiles (8192 tokens on 4096 x 4096: the
    // down-projection launch it then needs costs what the split wins).
    p.n_full = p.n_tiles; p.nsplit = 1; p.split_buf = nullptr;
    const int rem = pair_split_tiles(p.n_tiles, p.steps, pairs);
    if (rem > 0 && sync != nullptr && split_buf != nullptr && (size_t)rem * kSplitTileBytes <= split_bytes &&
        !(want_p && producers(2 * rem) == 0 && producers(p.n_tiles % pairs) > 0)) {
        p.n_full = p.n_tiles - rem; p.nsplit = 2; p.split_buf = static_cast<float4*>(split_buf);
    }
    if (want_p) p.n_prod = producers(p.nsplit > 1 ? 2 * rem : p.n_tiles % pairs);
    // dB on the producers' pass over dY (backward, ranks up to 16): every producer CTA leaves its part in the workspace
    // -- where the producers have a whole tile's time to spare: with a split last wave they are only half a tile ahead of
    // the others, and the extra work then lengthens the kernel (down_proj backward, r = 16: 159 against 140 us)
    const bool db_fits = transposed && p.n_prod > 0 && p.nsplit == 1 &&
                         p.n_prod * 2 * (d.r <= 8 ? LDS_MAXB : 3) >= n_blocks;   // (two rank tiles: three row blocks per producer CTA at most)
    if (plan_only) return db_fits ? p.n_prod : 0;
    p.with_db = 0;
    if (db != nullptr && db_fits && db->H != nullptr && db->dB != nullptr && db->part != nullptr &&
        (size_t)2 * p.n_prod * (size_t)T * d.r * sizeof(float) <= db->part_bytes) {
        p.with_db = 1; p.db_accumulate = db->accumulate; p.Hmat = db->H; p.db_part = db->part; p.db_out = db->dB;
        db->done = true;
    }
    CUtensorMap ta, tq, ts, tz;
    if (!make_map_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, In, (uint64_t)T, (uint64_t)M, 64, (uint32_t)kPairTok, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&tq, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, Q, (uint64_t)d.N, (uint64_t)(d.K * d.bits / 32), (uint32_t)p.packed_cols, (uint32_t)p.packed_rows, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&ts, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, scales, (uint64_t)d.N, (uint64_t)(d.K / d.group_size), (uint32_t)p.packed_cols, (uint32_t)p.scale_rows, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&tz, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, zeros, (uint64_t)d.N, (uint64_t)(d.K / d.group_size), (uint32_t)p.packed_cols, (uint32_t)p.scale_rows, CU_TENSOR_MAP_SWIZZLE_NONE))
        return QLORA_ERR_CUDA;

    if (want_p && p.n_prod == 0) {
        const int rc = launch_lora_down(M, T, d.r, !transposed, In, Ldown, Pmat, st);
        if (rc != QLORA_OK) return rc;
    }
    if (p.n_prod > 0 || p.nsplit > 1) {                      // the counters in the workspace are in use: zero them in stream order
        p.sync = sync;
        const int rc = zero_sync_pair(sync, st);
        if (rc != QLORA_OK) return rc;
    }
    const int grid = 2 * (p.n_tiles < pairs ? p.n_tiles + p.n_prod : pairs);
#define QLORA_LAUNCH_PAIR(B)                                                                              \
    return transposed ? launch_pair_impl<B, true>(ta, tq, ts, tz, p, smem_bytes, grid, st)                \
                      : launch_pair_impl<B, false>(ta, tq, ts, tz, p, smem_bytes, grid, st)
    switch (d.bits) {
        case 2: QLORA_LAUNCH_PAIR(2);
        case 3: QLORA_LAUNCH_PAIR(3);
        case 4: QLORA_LAUNCH_PAIR(4);
        case 8: QLORA_LAUNCH_PAIR(8);
    }
#undef QLORA_LAUNCH_PAIR
    return QLORA_ERR_UNSUPPORTED;
}

// Between 257 and 1024 tokens either tensor-core kernel may be the faster one: the pair kernel's tiles (512 tokens x 256
// weight rows) leave most SM pairs without one on a 4096-wide layer (42 us against 23 at 512 tokens), but fill a wave
// exactly where the single-CTA kernel's 128 x 256 tiles need two (11008 outputs: 45 against 68 us).  The choice follows
// a small cost model fitted to measurements: waves of tiles times (steps x time per step + fixed part) for each kernel.
static bool prefer_pair_kernel(const qlora_desc& d, int M, bool transposed) {
    if (M <= 256) return false;
    if (M > 1024) return true;
    const int T = transposed ? d.N : d.K, C = transposed ? d.K : d.N;
    const int steps = T / kStepC, sms = sm_count();
    const int tiles_mid = ((M + 255) / 256) * ((C + kWRows - 1) / kWRows);
    int split = 1;
    for (int sp = 4; sp >= 2; sp /= 2)
        if (tiles_mid * sp <= sms && steps % sp == 0 && steps / sp >= 4) { split = sp; break; }
    const int waves_mid = split > 1 ? 1 : (tiles_mid + sms - 1) / sms;
    const float mid_us = (float)waves_mid * ((float)(steps / split) * 0.29f + 15.0f);
    const int tiles_pair = ((M + 4 * kPairTok - 1) / (4 * kPairTok)) * ((C + 2 * kPairW - 1) / (2 * kPairW));
    const int waves_pair = (tiles_pair + sms / 2 - 1) / (sms / 2);
    const float pair_us = (float)waves_pair * ((float)steps * 0.62f + 4.0f);
    return pair_us < mid_us;
}

// The number of producer pairs on which the backward call of this shape, given its whole workspace, forms dB (on the current
// device: its SM count decides how many pairs the tiles leave idle); 0 when dB goes to the gradient kernels.
int umma_db_on_producers(const qlora_desc& d, int M) {
    if (M <= 256 || d.r == 0 || d.r > 16 || !umma_supported(d, M) || !prefer_pair_kernel(d, M, true)) return 0;
    const int rc = launch_umma_pair(d, M, true, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                                    nullptr, 0, nullptr, true);
    return rc > 0 ? rc : 0;
}

int launch_umma_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q, const void* scales,
                     const void* zeros, const void* L, float* Pmat, void* Out, cudaStream_t st, const void* Ldown,
                     unsigned int* sync, void* split_buf, size_t split_bytes, DbFuse* db) {
    if (prefer_pair_kernel(d, M, transposed))
        return launch_umma_pair(d, M, transposed, In, Q, scales, zeros, L, Pmat, Out, st, Ldown, sync, split_buf, split_bytes, db);
    Params p{};
    p.M = M; p.N = d.N; p.K = d.K; p.bits = d.bits; p.g = d.group_size; p.r = d.r; p.r_pad = (d.r + 15) / 16 * 16;
    p.C = transposed ? d.K : d.N;
    const int T = transposed ? d.N : d.K;
    p.BT = M > 128 ? 256 : (M > 64 ? 128 : (M > 32 ? 64 : 32));
    p.n_tok_tiles = (M + p.BT - 1) / p.BT;
    const int n_w_tiles = (p.C + kWRows - 1) / kWRows;
    p.n_tiles = p.n_tok_tiles * n_w_tiles;
    p.steps = T / kStepC;
    p.packed_cols = transposed ? 64 : 128;
    p.packed_rows = (transposed ? 128 : 64) * d.bits / 32;
    p.scale_rows = transposed ? (d.group_size >= 128 ? 1 : 128 / d.group_size) : 1;
    p.words_bytes = (uint32_t)(p.packed_rows * p.packed_cols * 4);
    p.scale_bytes = (uint32_t)(p.scale_rows * p.packed_cols * 2);
    p.packed_slot_bytes = (p.words_bytes + 2 * p.scale_bytes + 127u) / 128u * 128u;
    p.x_stage_bytes = (uint32_t)(p.BT * 128);
    p.s = d.r > 0 ? d.alpha / (float)d.r : 0.f;
    p.Pmat = Pmat; p.L = (const __nv_bfloat16*)L; p.Out = (__nv_bfloat16*)Out;

    // shared-memory plan (offsets from a 1024-byte aligned base)
    const uint32_t lora_a = (uint32_t)(kWRows * p.r_pad * 2), lora_p = (uint32_t)(p.BT * p.r_pad * 2);
    const uint32_t budget = 232448 - 1024 /*alignment slack*/ - 2048 /*static, barriers, padding*/;
    // With few tokens the kernel is bound by the latency of streaming cold packed weights through a handful of CTAs,
    // so the packed ring is deep (bytes in flight), at the cost of one or two operand stages.
    const uint32_t per_stage = p.x_stage_bytes + kWStageBytes;
    int S = 0;
    uint32_t fixed = 0;
    for (p.P = p.BT <= 128 ? 16 : 8; p.P >= 4; p.P -= 4) {   // the packed ring gives way until three operand stages fit
        fixed = lora_a + lora_p + p.P * p.packed_slot_bytes + 512;
        S = budget > fixed ? (int)((budget - fixed) / per_stage) : 0;
        if (S >= 3 || p.P == 4) break;
    }
    if (S > 8) S = 8;
    if (S < 2) return QLORA_ERR_UNSUPPORTED;
    p.S = S;
    p.off_x = 0;
    p.off_w = p.off_x + S * p.x_stage_bytes;
    p.off_p = p.off_w + S * kWStageBytes;
    p.off_lora_a = p.off_p + p.P * p.packed_slot_bytes;
    p.off_lora_p = p.off_lora_a + lora_a;
    p.off_bar = (p.off_lora_p + lora_p + 127u) / 128u * 128u;
    const size_t smem_bytes = (size_t)p.off_bar + 512 + 1024;

    CUtensorMap ta, tq, ts, tz;
    if (!make_map_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, In, (uint64_t)T, (uint64_t)M, 64, (uint32_t)p.BT, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&tq, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, Q, (uint64_t)d.N, (uint64_t)(d.K * d.bits / 32), (uint32_t)p.packed_cols, (uint32_t)p.packed_rows, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&ts, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, scales, (uint64_t)d.N, (uint64_t)(d.K / d.group_size), (uint32_t)p.packed_cols, (uint32_t)p.scale_rows, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&tz, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, zeros, (uint64_t)d.N, (uint64_t)(d.K / d.group_size), (uint32_t)p.packed_cols, (uint32_t)p.scale_rows, CU_TENSOR_MAP_SWIZZLE_NONE))
        return QLORA_ERR_CUDA;

    // Few tiles (few tokens): split each tile's contraction over a cluster of 2 or 4 CTAs so that the whole GPU streams
    // the weights.  Needs one tile per cluster, an even split of the steps, and room for the fp32 part in the operand ring.
    p.split = 1;
    for (int sp = 4; sp >= 2; sp /= 2) {
        if (p.n_tiles * sp <= sm_count() && p.steps % sp == 0 && p.steps / sp >= 4 && p.BT % sp == 0 &&
            (uint32_t)(kWRows * p.BT * 4) <= p.off_p) { p.split = sp; break; }
    }
    p.steps /= p.split;
    const int grid = p.split > 1 ? p.n_tiles * p.split : (p.n_tiles < sm_count() ? p.n_tiles : sm_count());
    p.T = T; p.In = (const __nv_bfloat16*)In; p.Ldown = (const __nv_bfloat16*)Ldown; p.Pout = Pmat;
    p.lds_stages = (int)((p.off_bar - LDS_BAR_BYTES) / LDS_STAGE_BYTES);
    if (p.lds_stages > 6) p.lds_stages = 6;
#define QLORA_LAUNCH(B)                                                                              \
    return transposed ? launch_impl<B, true>(ta, tq, ts, tz, p, smem_bytes, grid, st, Ldown, sync)  \
                      : launch_impl<B, false>(ta, tq, ts, tz, p, smem_bytes, grid, st, Ldown, sync)
    switch (d.bits) {
        case 2: QLORA_LAUNCH(2);
        case 3: QLORA_LAUNCH(3);
        case 4: QLORA_LAUNCH(4);
        case 8: QLORA_LAUNCH(8);
    }
#undef QLORA_LAUNCH
    return QLORA_ERR_UNSUPPORTED;
}

namespace {
// The give-up path of the bounded waits, exercised without stalling any real kernel: one thread of one CTA waits with
// the library's own mbar_wait on a barrier in shared memory that nobody ever arrives at, with `limit_us` as the limit.  The
// wait runs out, sets the sticky status word and returns false; the kernel then ends normally (no TMA, no tensor memory).
__global__ void wait_probe_kernel(int limit_us) {
    __shared__ uint64_t bar;
    __shared__ int flag[2];
    if (threadIdx.x == 0) {
        flag[0] = 0; flag[1] = limit_us;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) (void)mbar_wait(smem_u32(&bar), 0u, flag);
}
}  // namespace

int launch_wait_probe(int limit_us, cudaStream_t st) {
    wait_probe_kernel<<<1, 32, 0, st>>>(limit_us);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

int read_device_status(unsigned int* out, int clear) {
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)) != cudaSuccess) return QLORA_ERR_CUDA;
    if (clear && v != 0) {
        const unsigned int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return QLORA_ERR_CUDA;
    }
    *out = v;
    return QLORA_OK;
}

}  // namespace qlora
