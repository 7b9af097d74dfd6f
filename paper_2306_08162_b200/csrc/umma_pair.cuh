// CTA-pair variant of the tensor-core kernel (included by umma_kernel.cu, inside its anonymous namespace).
//
// Two CTAs on the two SMs of one TPC (a cluster of 2) work on one output tile of 512 tokens x 256 weight rows with
// tcgen05.mma.cta_group::2 (M = 256 across the pair, N = 256):
//   - tokens are the MMA's M side (A operand): each CTA stages 2 x 128 token rows per pipeline stage by TMA and owns the
//     accumulator rows of those tokens in its own tensor memory (two accumulators of 256 columns = all 512 columns);
//   - the dequantised weights are the N side (B operand): each CTA unpacks 128 weight rows per stage into its own shared
//     memory; the tensor cores of the pair exchange the halves, so a dequantised weight is reused by 512 tokens and each
//     SM reads only half of the weight operand and half of the activations a single-CTA tile would need.
// Per stage and per SM this is 1024 tensor-core cycles against 32 KB of TMA fill, 16 KB of dequant stores and 64 KB of
// operand reads, i.e. about half the shared-memory and L2 traffic per flop of the single-CTA kernel.
//
// The MMA is issued by one thread of the pair's first CTA (the leader).  Barriers the leader waits on (activation
// tile landed, weight tile written, accumulators drained, LoRA operands staged) live in the leader's shared memory
// and collect arrivals from both CTAs (remote mbarrier arrive / TMA complete_tx); barriers that both CTAs wait on
// (stage free, accumulators complete) exist in both and are signalled by one multicast tcgen05.commit.
// Every wait is bounded, as in the single-CTA kernel; the CTAs leave together through a cluster barrier.
//
// When some SM pairs have less to do than others -- no tile at all (fewer tiles than pairs), or one tile fewer than the
// rest (the last wave is partly filled) -- `n_prod` of them are producers: the first clusters of the grid (lowest block
// indices, so they are dispatched first and wait for nobody) first compute the LoRA down-projection P = In * Ldown
// (lora_down_stream.cuh) beside the others' main loops, publish it through a counter in device memory, and then take
// their own (fewer) tiles; a tile's epilogue warps wait for that counter before they stage P for the LoRA update, which is only needed
// once the tile's contraction is through.  The counter pair belongs to one launch at a time (the host hands out one
// pair per workspace) and the last CTA to have seen the count zeroes it again.

//
// When the tiles make more than one wave and at most half a wave is left over (172 tiles on 74 pairs: 24), each left-over
// tile is worked on by two pairs, one half of the contraction steps each, as the last thing both do.  The pair with the
// lower block indices then gives its half of the fp32 result away through the caller's workspace and is done; the other
// waits for it (bounded), adds the two halves and stores the tile -- so the third wave costs about three quarters of a tile
// instead of a whole one.  Every wait in this kernel points from higher block indices to lower ones (tiles wait for producer
// clusters, the finishing half of a split tile for the giving half), i.e. to CTAs that were dispatched earlier.

constexpr int kPairTok = 128;                          // token rows per CTA per accumulator
constexpr int kPairW = 128;                            // weight rows per CTA (256 per pair tile)
constexpr int kPairXSub = kPairTok * kStepC * 2;       // 16 KiB: one 128-token sub-tile of a stage
constexpr int kPairXStage = 2 * kPairXSub;             // two accumulators' sub-tiles

struct PairParams {
    int M, N, K, bits, g, r, r_pad;
    int C;                       // output columns (N forward, K backward)
    int n_tok_tiles, n_tiles, steps;
    // Last wave split along the contraction: tiles [n_full, n_tiles) are each worked on by two SM pairs (nsplit == 2), one
    // half of the steps each; nsplit == 1: n_full == n_tiles, nothing is split.
    int n_full, nsplit;
    float4* split_buf;           // fp32 exchange area of the split tiles (workspace)
    int S, P;
    int packed_cols, packed_rows, scale_rows;
    uint32_t words_bytes, scale_bytes, packed_slot_bytes;
    uint32_t off_x, off_w, off_p, off_lora_l, off_lora_p, off_bar;
    float s;
    const float* Pmat;           // H (forward) or G (backward), fp32 [M, r]
    const __nv_bfloat16* L;      // B [N, r] (forward) or A [r, K] (backward)
    __nv_bfloat16* Out;
    // producer clusters (n_prod > 0): P = In * Ldown is computed by this launch and written to Pout (== Pmat)
    int n_prod, T, lds_stages;
    unsigned int* sync;          // the launch's counter pair (n_prod > 0)
    int wait_limit_us;           // every wait inside the kernel gives up after this long
    const __nv_bfloat16* In;     // [M, T]
    const __nv_bfloat16* Ldown;  // A [r, K] (forward) or B [N, r] (backward)
    float* Pout;
    // backward with producer clusters only: dB = s dY^T H computed on the producers' pass over dY (with_db)
    int with_db, db_accumulate;
    const float* Hmat;           // H fp32 [M, r]
    float* db_part;              // [2 n_prod][N][r] fp32, one part per producer CTA (workspace)
    float* db_out;               // dB fp32 [N, r]
};


__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait on a barrier that receives arrivals from the peer CTA.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    uint64_t t0 = 0;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
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
// TMA tile load of a CTA pair: the transfer lands in this CTA's shared memory, its bytes are counted on `bar`, which may
// be the leader's barrier (a shared::cluster address).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on the barrier at the same shared-memory offset in both CTAs of the pair once all MMAs issued so far complete.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// Instruction descriptor for the pair: bf16 x bf16 -> fp32, M = 256 across the two CTAs.
__device__ __forceinline__ uint32_t instr_desc_pair(uint32_t n_mma, uint32_t a_mn_major, uint32_t b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major << 15) | (b_mn_major << 16) | ((n_mma >> 3) << 17) |
           ((256u >> 4) << 24);
}

// What worker pair `w` of `W` does, in order: the whole tiles w, w + W, ... below n_full, then (last, if at all) its half
// of a split tile.  Workers 2i and 2i + 1 share split tile n_full + i.
struct PairItem { int tile, s0, s1, part, nparts; };
__device__ __forceinline__ int pair_item_count(const PairParams& p, int w, int W) {
    const int full = w < p.n_full ? (p.n_full - w + W - 1) / W : 0;
    return full + ((p.nsplit > 1 && w < (p.n_tiles - p.n_full) * p.nsplit) ? 1 : 0);
}
__device__ __forceinline__ PairItem pair_item(const PairParams& p, int w, int W, int it) {
    PairItem r;
    const int full = w < p.n_full ? (p.n_full - w + W - 1) / W : 0;
    if (it < full) { r.tile = w + it * W; r.s0 = 0; r.s1 = p.steps; r.part = 0; r.nparts = 1; }
    else {
        r.tile = p.n_full + w / p.nsplit; r.part = w % p.nsplit; r.nparts = p.nsplit;
        // (the giving half, part 0, takes 27 of 64 steps: it has its result to write out before the other half, which waits
        // for it, can begin to add; 25 .. 33 were timed, 27 is the shallow minimum)
        const int cut = p.steps * 27 / 64;
        r.s0 = r.part == 0 ? 0 : cut; r.s1 = r.part == 0 ? cut : p.steps;
    }
    return r;
}

template <int BITS, bool TRANSPOSED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_q,
                 const __grid_constant__ CUtensorMap tm_scales, const __grid_constant__ CUtensorMap tm_zeros,
                 const PairParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s[2];   // [0] set when a wait gave up, [1] the launch's wait limit in microseconds
    volatile int* abort_flag = abort_flag_s;
    pdl_launch_dependents();

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem0 - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t S = (uint32_t)p.S, P = (uint32_t)p.P;
    const uint32_t cta = cluster_ctarank();            // 0 = leader (issues the MMAs), 1 = follower
    // Work distribution: the launch has `tile_stride` worker pairs; worker w takes tiles w, w + tile_stride, ...  The first
    // n_prod clusters of the grid are producers (down-projection first, see above) and take the HIGHEST worker indices,
    // i.e. the workers with the fewest tiles -- none at all when the tiles do not fill a wave.
    const int tile_stride = (int)(gridDim.x >> 1);
    const bool is_producer = (int)(blockIdx.x >> 1) < p.n_prod;
    const int first_tile = is_producer ? tile_stride - 1 - (int)(blockIdx.x >> 1) : (int)(blockIdx.x >> 1) - p.n_prod;   // = the worker index
    const int n_items = pair_item_count(p, first_tile, tile_stride);

    // barriers (same offsets in both CTAs)
    // One "stage full" barrier per slot collects both operand streams -- the TMA bytes of both CTAs' activation sub-tiles
    // (one expect_tx arrival) and the arrivals of both CTAs' dequant warps: the MMA-issuing thread's per-stage work (eight
    // tcgen05.mma, one wait, one commit) is what paces the main loop, and a second wait per stage cost 4 % of the kernel.
    const uint32_t bar_full_x = smem0 + p.off_bar;          // [S] leader's: activation sub-tiles landed (TMA) + weight tiles written
    const uint32_t bar_full_w = bar_full_x;                 //     (the same barriers: dequant warps arrive on them)
    const uint32_t bar_empty = bar_full_x + 8 * S;          // [S] both: MMAs reading the stage have completed (multicast commit)
    const uint32_t bar_full_p = bar_empty + 8 * S;          // [P] local: packed words + group parameters landed (TMA)
    const uint32_t bar_empty_p = bar_full_p + 8 * P;        // [P] local: the dequant group has read them into registers
    const uint32_t bar_acc_full = bar_empty_p + 8 * P;      // [1] both: accumulators complete (multicast commit)
    const uint32_t bar_acc_empty = bar_acc_full + 8;        // [1] leader's: both CTAs' epilogues have drained the accumulators
    const uint32_t bar_lora_full = bar_acc_empty + 8;       // [1] leader's: both CTAs' LoRA operand tiles staged

    if (threadIdx.x == 0) {
        abort_flag_s[0] = 0; abort_flag_s[1] = p.wait_limit_us;
        for (uint32_t i = 0; i < S; ++i) {
            mbar_init(bar_full_x + 8 * i, 1 + 2 * kGroupWarps);
            mbar_init(bar_empty + 8 * i, 1);
        }
        for (uint32_t i = 0; i < P; ++i) {
            mbar_init(bar_full_p + 8 * i, 1);
            mbar_init(bar_empty_p + 8 * i, kGroupWarps);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 2 * kEpiWarps);
        mbar_init(bar_lora_full, 2 * kEpiWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // whole warp, in both CTAs: all 512 tensor-memory columns of each SM of the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the peer's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // Set-up done.  The weight producer starts at once (the frozen weights are read-only for every call of the library);
    // the roles that touch activations, P or the output call pdl_wait() first.

    if (is_producer) {
        // ------------------------------------------------------------------ producer cluster: LoRA down-projection first
        // (this CTA's row blocks: blockIdx.x, blockIdx.x + 2 n_prod, ...; the ring takes the operand area, below the barriers)
        pdl_wait();
        bool db_here = false;                // (the parts are added up by the tile CTAs, see the epilogue)
        if constexpr (TRANSPOSED) {
            if (p.with_db) {       // the same pass over dY also gives this CTA's part of dB
                db_here = true;
                float* part = p.db_part + (size_t)blockIdx.x * p.T * p.r;
                if (p.r <= 8) lora_down_stream<false, 1, true>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, 2 * p.n_prod, smem_gen, p.lds_stages, abort_flag, p.Hmat, part);
                else          lora_down_stream<false, 2, true, 3>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, 2 * p.n_prod, smem_gen, p.lds_stages, abort_flag, p.Hmat, part);   // (two rank tiles: registers for three row blocks per CTA only; the host sees to it)
            }
        }
        if (!db_here) {
            if (p.r <= 8) lora_down_stream<!TRANSPOSED, 1>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, 2 * p.n_prod, smem_gen, p.lds_stages, abort_flag);
            else          lora_down_stream<!TRANSPOSED, 2>(p.M, p.T, p.r, p.In, p.Ldown, p.Pout, (int)blockIdx.x, 2 * p.n_prod, smem_gen, p.lds_stages, abort_flag);
        }
        __threadfence();       // every thread's rows of P (and of its part of dB) are visible device-wide before the CTA is counted
        __syncthreads();
        if (threadIdx.x == 0) atomicAdd(&p.sync[0], 1u);
        fence_proxy_async();   // the shared memory just used goes to the TMA / tensor-core side for this cluster's tiles, if any
        __syncthreads();
    }
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: activation sub-tiles
        if (lane == 0) {
            pdl_wait();
            Ring ring;
            const uint32_t leader_full_x = map_to_cta(bar_full_x, 0);
            for (int it = 0; it < n_items; ++it) {
                const PairItem item = pair_item(p, first_tile, tile_stride, it);
                const int tile = item.tile;
                const int m0 = (tile % p.n_tok_tiles) * (4 * kPairTok) + (int)cta * kPairTok;
                for (int step = item.s0; step < item.s1; ++step) {
                    if (!mbar_wait(bar_empty + 8 * ring.slot, ring.phase ^ 1u, abort_flag)) goto done;
                    if (cta == 0) mbar_expect_tx(bar_full_x + 8 * ring.slot, 2 * kPairXStage);   // both CTAs' bytes
                    const uint32_t dst = smem0 + p.off_x + ring.slot * kPairXStage;
                    const uint32_t bar = leader_full_x + 8 * ring.slot;
                    tma_load_2d_pair(dst, &tm_act, bar, step * kStepC, m0);
                    tma_load_2d_pair(dst + kPairXSub, &tm_act, bar, step * kStepC, m0 + 2 * kPairTok);
                    ring.advance(S);
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ TMA producer: packed codes, scales, zeros (local)
        if (lane == 0) {
            Ring ring;
            const uint32_t tx_bytes = p.words_bytes + 2 * p.scale_bytes;
            for (int it = 0; it < n_items; ++it) {
                const PairItem item = pair_item(p, first_tile, tile_stride, it);
                const int tile = item.tile;
                const int w0 = (tile / p.n_tok_tiles) * (2 * kPairW) + (int)cta * kPairW;
                const int g_row = TRANSPOSED ? w0 / p.g : 0;
                for (int step = item.s0; step < item.s1; ++step) {
                    if (!mbar_wait(bar_empty_p + 8 * ring.slot, ring.phase ^ 1u, abort_flag)) goto done;
                    const uint32_t dst = smem0 + p.off_p + ring.slot * p.packed_slot_bytes;
                    const uint32_t bar = bar_full_p + 8 * ring.slot;
                    mbar_expect_tx(bar, tx_bytes);
                    const int c0 = step * kStepC;
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
        // ------------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (lane == 0 && cta == 0) {
            const uint32_t idesc = instr_desc_pair(2 * kPairW, 0u, TRANSPOSED ? 1u : 0u);
            const uint32_t idesc_lora = instr_desc_pair(2 * kPairW, 0u, 0u);
            // activation sub-tile (A operand): contraction-contiguous rows of 128 B, 128-byte swizzle, 8-row groups 1024 B apart.
            // weight tile (B operand): forward = the same layout (rows n); backward = rows are the contraction (n) with 64 k
            //   contiguous: MN-major, 64-element atoms 8192 B apart (LBO), 8-row contraction groups 1024 B apart (SBO).
            const uint64_t a_desc0 = smem_desc(smem0 + p.off_x, 16, 1024, 2);
            const uint64_t b_desc0 = TRANSPOSED ? smem_desc(smem0 + p.off_w, 8192, 1024, 2) : smem_desc(smem0 + p.off_w, 16, 1024, 2);
            constexpr uint32_t b_k16 = TRANSPOSED ? (2048u >> 4) : (32u >> 4);
            Ring ring;
            uint32_t tile_it = 0;
            for (int it = 0; it < n_items; ++it, ++tile_it) {
                const PairItem item = pair_item(p, first_tile, tile_stride, it);
                if (!mbar_wait_cluster(bar_acc_empty, (tile_it & 1u) ^ 1u, abort_flag)) goto done;
                tc_fence_after();
                uint32_t acc = 0;
                for (int step = item.s0; step < item.s1; ++step) {
                    if (!mbar_wait_cluster(bar_full_x + 8 * ring.slot, ring.phase, abort_flag)) goto done;
                    tc_fence_after();
                    const uint64_t a_desc = a_desc0 + ring.slot * (uint32_t)(kPairXStage >> 4);
                    const uint64_t b_desc = b_desc0 + ring.slot * (uint32_t)(kWStageBytes >> 4);
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int k16 = 0; k16 < kStepC / 16; ++k16)
                            tc_mma_pair(tmem_base + a * kAccStride, a_desc + a * (kPairXSub >> 4) + k16 * 2, b_desc + k16 * b_k16,
                                        idesc, acc | (uint32_t)(k16 > 0));
                    acc = 1;
                    tc_commit_pair(bar_empty + 8 * ring.slot);
                    ring.advance(S);
                }
                if (p.r > 0 && item.part == 0) {       // (the LoRA update goes into part 0's sum only; a split item is a worker's last)
                    if (!mbar_wait_cluster(bar_lora_full, tile_it & 1u, abort_flag)) goto done;
                    tc_fence_after();
                    for (int a = 0; a < 2; ++a)
                        for (int jb = 0; jb < p.r_pad / 16; ++jb) {
                            // un-swizzled operands: 8-row x 16-byte core matrices 128 B apart (SBO), contraction halves LBO apart
                            const uint64_t a_desc = smem_desc(smem0 + p.off_lora_p + a * (kPairTok * p.r_pad * 2) + jb * 2 * (kPairTok * 16),
                                                              kPairTok * 16, 128, 0);
                            const uint64_t b_desc = smem_desc(smem0 + p.off_lora_l + jb * 2 * (kPairW * 16), kPairW * 16, 128, 0);
                            tc_mma_pair(tmem_base + a * kAccStride, a_desc, b_desc, idesc_lora, 1u);
                        }
                }
                tc_commit_pair(bar_acc_full);
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kDequantWarp0) {
        // ------------------------------------------------------------------ epilogue (+ LoRA operand staging), both CTAs
        const int q = warp & 3;                      // tensor-memory lane quarter this warp may read
        const int et = threadIdx.x - kEpiWarp0 * 32; // 0..127
        const uint32_t leader_acc_empty = map_to_cta(bar_acc_empty, 0);
        const uint32_t leader_lora_full = map_to_cta(bar_lora_full, 0);
        pdl_wait();
        uint32_t tile_it = 0;
        for (int it = 0; it < n_items; ++it, ++tile_it) {
            const PairItem item = pair_item(p, first_tile, tile_stride, it);
            const int tile = item.tile;
            const int wt = tile / p.n_tok_tiles, tt = tile % p.n_tok_tiles;
            const int w0 = wt * (2 * kPairW);                          // first weight row (output column) of the pair tile
            const int m0 = tt * (4 * kPairTok) + (int)cta * kPairTok;  // this CTA's first token row of accumulator 0
            if (p.n_prod > 0 && tile_it == 0) {
                // P is being computed by the producer clusters of this launch: one thread waits for all of their CTAs, is
                // counted as done with the counter, and the last such CTA of the launch zeroes the pair for the next one.
                if (et == 0 && wait_counter(&p.sync[0], 2u * (unsigned)p.n_prod, abort_flag)) {
                    const unsigned n_cons = 2u * (unsigned)(p.n_tiles < tile_stride ? p.n_tiles : tile_stride);   // CTAs that have a tile
                    if (atomicAdd(&p.sync[1], 1u) == n_cons - 1u) {
                        atomicExch(&p.sync[0], 0u);
                        atomicExch(&p.sync[1], 0u);
                    }
                }
                asm volatile("bar.sync 2, %0;" ::"r"(kEpiWarps * 32) : "memory");
                if (*abort_flag) break;
                if constexpr (TRANSPOSED) {
                    if (p.with_db) {
                        // dB: every producer CTA has left its part of s dY^T H in the workspace.  The CTAs that have a tile share
                        // the columns; each adds the parts in producer order for its share, scales and writes dB -- here, while
                        // its main loop still runs and these warps would only wait for it.  (A wait of producers for one
                        // another would point from low block indices to high ones; this one points the safe way.)
                        const int n_cons = 2 * (p.n_tiles < tile_stride ? p.n_tiles : tile_stride);
                        const int me = 2 * first_tile + (int)cta;
                        const int n_blocks = (p.M + 15) >> 4, n_ctas = 2 * p.n_prod;
                        const int n_src = n_ctas < n_blocks ? n_ctas : n_blocks;            // producer CTAs beyond the row blocks wrote nothing
                        const size_t part_elems = (size_t)p.T * p.r, total4 = part_elems / 4;
                        const size_t e_lo = total4 * me / n_cons, e_hi = total4 * (me + 1) / n_cons;
                        for (size_t e4 = e_lo + et; e4 < e_hi; e4 += kEpiWarps * 32) {
                            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                            int src = 0;
                            for (; src + 4 <= n_src; src += 4) {       // four parts in flight, added in producer order
                                float4 x[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) x[i] = __ldcg(reinterpret_cast<const float4*>(p.db_part + (size_t)(src + i) * part_elems) + e4);
#pragma unroll
                                for (int i = 0; i < 4; ++i) { v.x += x[i].x; v.y += x[i].y; v.z += x[i].z; v.w += x[i].w; }
                            }
                            for (; src < n_src; ++src) {
                                const float4 x = __ldcg(reinterpret_cast<const float4*>(p.db_part + (size_t)src * part_elems) + e4);
                                v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
                            }
                            v.x *= p.s; v.y *= p.s; v.z *= p.s; v.w *= p.s;
                            float4* dst = reinterpret_cast<float4*>(p.db_out) + e4;
                            if (p.db_accumulate) { const float4 o = *dst; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
                            *dst = v;
                        }
                    }
                }
            }
            if (p.r > 0 && item.part == 0) {
                // (the previous tile's LoRA MMA has completed: its accumulator-full barrier was observed below)
                uint8_t* ll = smem_gen + p.off_lora_l;
                uint8_t* lp = smem_gen + p.off_lora_p;
                {   // this CTA's 128 weight rows of B (forward) / columns of A (backward)
                    const int row = et, wrow = w0 + (int)cta * kPairW + row;
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
                        *reinterpret_cast<uint4*>(ll + jc * (kPairW * 16) + (row >> 3) * 128 + (row & 7) * 16) = v;
                    }
                }
#pragma unroll
                for (int a = 0; a < 2; ++a) {   // this CTA's token rows of s * H (or s * G) for both accumulators
                    const int m = m0 + a * (2 * kPairTok) + et;
                    for (int jc = 0; jc < p.r_pad / 8; ++jc) {
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (jc * 8 < p.r && m < p.M) {
                            // (not the read-only path: P may have been written by this launch's producer clusters)
                            const float4 x = __ldcg(reinterpret_cast<const float4*>(p.Pmat + (size_t)m * p.r + jc * 8));
                            const float4 y = __ldcg(reinterpret_cast<const float4*>(p.Pmat + (size_t)m * p.r + jc * 8 + 4));
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(p.s * x.x, p.s * x.y), h1 = __floats2bfloat162_rn(p.s * x.z, p.s * x.w);
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(p.s * y.x, p.s * y.y), h3 = __floats2bfloat162_rn(p.s * y.z, p.s * y.w);
                            v = make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                                           *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
                        }
                        *reinterpret_cast<uint4*>(lp + a * (kPairTok * p.r_pad * 2) + jc * (kPairTok * 16) + (et >> 3) * 128 + (et & 7) * 16) = v;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_lora_full);
            }
            if (!warp_wait(bar_acc_full, tile_it & 1u, abort_flag, lane)) break;
            tc_fence_after();
            // Tensor memory hands each thread one token row: 32 consecutive output columns per load = 64 bytes of bf16.  Stored
            // straight from there, one warp instruction would touch 32 different rows (32 cache lines, 16 bytes each), so the
            // chunk takes a turn through a 2 KiB per-warp staging slice (in the LoRA operand area, idle by now): written by
            // row, read back so that four lanes cover the 64 bytes of one row and an instruction covers 8 rows.  The 16-byte
            // pieces are XOR-swizzled by row so that both passes are free of bank conflicts.  Two register buffers: the
            // tensor-memory load of the next 32 columns is in flight while the current ones are converted and stored.
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            uint8_t* slice = smem_gen + p.off_lora_l + (et >> 5) * 2048;
            const int m_w0 = m0 + q * 32;                               // this warp's first token row in accumulator 0
            auto store_chunk = [&](const uint32_t (&v)[32], int idx) {  // chunk idx: accumulator idx / 8, columns (idx % 8) * 32 ..
                __syncwarp();                                           // the previous chunk has been read back
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const __nv_bfloat162 pr = __floats2bfloat162_rn(__uint_as_float(v[c8 * 8 + 2 * j]),
                                                                        __uint_as_float(v[c8 * 8 + 2 * j + 1]));
                        o[j] = *reinterpret_cast<const uint32_t*>(&pr);
                    }
                    *reinterpret_cast<uint4*>(slice + lane * 64 + ((c8 ^ ((lane >> 1) & 3)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
                __syncwarp();
                const int cb = (idx & 7) * 32 + (lane & 3) * 8;         // this lane's 8 columns of the chunk
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int R = 8 * i + (lane >> 2);
                    const uint4 val = *reinterpret_cast<const uint4*>(slice + R * 64 + (((lane & 3) ^ ((R >> 1) & 3)) << 4));
                    const int m = m_w0 + (idx >> 3) * (2 * kPairTok) + R;
                    if (m < p.M && w0 + cb < p.C)                       // C is a multiple of 8: 8 columns are all-in or all-out
                        *reinterpret_cast<uint4*>(p.Out + (size_t)m * p.C + w0 + cb) = val;
                }
            };
            if (item.nparts > 1) {
                // A split tile: this pair holds the sum over its half of the contraction.  The pair with the lower block indices
                // (part 0, whose sum also carries the LoRA update) gives its whole half away -- fp32 through the workspace, laid out
                // so that a warp's stores and the reader's loads are contiguous -- counts its two CTAs in at the tile's counter
                // and is done; the other pair waits for that count (bounded), adds the peer's part to its own chunk by chunk, and
                // stores the tile.  The wait points from high block indices to low ones only: the pair waited for was dispatched
                // first and waits for nobody, whatever else shares the GPU.  (a + b is the same in either order.)
                const int slot = tile - p.n_full;
                float4* buf = p.split_buf + (size_t)(slot * 2 + (int)cta) * (16 * 8 * 128);     // [chunk][j4][thread]
                auto chunk_addr = [&](int idx) { return taddr + (uint32_t)((idx >> 3) * kAccStride + (idx & 7) * 32); };
                if (item.part == 0) {
                    auto give = [&](const uint32_t (&v)[32], int idx) {
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4)
                            buf[(idx * 8 + j4) * 128 + et] = make_float4(__uint_as_float(v[4 * j4]), __uint_as_float(v[4 * j4 + 1]),
                                                                         __uint_as_float(v[4 * j4 + 2]), __uint_as_float(v[4 * j4 + 3]));
                    };
                    uint32_t va[32], vb[32];                 // the tensor-memory load of the next chunk is in flight while this one is stored
                    tc_ld32(chunk_addr(0), va);
#pragma unroll 1
                    for (int idx = 0; idx < 16; idx += 2) {
                        tc_wait_ld();
                        tc_ld32(chunk_addr(idx + 1), vb);
                        give(va, idx);
                        tc_wait_ld();
                        if (idx + 2 < 16) tc_ld32(chunk_addr(idx + 2), va);
                        give(vb, idx + 1);
                    }
                    __threadfence();
                    asm volatile("bar.sync 2, %0;" ::"r"(kEpiWarps * 32) : "memory");
                    if (et == 0) atomicAdd(&p.sync[2 + slot], 1u);
                } else {
                    if (et == 0) wait_counter(&p.sync[2 + slot], 2u, abort_flag);
                    asm volatile("bar.sync 2, %0;" ::"r"(kEpiWarps * 32) : "memory");
                    if (*abort_flag) break;
                    uint32_t va[32];
                    float4 pa[8], pb[8];                     // the peer's part of the next chunk is requested before this one is added and stored
                    auto take = [&](float4 (&pv)[8], int idx) {
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4) pv[j4] = __ldcg(buf + (idx * 8 + j4) * 128 + et);
                    };
                    auto add = [&](uint32_t (&v)[32], const float4 (&pv)[8]) {
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4) {
                            v[4 * j4] = __float_as_uint(__uint_as_float(v[4 * j4]) + pv[j4].x);
                            v[4 * j4 + 1] = __float_as_uint(__uint_as_float(v[4 * j4 + 1]) + pv[j4].y);
                            v[4 * j4 + 2] = __float_as_uint(__uint_as_float(v[4 * j4 + 2]) + pv[j4].z);
                            v[4 * j4 + 3] = __float_as_uint(__uint_as_float(v[4 * j4 + 3]) + pv[j4].w);
                        }
                    };
                    take(pa, 0);
#pragma unroll 1
                    for (int idx = 0; idx < 16; idx += 2) {
                        tc_ld32(chunk_addr(idx), va);
                        take(pb, idx + 1);
                        tc_wait_ld();
                        add(va, pa);
                        store_chunk(va, idx);
                        tc_ld32(chunk_addr(idx + 1), va);
                        if (idx + 2 < 16) take(pa, idx + 2);
                        tc_wait_ld();
                        add(va, pb);
                        store_chunk(va, idx + 1);
                    }
                }
            } else {
                uint32_t va[32], vb[32];
                tc_ld32(taddr, va);
#pragma unroll 1
                for (int idx = 0; idx < 16; idx += 2) {
                    tc_wait_ld();
                    tc_ld32(taddr + ((idx + 1) >> 3) * kAccStride + ((idx + 1) & 7) * 32, vb);
                    store_chunk(va, idx);
                    tc_wait_ld();
                    if (idx + 2 < 16) tc_ld32(taddr + ((idx + 2) >> 3) * kAccStride + ((idx + 2) & 7) * 32, va);
                    store_chunk(vb, idx + 1);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
        }
    } else if (warp >= kDequantWarp0) {
        // ------------------------------------------------------------------ unpack + dequant of this CTA's 128 weight rows
        const int group = (warp - kDequantWarp0) / kGroupWarps;    // 0 or 1: the groups take alternate stages
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
        const uint32_t leader_full_w = map_to_cta(bar_full_w, 0);
        int total = 0;                                           // this worker's stages, whole tiles and split item alike
        for (int it = 0; it < n_items; ++it) {
            const PairItem item = pair_item(p, first_tile, tile_stride, it);
            total += item.s1 - item.s0;
        }
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
            if (lane == 0) mbar_arrive_cluster(leader_full_w + 8 * ring_w.slot);
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
    cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while its peer may still signal it or read its operands
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

template <int BITS, bool TRANSPOSED>
int launch_pair_impl(const CUtensorMap& ta, const CUtensorMap& tq, const CUtensorMap& ts, const CUtensorMap& tz, const PairParams& p,
                     size_t smem_bytes, int grid, cudaStream_t st) {
    static SmemLimit limit;
    auto kern = umma_pair_kernel<BITS, TRANSPOSED>;
    if (!limit.raise(kern, 232448 - 1024)) return QLORA_ERR_CUDA;
    return launch_pdl(kern, dim3((unsigned)grid), dim3(kThreads), smem_bytes, st, 1, ta, tq, ts, tz, p) == cudaSuccess
               ? QLORA_OK : QLORA_ERR_CUDA;   // (the cluster width of 2 is a compile-time attribute of the kernel)
}
