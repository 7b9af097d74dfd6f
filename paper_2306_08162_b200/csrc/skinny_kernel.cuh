// Small-token-count kernels (M <= 32) of the quantized-linear + LoRA layer; included by umma_kernel.cu inside its
// anonymous namespace after umma_pair.cuh (they share the TMA / mbarrier / cluster helpers and the device status word).
//
// With a handful of tokens the layer is bound by streaming the packed weights from HBM once, so these kernels are built
// around bytes in flight and around not re-reading anything else: a cluster of four CTAs owns 128 output columns and
// splits the CONTRACTION four ways (CTA rank i takes the 256-wide stages i, i + 4, ...), so the 16-token activation tile
// and the adapter tile of a stage are fetched by one CTA per 128 columns rather than by every CTA, and a LLaMA-7B
// projection still spreads over 128 or more SMs.  A producer warp issues
// TMA loads of the packed-word tile, the scale / zero rows, the activation tile (128-byte swizzle) and the adapter tile
// into a shared-memory ring; sixteen consumer warps unpack from shared memory and feed the warp-level tensor-core
// instruction (mma.sync m16n8k16, bf16 in, fp32 accumulate).  The partial tiles are then added in (rank, plane) order
// through distributed shared memory (CTA i reduces columns 32 i .. 32 i + 31: fixed order, deterministic), the LoRA
// update is applied in fp32 and the result rounded once to bf16.  A CTA layer (blockIdx.z) covers 16 tokens; more
// tokens re-read the weights through L2.
//
//   forward  (Y = X W^T + s H B^T): stage = 256 k x 128 columns n.  Warps 0-7 take the CTA's even stages, warps 8-15 the odd
//     ones; within a stage a warp takes 32 columns and 128 k.  Lane (g, q) owns the 32 consecutive-k codes of block
//     4 (k half) + q for the four columns 4g .. 4g+3 (one 16-byte
//     shared-memory read per packed row), dequantises them with the library's dequant32 and uses them as B fragments; the
//     contraction index inside the 128 is permuted the same way for the activation fragments, which leaves the sum unchanged.
//   backward (dX = dY W + s G A): stage = 256 n x 128 output features k.  The contraction now runs across packed columns,
//     so a fragment register needs two neighbouring n for one k: each lane extracts the two codes (k, k+1) of its own
//     column and the 8 x 8 tile is transposed across the warp with movmatrix -- the register-level form of the paper's
//     "transpose of the packed matrix" (Section 3.1).  A warp takes 32 output features and 128 n of its stages.
// LoRA: for r <= 16 the down-projection (H = X A^T, G = dY B) rides along as one or two extra fragment tiles, so there is
// no separate launch; larger ranks read H / G computed by the skinny pre-kernel.

constexpr int SK_WARPS = 16;                        // consumer warps; warp 16 is the TMA producer
constexpr int SK_THREADS = (SK_WARPS + 1) * 32;
constexpr int SK_STAGE = 256;                       // contraction elements per ring stage
constexpr int SK_TILE = 128;                        // output columns per cluster (32 per CTA after the reduction)
constexpr int SK_SPLIT = 4;                         // CTAs per cluster = ways the contraction is split
constexpr int SK_MAX_STAGES = 8;
constexpr int SK_PW = SK_TILE + 16;                 // row pitch (floats) of a partial tile: 128 outputs + 16 fused H / G columns
constexpr int SK_PLANES = 4;                        // partial tiles per CTA: (even / odd stages) x (two halves of a stage)

struct SkinnyParams {
    int M, N, K, bits, g, r;
    int T;                       // contraction length (K forward, N backward)
    int C;                       // output columns (N forward, K backward)
    int stages_total, S;
    int scale_rows;              // group rows per stage
    uint32_t words_bytes, scale_bytes, stage_bytes;
    uint32_t off_scale, off_zero, off_act, off_l;   // inside a stage; activation and adapter tiles 1024-aligned
    uint32_t act_bytes, l_bytes; // bytes the TMA loads of a stage bring for them
    uint32_t off_p, off_bar;
    float s;
    const __nv_bfloat16* Lup;    // B [N, r] (forward) or A [r, K] (backward): the adapter applied second
    const __nv_bfloat16* Ldown;  // A [r, K] (forward) or B [N, r] (backward): the adapter applied first (fused ranks only)
    float* P;                    // H / G fp32 [M, r]: written by one CTA when fused, read otherwise
    int p_is_input;
    __nv_bfloat16* Out;
};

// Two consecutive codes (2 * pair_in_tile, +1 of the 8-code tile `t` of a 32-code block) of one column -> bf16 pair.
template <int BITS>
__device__ __forceinline__ uint32_t dequant_pair(const uint32_t (&w)[BITS], int t, int qq, const GroupParams& gp) {
    uint32_t c0, c1;
    if constexpr (BITS == 4) {
        const uint32_t v = w[t] >> (8 * qq);
        c0 = v & 0xFu; c1 = (v >> 4) & 0xFu;
    } else if constexpr (BITS == 2) {
        const uint32_t v = w[t >> 1] >> (16 * (t & 1) + 4 * qq);
        c0 = v & 0x3u; c1 = (v >> 2) & 0x3u;
    } else if constexpr (BITS == 8) {
        const uint32_t v = ((qq & 2) ? w[2 * t + 1] : w[2 * t]) >> (16 * (qq & 1));
        c0 = v & 0xFFu; c1 = (v >> 8) & 0xFFu;
    } else {   // 3 bits: 6 bits at stream position 24 t + 6 qq, possibly straddling two words
        const uint32_t sh = 24u * (uint32_t)t + 6u * (uint32_t)qq;
        const uint32_t wi = sh >> 5;
        const uint32_t lo = wi == 0 ? w[0] : (wi == 1 ? w[1] : w[2]);
        const uint32_t hi = wi == 0 ? w[1] : (wi == 1 ? w[2] : 0u);
        const uint32_t v = __funnelshift_r(lo, hi, sh & 31u);
        c0 = v & 0x7u; c1 = (v >> 3) & 0x7u;
    }
    if constexpr (BITS == 2 || BITS == 4) {
        return bf16x2_scale((c0 | (c1 << 16)) | 0x43004300u, gp);
    } else {
        const float f0 = (__uint_as_float(c0 | 0x4B000000u) - gp.bias) * gp.scale;
        const float f1 = (__uint_as_float(c1 | 0x4B000000u) - gp.bias) * gp.scale;
        const __nv_bfloat162 pr = __floats2bfloat162_rn(f0, f1);
        return *reinterpret_cast<const uint32_t*>(&pr);
    }
}

__device__ __forceinline__ void sk_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t sk_movmatrix(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t sk_comp(const uint4& v, int i) { return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w)); }
// Producer warp.  Issuing a TMA load costs its thread some tens of nanoseconds, so the loads of a stage are spread over
// four lanes and the ring slots over the lane quads: lanes 4 s .. 4 s + 3 own slot s and issue its stages in order (one
// owner per slot keeps the parity waits on the slot's barriers one phase apart).
//   x_pack, y_pack: coordinates of the stage-0 packed tile; the stage index advances y (forward) or x (backward).
template <bool TRANSPOSED, int NTL>
__device__ __forceinline__ void sk_producer(const SkinnyParams& p, const CUtensorMap* tq, const CUtensorMap* ts, const CUtensorMap* tz,
                                            const CUtensorMap* tact, const CUtensorMap* tl, uint32_t smem0, uint32_t bar_full,
                                            uint32_t bar_empty, int c0, int mrow0, int rank, int lane, volatile int* abort_flag) {
    const int slot = lane >> 2, job = lane & 3;
    if (slot >= p.S || job == 3 || (job == 2 && (NTL == 0 || !TRANSPOSED))) return;   // (forward: the consumers read A themselves)
    if (job == 1) pdl_wait();                                            // the activations may come from the preceding kernel
    int it = slot;                                                       // this CTA's it-th stage
    for (int st = rank + SK_SPLIT * slot; st < p.stages_total; st += SK_SPLIT * p.S, it += p.S) {
        const uint32_t lap = (uint32_t)(it / p.S);
        if (!mbar_wait(bar_empty + 8 * slot, (lap & 1u) ^ 1u, abort_flag)) return;
        const uint32_t dst = smem0 + (uint32_t)slot * p.stage_bytes;
        const uint32_t bar = bar_full + 8 * slot;
        const int t0 = st * SK_STAGE;                                   // first contraction index of the stage
        if (job == 0) {
            mbar_expect_tx(bar, p.words_bytes + 2 * p.scale_bytes + p.act_bytes + (NTL > 0 && TRANSPOSED ? p.l_bytes : 0u));
            if (!TRANSPOSED) {   // c0 = first output column n; packed rows walk K
                tma_load_2d(dst, tq, bar, c0, st * (SK_STAGE / 32) * p.bits);
                tma_load_2d(dst + p.off_scale, ts, bar, c0, t0 / p.g);
                tma_load_2d(dst + p.off_zero, tz, bar, c0, t0 / p.g);
            } else {             // c0 = first output feature k (multiple of 256); packed columns walk N
                tma_load_2d(dst, tq, bar, t0, (c0 / 32) * p.bits);
                tma_load_2d(dst + p.off_scale, ts, bar, t0, c0 / p.g);
                tma_load_2d(dst + p.off_zero, tz, bar, t0, c0 / p.g);
            }
        } else if (job == 1) {
#pragma unroll
            for (int sb = 0; sb < SK_STAGE / 64; ++sb)                   // 16 token rows x 64 contraction elements per box
                tma_load_2d(dst + p.off_act + sb * 2048, tact, bar, t0 + 64 * sb, mrow0);
        } else {
            tma_load_2d(dst + p.off_l, tl, bar, 0, t0);                 // backward: B[n, 0 .. r) for the stage's 256 n
        }
    }
}

// part: [SK_PLANES][16][SK_PW] fp32 in every CTA of the cluster (columns 128.. hold the fused H / G partials).  CTA `rank`
// adds the partial tiles in (rank, plane) order for its 32 columns, applies the LoRA update and stores bf16.
template <bool TRANSPOSED, int NTL>
__device__ __forceinline__ void sk_cluster_epilogue(const SkinnyParams& p, uint32_t part_addr, float* ps, int c0, int mrow0, int rank) {
    const int tid = threadIdx.x;
    uint32_t peer[SK_SPLIT];
#pragma unroll
    for (int rk = 0; rk < SK_SPLIT; ++rk) peer[rk] = map_to_cta(part_addr, (uint32_t)rk);
    // This thread's output element (threads 0 .. 511), its row of the second adapter (requested first, so that the global
    // loads are in flight during the reductions) and its sum over the partial tiles.
    const bool has_out = tid < 16 * 32;
    const int m = tid >> 5, c = tid & 31;
    const int row = mrow0 + m, col = c0 + 32 * rank + c;
    const bool live = has_out && row < p.M && col < p.C;
    float lup[8 * (NTL > 0 ? NTL : 1)];
    if constexpr (NTL > 0) {
#pragma unroll
        for (int j = 0; j < 8 * NTL; ++j) lup[j] = 0.f;
        if (live) {
            if (!TRANSPOSED) {        // B[n, 0 .. r): 16 bytes per eight ranks (backward: A[j, k] is strided, read below)
#pragma unroll
                for (int lt = 0; lt < NTL; ++lt)
                    if (lt * 8 < p.r) {
                        const uint4 b = __ldg(reinterpret_cast<const uint4*>(p.Lup + (size_t)col * p.r + lt * 8));
                        lup[lt * 8 + 0] = bf16_lo(b.x); lup[lt * 8 + 1] = bf16_hi(b.x); lup[lt * 8 + 2] = bf16_lo(b.y); lup[lt * 8 + 3] = bf16_hi(b.y);
                        lup[lt * 8 + 4] = bf16_lo(b.z); lup[lt * 8 + 5] = bf16_hi(b.z); lup[lt * 8 + 6] = bf16_lo(b.w); lup[lt * 8 + 7] = bf16_hi(b.w);
                    }
            }
        }
    }
    float v = 0.f;
    if (has_out) {
#pragma unroll
        for (int rk = 0; rk < SK_SPLIT; ++rk)
#pragma unroll
            for (int h = 0; h < SK_PLANES; ++h) v += ld_cluster_f32(peer[rk] + (uint32_t)(((h * 16 + m) * SK_PW + 32 * rank + c) * 4));
    }
    if constexpr (NTL > 0) {
        for (int e = tid; e < 16 * 8 * NTL; e += SK_THREADS) {
            const int mm = e / (8 * NTL), j = e % (8 * NTL);
            float h = 0.f;
#pragma unroll
            for (int rk = 0; rk < SK_SPLIT; ++rk)
#pragma unroll
                for (int pl = 0; pl < SK_PLANES; ++pl) h += ld_cluster_f32(peer[rk] + (uint32_t)(((pl * 16 + mm) * SK_PW + SK_TILE + j) * 4));
            ps[mm * 16 + j] = h;
            if (blockIdx.y == 0 && rank == 0 && mrow0 + mm < p.M && j < p.r) p.P[(size_t)(mrow0 + mm) * p.r + j] = h;
        }
        __syncthreads();
    }
    if (!live) return;
    if (p.r > 0) {
        float lo = 0.f;
        if constexpr (NTL > 0 && !TRANSPOSED) {
#pragma unroll
            for (int j = 0; j < 8 * NTL; ++j) lo = fmaf(ps[m * 16 + j], lup[j], lo);     // ranks beyond r: zero times zero
        } else if constexpr (NTL > 0) {
            for (int j = 0; j < p.r; ++j) lo = fmaf(ps[m * 16 + j], __bfloat162float(p.Lup[(size_t)j * p.K + col]), lo);   // A[j, k]
        } else {
            for (int j = 0; j < p.r; ++j) {
                const float pj = __ldg(p.P + (size_t)row * p.r + j);
                const float l = TRANSPOSED ? __bfloat162float(p.Lup[(size_t)j * p.K + col])     // A[j, k]
                                           : __bfloat162float(p.Lup[(size_t)col * p.r + j]);    // B[n, j]
                lo = fmaf(pj, l, lo);
            }
        }
        v += p.s * lo;
    }
    p.Out[(size_t)row * p.C + col] = __float2bfloat16_rn(v);
}

#define SK_COMMON_PROLOGUE()                                                                                         \
    pdl_launch_dependents();                                                                                        \
    extern __shared__ uint8_t smem_raw[];                                                                           \
    __shared__ int abort_flag_s;                                                                                    \
    volatile int* abort_flag = &abort_flag_s;                                                                       \
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;                                                   \
    uint8_t* smem_gen = smem_raw + (smem0 - smem_u32(smem_raw));                                                    \
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;                                                     \
    const int g = lane >> 2, q = lane & 3;                                                                          \
    const uint32_t bar_full = smem0 + p.off_bar, bar_empty = bar_full + 8 * SK_MAX_STAGES;                          \
    float* part = reinterpret_cast<float*>(smem_gen);          /* reuses the ring after the main loop */            \
    float* ps = reinterpret_cast<float*>(smem_gen + p.off_p);                                                       \
    const int rank = (int)cluster_ctarank();                                                                        \
    const int c0 = blockIdx.y * SK_TILE;                                                                            \
    const int mrow0 = blockIdx.z * 16;                                                                              \
    if (threadIdx.x == 0) {                                                                                         \
        abort_flag_s = 0;                                                                                           \
        for (int i = 0; i < p.S; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, SK_WARPS / 2); } \
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");                                          \
    }                                                                                                               \
    __syncthreads();   /* set-up done.  The frozen weights and the adapters are read-only for every call of the library, so  \
                          their loads start at once; whatever the preceding work in the stream may have produced (the      \
                          activations, P) or may still be reading (the outputs) is touched only after pdl_wait().  */

// After the main loop: every consumer warp has read every stage this CTA loaded, so no TMA write is still to come and
// the ring's memory can hold the partial tiles; then the cluster reduces them.  On an abort nothing is stored.
#define SK_COMMON_EPILOGUE(TRANSPOSED_)                                                                              \
    __syncthreads();                                                                                                \
    if (*abort_flag) for (int i = 0; i < 200; ++i) __nanosleep(1000);   /* let copies in flight land */               \
    __syncwarp();                                                                                                   \
    cluster_sync_all();                    /* all eight partial tiles are written */                                \
    pdl_wait();                            /* P may come from, and Out may still be read by, the preceding kernel */ \
    if (!*abort_flag) sk_cluster_epilogue<TRANSPOSED_, NTL>(p, smem0, ps, c0, mrow0, rank);                          \
    __syncwarp();                                                                                                   \
    cluster_sync_all();                    /* nobody leaves while a peer may still read its partial tile */

template <int BITS, int NTL>
__global__ void __cluster_dims__(SK_SPLIT, 1, 1) __launch_bounds__(SK_THREADS, 1)
skinny_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_s,
                  const __grid_constant__ CUtensorMap tm_z, const __grid_constant__ CUtensorMap tm_act,
                  const __grid_constant__ CUtensorMap tm_l, const SkinnyParams p) {
    SK_COMMON_PROLOGUE();
    float acc[4][4], accL[NTL > 0 ? NTL : 1][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
    for (int i = 0; i < (NTL > 0 ? NTL : 1); ++i) accL[i][0] = accL[i][1] = accL[i][2] = accL[i][3] = 0.f;
    if (warp == SK_WARPS) {
        sk_producer<false, NTL>(p, &tm_q, &tm_s, &tm_z, &tm_act, &tm_l, smem0, bar_full, bar_empty, c0, mrow0, rank, lane, abort_flag);
    } else {
        const int cg = warp & 3, kh = (warp >> 2) & 1, sh = warp >> 3;   // 32 columns cg, 128 k kh of this CTA's stages of parity sh
        const int blk = 4 * kh + q;                               // this lane's 32-code block inside the stage
        for (int it = sh, st = rank + SK_SPLIT * sh; st < p.stages_total; st += 2 * SK_SPLIT, it += 2) {
            const uint32_t slot = (uint32_t)(it % p.S), lap = (uint32_t)(it / p.S);
            // the fused H tile (computed once per cluster column block): this lane's A fragments -- rank lt * 8 + g, its 32 k
            // -- come straight from global memory (A is small, read-only and shared by every CTA, so it sits in L2),
            // requested before the wait for the stage, which hides their latency
            uint4 la[NTL > 0 ? NTL : 1][4];
            if (NTL > 0 && cg == 0) {
                const int k0 = st * SK_STAGE + 32 * blk;
#pragma unroll
                for (int lt = 0; lt < NTL; ++lt)
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
                        la[lt][jj] = (lt * 8 + g < p.r && k0 + 8 * jj < p.K)
                                         ? __ldg(reinterpret_cast<const uint4*>(p.Ldown + (size_t)(lt * 8 + g) * p.K + k0 + 8 * jj))
                                         : make_uint4(0, 0, 0, 0);
            }
            if (!warp_wait(bar_full + 8 * slot, lap & 1u, abort_flag, lane)) break;
            const uint8_t* stg = smem_gen + slot * p.stage_bytes;
            uint4 w4[BITS];
#pragma unroll
            for (int u = 0; u < BITS; ++u)
                w4[u] = *reinterpret_cast<const uint4*>(stg + ((size_t)(blk * BITS + u) * SK_TILE + 32 * cg + 4 * g) * 4);
            const int srow = p.scale_rows > 1 ? (blk * 32) / p.g : 0;
            const uint2 sc2 = *reinterpret_cast<const uint2*>(stg + p.off_scale + ((size_t)srow * SK_TILE + 32 * cg + 4 * g) * 2);
            const uint2 zp2 = *reinterpret_cast<const uint2*>(stg + p.off_zero + ((size_t)srow * SK_TILE + 32 * cg + 4 * g) * 2);
            // activation fragments: token rows g and g + 8, this lane's 32 k = 64 bytes = chunks 4 (blk & 1) .. + 3 of the
            // 128-byte row of sub-box blk / 2 (chunk index XOR row, the TMA's 128-byte swizzle); rows beyond M are zero
            const uint8_t* xrow = stg + p.off_act + (blk >> 1) * 2048 + g * 128;
            uint4 xa[4], xb[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int off = (((4 * (blk & 1) + jj) ^ g) << 4);
                xa[jj] = *reinterpret_cast<const uint4*>(xrow + off);
                xb[jj] = *reinterpret_cast<const uint4*>(xrow + 1024 + off);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t w[BITS];
#pragma unroll
                for (int u = 0; u < BITS; ++u) w[u] = sk_comp(w4[u], i);
                const uint32_t sraw = (i < 2 ? sc2.x : sc2.y) >> (16 * (i & 1));
                const uint32_t zraw = (i < 2 ? zp2.x : zp2.y) >> (16 * (i & 1));
                const GroupParams gp = group_params(__ushort_as_half((unsigned short)(sraw & 0xFFFFu)),
                                                    __ushort_as_half((unsigned short)(zraw & 0xFFFFu)));
                uint32_t out[16];
                dequant32<BITS>(w, gp, out);
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    sk_mma(acc[i], xa[jj].x, xb[jj].x, xa[jj].y, xb[jj].y, out[4 * jj], out[4 * jj + 1]);
                    sk_mma(acc[i], xa[jj].z, xb[jj].z, xa[jj].w, xb[jj].w, out[4 * jj + 2], out[4 * jj + 3]);
                }
            }
            if (NTL > 0 && cg == 0) {
#pragma unroll
                for (int lt = 0; lt < NTL; ++lt)
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        sk_mma(accL[lt], xa[jj].x, xb[jj].x, xa[jj].y, xb[jj].y, la[lt][jj].x, la[lt][jj].y);
                        sk_mma(accL[lt], xa[jj].z, xb[jj].z, xa[jj].w, xb[jj].w, la[lt][jj].z, la[lt][jj].w);
                    }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(SK_WARPS * 32) : "memory");   // all consumer warps are out of the ring
        // accumulator element (i, c): token g (+8 for c >= 2), column 32 cg + 4 (2q + (c & 1)) + i; plane 2 sh + kh
        float* mine = part + (size_t)(2 * sh + kh) * 16 * SK_PW;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * SK_PW + 32 * cg + 4 * (2 * q + (c & 1)) + i] = acc[i][c];
        if (cg == 0) {
#pragma unroll
            for (int lt = 0; lt < 2; ++lt)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    mine[(g + ((c & 2) ? 8 : 0)) * SK_PW + SK_TILE + lt * 8 + 2 * q + (c & 1)] = lt < NTL ? accL[lt < NTL ? lt : 0][c] : 0.f;
        }
    }
    SK_COMMON_EPILOGUE(false)
}

template <int BITS, int NTL>
__global__ void __cluster_dims__(SK_SPLIT, 1, 1) __launch_bounds__(SK_THREADS, 1)
skinny_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_s,
                  const __grid_constant__ CUtensorMap tm_z, const __grid_constant__ CUtensorMap tm_act,
                  const __grid_constant__ CUtensorMap tm_l, const SkinnyParams p) {
    SK_COMMON_PROLOGUE();
    float acc[4][4], accG[NTL > 0 ? NTL : 1][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
    for (int i = 0; i < (NTL > 0 ? NTL : 1); ++i) accG[i][0] = accG[i][1] = accG[i][2] = accG[i][3] = 0.f;
    if (warp == SK_WARPS) {
        sk_producer<true, NTL>(p, &tm_q, &tm_s, &tm_z, &tm_act, &tm_l, smem0, bar_full, bar_empty, c0, mrow0, rank, lane, abort_flag);
    } else {
        const int kbl = warp & 3, nh = (warp >> 2) & 1, sh = warp >> 3;   // 32 output features kbl, 128 contraction columns nh, stage parity sh
        const int srow = p.scale_rows > 1 ? (kbl * 32) / p.g : 0;
        for (int it = sh, st = rank + SK_SPLIT * sh; st < p.stages_total; st += 2 * SK_SPLIT, it += 2) {
            const uint32_t slot = (uint32_t)(it % p.S), lap = (uint32_t)(it / p.S);
            if (!warp_wait(bar_full + 8 * slot, lap & 1u, abort_flag, lane)) break;
            const uint8_t* stg = smem_gen + slot * p.stage_bytes;
            const uint32_t* pw = reinterpret_cast<const uint32_t*>(stg) + (size_t)kbl * BITS * SK_STAGE;
            const __half* psc = reinterpret_cast<const __half*>(stg + p.off_scale) + (size_t)srow * SK_STAGE;
            const __half* pzp = reinterpret_cast<const __half*>(stg + p.off_zero) + (size_t)srow * SK_STAGE;
#pragma unroll 2
            for (int sidx = 0; sidx < 8; ++sidx) {                // 16-wide contraction steps of this warp's 128 columns
                const int nl = 128 * nh + 16 * sidx;
                // dY fragments: rows g, g + 8 of sub-box nl / 64; byte 2 (nl % 64) + 4q of the 128-byte row (+16 for n + 8),
                // 16-byte chunk index XOR row (the TMA's 128-byte swizzle); rows beyond M and columns beyond N are zero
                const uint8_t* yrow = stg + p.off_act + (nl >> 6) * 2048 + g * 128;
                const int bo = 2 * (nl & 63) + 4 * q;
                uint32_t a[4];
                a[0] = *reinterpret_cast<const uint32_t*>(yrow + ((((bo >> 4)) ^ g) << 4) + (bo & 15));
                a[1] = *reinterpret_cast<const uint32_t*>(yrow + 1024 + ((((bo >> 4)) ^ g) << 4) + (bo & 15));
                a[2] = *reinterpret_cast<const uint32_t*>(yrow + ((((bo >> 4) + 1) ^ g) << 4) + (bo & 15));
                a[3] = *reinterpret_cast<const uint32_t*>(yrow + 1024 + ((((bo >> 4) + 1) ^ g) << 4) + (bo & 15));
                uint32_t w[2][BITS];                              // columns nl + g and nl + 8 + g
                __half sc[2], zp[2];
#pragma unroll
                for (int cset = 0; cset < 2; ++cset) {
                    const int col = nl + 8 * cset + g;
#pragma unroll
                    for (int u = 0; u < BITS; ++u) w[cset][u] = pw[u * SK_STAGE + col];
                    sc[cset] = psc[col];
                    zp[cset] = pzp[col];
                }
                const GroupParams gpa = group_params(sc[0], zp[0]);
                const GroupParams gpb = group_params(sc[1], zp[1]);
#pragma unroll
                for (int t = 0; t < 4; ++t) {                     // output features 32 kbl + 8t .. + 7
                    const uint32_t b0 = sk_movmatrix(dequant_pair<BITS>(w[0], t, q, gpa));
                    const uint32_t b1 = sk_movmatrix(dequant_pair<BITS>(w[1], t, q, gpb));
                    sk_mma(acc[t], a[0], a[1], a[2], a[3], b0, b1);
                }
                if (NTL > 0 && kbl == 0) {                        // G = dY B, once per cluster: rank pairs transposed into contraction pairs
#pragma unroll
                    for (int lt = 0; lt < NTL; ++lt) {
                        const uint8_t* lrow = stg + p.off_l + (size_t)(nl + g) * (2 * p.r) + lt * 16 + 4 * q;
                        const uint32_t va = *reinterpret_cast<const uint32_t*>(lrow);
                        const uint32_t vb = *reinterpret_cast<const uint32_t*>(lrow + 8 * (2 * p.r));
                        sk_mma(accG[lt], a[0], a[1], a[2], a[3], sk_movmatrix(va), sk_movmatrix(vb));
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
        }
        asm volatile("bar.sync 1, %0;" ::"r"(SK_WARPS * 32) : "memory");   // all consumer warps are out of the ring
        // accumulator element (t, c): token g (+8 for c >= 2), output feature 32 kbl + 8t + 2q + (c & 1); plane 2 sh + nh
        float* mine = part + (size_t)(2 * sh + nh) * 16 * SK_PW;
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * SK_PW + 32 * kbl + 8 * t + 2 * q + (c & 1)] = acc[t][c];
        if (kbl == 0) {
#pragma unroll
            for (int lt = 0; lt < 2; ++lt)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    mine[(g + ((c & 2) ? 8 : 0)) * SK_PW + SK_TILE + lt * 8 + 2 * q + (c & 1)] = lt < NTL ? accG[lt < NTL ? lt : 0][c] : 0.f;
        }
    }
    SK_COMMON_EPILOGUE(true)
}

template <int BITS, int NTL, bool TRANSPOSED>
int launch_skinny_impl(const CUtensorMap& tq, const CUtensorMap& ts, const CUtensorMap& tz, const CUtensorMap& ta, const CUtensorMap& tl,
                       const SkinnyParams& p, size_t smem_bytes, dim3 grid, cudaStream_t st) {
    static bool configured = false;
    cudaError_t err;
    if (TRANSPOSED) {
        auto kern = skinny_bwd_kernel<BITS, NTL>;
        if (!configured) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024) != cudaSuccess) return QLORA_ERR_CUDA;
            configured = true;
        }
        err = launch_pdl(kern, grid, dim3(SK_THREADS), smem_bytes, st, 1, tq, ts, tz, ta, tl, p);
    } else {
        auto kern = skinny_fwd_kernel<BITS, NTL>;
        if (!configured) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024) != cudaSuccess) return QLORA_ERR_CUDA;
            configured = true;
        }
        err = launch_pdl(kern, grid, dim3(SK_THREADS), smem_bytes, st, 1, tq, ts, tz, ta, tl, p);
    }
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}
