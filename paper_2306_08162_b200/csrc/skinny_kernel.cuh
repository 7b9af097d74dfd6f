// Small-token-count kernels (M <= 64) of the quantized-linear + LoRA layer; included by umma_kernel.cu inside its
// anonymous namespace (they share its TMA / mbarrier helpers and the device status word).
//
// With a handful of tokens the layer is bound by streaming the packed weights from HBM once, so these kernels are built
// around bytes in flight rather than tensor throughput: one elected thread per CTA issues TMA loads of packed-word tiles
// (plus the matching scale / zero rows) into a shared-memory ring deep enough to hold the CTA's whole weight slice, and
// eight consumer warps unpack from shared memory and feed the warp-level tensor-core instruction (mma.sync m16n8k16,
// bf16 in, fp32 accumulate).  A CTA row (blockIdx.y) covers 16 tokens; more tokens re-read the weights through L2.
//
//   forward  (Y = X W^T + s H B^T): a CTA owns 32 output columns n and walks K in stages of 256.  Lane (g, q) of a warp
//     owns, per 128-wide step, the 32 consecutive-k codes k0 + 32q .. + 31 of the four columns 4g .. 4g+3 (one 16-byte
//     shared-memory read per packed row), dequantises them with the library's dequant32 and uses them as B fragments; the
//     contraction index inside a step is permuted the same way for the activation fragments (64 contiguous bytes of X
//     per lane and token row), which leaves the sum unchanged.
//   backward (dX = dY W + s G A): a CTA owns 32 consecutive k (BITS packed rows) and walks N in stages of 256 columns.  The
//     contraction now runs across packed columns, so a fragment register needs two neighbouring n for one k: each lane
//     extracts the two codes (k, k+1) of its own column and the 8 x 8 tile is transposed across the warp with movmatrix
//     -- the register-level form of the paper's "transpose of the packed matrix" (Section 3.1).
// LoRA: for r <= 16 the down-projection (H = X A^T, G = dY B) rides along as one or two extra fragment tiles, so there is
// no separate launch; larger ranks read H / G computed by the skinny pre-kernel.  The eight warps' partial sums are added
// in warp order through shared memory (fixed order, deterministic), the LoRA update is applied in fp32, the result is
// rounded once to bf16.

constexpr int SK_WARPS = 8;                         // consumer warps; warp 8 is the TMA producer
constexpr int SK_THREADS = (SK_WARPS + 1) * 32;
constexpr int SK_STAGE = 256;                       // contraction elements per ring stage
constexpr int SK_COLS = 32;                         // output columns per CTA
constexpr int SK_MAX_STAGES = 16;

struct SkinnyParams {
    int M, N, K, bits, g, r;
    int T;                       // contraction length (K forward, N backward)
    int C;                       // output columns (N forward, K backward)
    int stages_total, S;
    int scale_rows;              // group rows per stage (forward); 1 backward
    uint32_t words_bytes, scale_bytes, scale_stride, stage_bytes;   // scale_bytes: bytes one TMA brings; scale_stride: its 128-aligned slot
    uint32_t off_red, off_p, off_bar;
    float s;
    const __nv_bfloat16* In;     // X (forward) or dY (backward)
    const __nv_bfloat16* Ldown;  // A [r, K] (forward) or B [N, r] (backward): the adapter applied first
    const __nv_bfloat16* Lup;    // B [N, r] (forward) or A [r, K] (backward): the adapter applied second
    float* P;                    // H / G fp32 [M, r]: written by CTA column 0 when fused, read otherwise
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

// Shared by both directions: barrier set-up, the producer loop and the final reduction + LoRA epilogue.
template <bool TRANSPOSED>
__device__ __forceinline__ void sk_producer(const SkinnyParams& p, const CUtensorMap* tq, const CUtensorMap* ts, const CUtensorMap* tz,
                                            uint32_t smem0, uint32_t bar_full, uint32_t bar_empty, int x0, volatile int* abort_flag) {
    for (int st = 0; st < p.stages_total; ++st) {
        const uint32_t slot = (uint32_t)(st % p.S), lap = (uint32_t)(st / p.S);
        if (!mbar_wait(bar_empty + 8 * slot, (lap & 1u) ^ 1u, abort_flag)) return;
        const uint32_t dst = smem0 + slot * p.stage_bytes;
        const uint32_t bar = bar_full + 8 * slot;
        mbar_expect_tx(bar, p.words_bytes + 2 * p.scale_bytes);
        if (!TRANSPOSED) {   // x0 = first output column n; rows walk K
            tma_load_2d(dst, tq, bar, x0, st * (SK_STAGE / 32) * p.bits);
            tma_load_2d(dst + p.words_bytes, ts, bar, x0, (st * SK_STAGE) / p.g);
            tma_load_2d(dst + p.words_bytes + p.scale_stride, tz, bar, x0, (st * SK_STAGE) / p.g);
        } else {             // x0 = first output feature k (multiple of 32); columns walk N
            tma_load_2d(dst, tq, bar, st * SK_STAGE, (x0 / 32) * p.bits);
            tma_load_2d(dst + p.words_bytes, ts, bar, st * SK_STAGE, x0 / p.g);
            tma_load_2d(dst + p.words_bytes + p.scale_stride, tz, bar, st * SK_STAGE, x0 / p.g);
        }
    }
}

// red: [SK_WARPS][16][32 + 8 NTL] fp32 partial tiles (columns 32.. hold the fused H / G partials).
template <bool TRANSPOSED, int NTL>
__device__ __forceinline__ void sk_epilogue(const SkinnyParams& p, const float* red, float* ps, int c0, int mrow0) {
    constexpr int RW = 32 + 8 * NTL;
    const int tid = threadIdx.x;
    if (NTL > 0) {
        for (int e = tid; e < 16 * 8 * NTL; e += SK_THREADS) {
            const int m = e / (8 * NTL), j = e % (8 * NTL);
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < SK_WARPS; ++w) v += red[(w * 16 + m) * RW + 32 + j];
            ps[m * 16 + j] = v;
            if (blockIdx.x == 0 && mrow0 + m < p.M && j < p.r) p.P[(size_t)(mrow0 + m) * p.r + j] = v;
        }
        __syncthreads();
    }
    for (int e = tid; e < 16 * 32; e += SK_THREADS) {
        const int m = e >> 5, c = e & 31;
        const int row = mrow0 + m, col = c0 + c;
        if (row >= p.M || col >= p.C) continue;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < SK_WARPS; ++w) v += red[(w * 16 + m) * RW + c];
        if (p.r > 0) {
            float lo = 0.f;
            for (int j = 0; j < p.r; ++j) {
                const float pj = NTL > 0 ? ps[m * 16 + j] : __ldg(p.P + (size_t)row * p.r + j);
                const float l = TRANSPOSED ? __bfloat162float(p.Lup[(size_t)j * p.K + col])     // A[j, k]
                                           : __bfloat162float(p.Lup[(size_t)col * p.r + j]);    // B[n, j]
                lo = fmaf(pj, l, lo);
            }
            v += p.s * lo;
        }
        p.Out[(size_t)row * p.C + col] = __float2bfloat16_rn(v);
    }
}

#define SK_COMMON_PROLOGUE()                                                                                         \
    extern __shared__ uint8_t smem_raw[];                                                                           \
    __shared__ int abort_flag_s;                                                                                    \
    volatile int* abort_flag = &abort_flag_s;                                                                       \
    const uint32_t smem0 = (smem_u32(smem_raw) + 127u) & ~127u;                                                     \
    uint8_t* smem_gen = smem_raw + (smem0 - smem_u32(smem_raw));                                                    \
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;                                                     \
    const int g = lane >> 2, q = lane & 3;                                                                          \
    const uint32_t bar_full = smem0 + p.off_bar, bar_empty = bar_full + 8 * SK_MAX_STAGES;                          \
    float* red = reinterpret_cast<float*>(smem_gen + p.off_red);                                                    \
    float* ps = reinterpret_cast<float*>(smem_gen + p.off_p);                                                       \
    const int mrow0 = blockIdx.y * 16;

template <int BITS, int NTL>
__global__ void __launch_bounds__(SK_THREADS)
skinny_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_s,
                  const __grid_constant__ CUtensorMap tm_z, const SkinnyParams p) {
    SK_COMMON_PROLOGUE();
    const int n0 = blockIdx.x * SK_COLS;
    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int i = 0; i < p.S; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 2); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == SK_WARPS) {
        if (lane == 0) sk_producer<false>(p, &tm_q, &tm_s, &tm_z, smem0, bar_full, bar_empty, n0, abort_flag);
    } else {
        float acc[4][4], accL[NTL > 0 ? NTL : 1][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
        for (int i = 0; i < (NTL > 0 ? NTL : 1); ++i) accL[i][0] = accL[i][1] = accL[i][2] = accL[i][3] = 0.f;
        const int K = p.K;
        const bool v0 = mrow0 + g < p.M, v1 = mrow0 + g + 8 < p.M;
        const __nv_bfloat16* x0 = p.In + (size_t)(mrow0 + g) * K;
        const __nv_bfloat16* x1 = x0 + (size_t)8 * K;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        const int steps = (K + 127) / 128;
        for (int ws = warp; ws < steps; ws += SK_WARPS) {
            const int stage = ws >> 1;
            const uint32_t slot = (uint32_t)(stage % p.S), lap = (uint32_t)(stage / p.S);
            const int kq = ws * 128 + 32 * q;                     // this lane's 32 consecutive k
            const bool kin = kq < K;                              // K is a multiple of 32
            uint4 xa[4], xb[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                xa[jj] = (v0 && kin) ? __ldg(reinterpret_cast<const uint4*>(x0 + kq + 8 * jj)) : zero4;
                xb[jj] = (v1 && kin) ? __ldg(reinterpret_cast<const uint4*>(x1 + kq + 8 * jj)) : zero4;
            }
            if (!warp_wait(bar_full + 8 * slot, lap & 1u, abort_flag, lane)) break;
            const uint8_t* stg = smem_gen + slot * p.stage_bytes;
            const int blk = (ws & 1) * 4 + q;                     // 32-code block inside the stage
            uint4 w4[BITS];
#pragma unroll
            for (int u = 0; u < BITS; ++u)
                w4[u] = *reinterpret_cast<const uint4*>(stg + ((size_t)(blk * BITS + u) * SK_COLS + 4 * g) * 4);
            const int srow = p.scale_rows > 1 ? (blk * 32) / p.g : 0;
            const uint2 sc2 = *reinterpret_cast<const uint2*>(stg + p.words_bytes + ((size_t)srow * SK_COLS + 4 * g) * 2);
            const uint2 zp2 = *reinterpret_cast<const uint2*>(stg + p.words_bytes + p.scale_stride + ((size_t)srow * SK_COLS + 4 * g) * 2);
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
#pragma unroll
            for (int lt = 0; lt < NTL; ++lt) {
                const int j = lt * 8 + g;
                const __nv_bfloat16* arow = p.Ldown + (size_t)j * K + kq;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const uint4 la = (kin && j < p.r) ? __ldg(reinterpret_cast<const uint4*>(arow + 8 * jj)) : zero4;
                    sk_mma(accL[lt], xa[jj].x, xb[jj].x, xa[jj].y, xb[jj].y, la.x, la.y);
                    sk_mma(accL[lt], xa[jj].z, xb[jj].z, xa[jj].w, xb[jj].w, la.z, la.w);
                }
            }
        }
        // accumulator element (i, c): token g (+8 for c >= 2), column 4 (2q + (c & 1)) + i of the CTA's 32
        constexpr int RW = 32 + 8 * NTL;
        float* mine = red + (size_t)warp * 16 * RW;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * RW + 4 * (2 * q + (c & 1)) + i] = acc[i][c];
#pragma unroll
        for (int lt = 0; lt < NTL; ++lt)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * RW + 32 + lt * 8 + 2 * q + (c & 1)] = accL[lt][c];
    }
    __syncthreads();
    if (!*abort_flag) sk_epilogue<false, NTL>(p, red, ps, n0, mrow0);
}

template <int BITS, int NTL>
__global__ void __launch_bounds__(SK_THREADS)
skinny_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_s,
                  const __grid_constant__ CUtensorMap tm_z, const SkinnyParams p) {
    SK_COMMON_PROLOGUE();
    const int kb = blockIdx.x * SK_COLS;                          // this CTA's 32 output features k
    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int i = 0; i < p.S; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, SK_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == SK_WARPS) {
        if (lane == 0) sk_producer<true>(p, &tm_q, &tm_s, &tm_z, smem0, bar_full, bar_empty, kb, abort_flag);
    } else {
        float acc[4][4], accG[NTL > 0 ? NTL : 1][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
        for (int i = 0; i < (NTL > 0 ? NTL : 1); ++i) accG[i][0] = accG[i][1] = accG[i][2] = accG[i][3] = 0.f;
        const int N = p.N;
        const bool v0 = mrow0 + g < p.M, v1 = mrow0 + g + 8 < p.M;
        const __nv_bfloat16* y0 = p.In + (size_t)(mrow0 + g) * N;
        const __nv_bfloat16* y1 = y0 + (size_t)8 * N;
        for (int stage = 0; stage < p.stages_total; ++stage) {
            const uint32_t slot = (uint32_t)(stage % p.S), lap = (uint32_t)(stage / p.S);
            const int nl = 32 * warp;                             // this warp's 32 columns inside the stage
            const int nbase = stage * SK_STAGE + nl;
            uint32_t a[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {                         // dY fragments of the two 16-wide contraction steps
                const int n = nbase + 16 * h + 2 * q;             // N is a multiple of 8: pairs are all-in or all-out
                a[h][0] = (v0 && n < N) ? __ldg(reinterpret_cast<const uint32_t*>(y0 + n)) : 0u;
                a[h][1] = (v1 && n < N) ? __ldg(reinterpret_cast<const uint32_t*>(y1 + n)) : 0u;
                a[h][2] = (v0 && n + 8 < N) ? __ldg(reinterpret_cast<const uint32_t*>(y0 + n + 8)) : 0u;
                a[h][3] = (v1 && n + 8 < N) ? __ldg(reinterpret_cast<const uint32_t*>(y1 + n + 8)) : 0u;
            }
            if (!warp_wait(bar_full + 8 * slot, lap & 1u, abort_flag, lane)) break;
            const uint8_t* stg = smem_gen + slot * p.stage_bytes;
            const uint32_t* pw = reinterpret_cast<const uint32_t*>(stg);
            const __half* psc = reinterpret_cast<const __half*>(stg + p.words_bytes);
            const __half* pzp = reinterpret_cast<const __half*>(stg + p.words_bytes + p.scale_stride);
            uint32_t w[4][BITS];                                  // columns nl + g, + 8, + 16, + 24
            __half sc[4], zp[4];
#pragma unroll
            for (int cset = 0; cset < 4; ++cset) {
                const int col = nl + 8 * cset + g;
#pragma unroll
                for (int u = 0; u < BITS; ++u) w[cset][u] = pw[u * SK_STAGE + col];
                sc[cset] = psc[col];
                zp[cset] = pzp[col];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const GroupParams gpa = group_params(sc[2 * h], zp[2 * h]);
                const GroupParams gpb = group_params(sc[2 * h + 1], zp[2 * h + 1]);
#pragma unroll
                for (int t = 0; t < 4; ++t) {                     // output features kb + 8t .. 8t + 7
                    const uint32_t b0 = sk_movmatrix(dequant_pair<BITS>(w[2 * h], t, q, gpa));
                    const uint32_t b1 = sk_movmatrix(dequant_pair<BITS>(w[2 * h + 1], t, q, gpb));
                    sk_mma(acc[t], a[h][0], a[h][1], a[h][2], a[h][3], b0, b1);
                }
#pragma unroll
                for (int lt = 0; lt < NTL; ++lt) {                // G = dY B: B [N, r] rows loaded pairwise along r, transposed
                    const int na = nbase + 16 * h + g, nb2 = na + 8;
                    uint32_t va = 0, vb = 0;
                    if (lt * 8 < p.r) {
                        if (na < N) va = __ldg(reinterpret_cast<const uint32_t*>(p.Ldown + (size_t)na * p.r + lt * 8 + 2 * q));
                        if (nb2 < N) vb = __ldg(reinterpret_cast<const uint32_t*>(p.Ldown + (size_t)nb2 * p.r + lt * 8 + 2 * q));
                    }
                    sk_mma(accG[lt], a[h][0], a[h][1], a[h][2], a[h][3], sk_movmatrix(va), sk_movmatrix(vb));
                }
            }
        }
        // accumulator element (t, c): token g (+8 for c >= 2), output feature 8t + 2q + (c & 1) of the CTA's 32
        constexpr int RW = 32 + 8 * NTL;
        float* mine = red + (size_t)warp * 16 * RW;
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * RW + 8 * t + 2 * q + (c & 1)] = acc[t][c];
#pragma unroll
        for (int lt = 0; lt < NTL; ++lt)
#pragma unroll
            for (int c = 0; c < 4; ++c) mine[(g + ((c & 2) ? 8 : 0)) * RW + 32 + lt * 8 + 2 * q + (c & 1)] = accG[lt][c];
    }
    __syncthreads();
    if (!*abort_flag) sk_epilogue<true, NTL>(p, red, ps, kb, mrow0);
}

template <int BITS, int NTL, bool TRANSPOSED>
int launch_skinny_impl(const CUtensorMap& tq, const CUtensorMap& ts, const CUtensorMap& tz, const SkinnyParams& p, size_t smem_bytes,
                       dim3 grid, cudaStream_t st) {
    static bool configured = false;
    if (TRANSPOSED) {
        auto kern = skinny_bwd_kernel<BITS, NTL>;
        if (!configured) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return QLORA_ERR_CUDA;
            configured = true;
        }
        kern<<<grid, SK_THREADS, smem_bytes, st>>>(tq, ts, tz, p);
    } else {
        auto kern = skinny_fwd_kernel<BITS, NTL>;
        if (!configured) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return QLORA_ERR_CUDA;
            configured = true;
        }
        kern<<<grid, SK_THREADS, smem_bytes, st>>>(tq, ts, tz, p);
    }
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}
