// Few-token kernels (M <= 16) of the quantized-linear + LoRA layer, both directions.
//
// With a handful of tokens the layer is bound by reading the packed weights once, so these kernels are built around
// bytes in flight and around what a thread has to issue per weight:
//   - every warp streams its own slice of the packed matrix with 16-byte cp.async copies from all lanes into a private
//     shared-memory ring (no barrier between warps in the main loop); the copies of the first ring-full are issued before
//     the kernel waits for its predecessor in the stream (griddepcontrol.wait), so the frozen weights of a call are in
//     flight while the preceding call is still computing.  Only Q, scales and zeros are touched before that wait: the
//     activations, the adapters (which an optimizer rewrites every step), H / G and the outputs come after it;
//   - the codes go to the warp-level tensor-core instruction (mma.sync m16n8k16, weights as the 16-row operand, tokens as
//     the 8 columns) as RAW integers: a code is ORed into the mantissa of the bf16 constant 128 (one shift + one logic
//     operation per pair of codes), so the operand is 128 + q.  The group scale and the zero-point are applied outside the
//     per-weight path:
//       forward   Y[m,n] = sum_groups s[G,n] * ( sum_{k in G} X[m,k] (128 + q[k,n])  -  (128 + z[G,n]) * sum_{k in G} X[m,k] )
//                 (one accumulator per group; the scaling is a few FMAs per group, the activation sums are made once
//                 per CTA when the activation slice is staged);
//       backward  dX[m,k] = sum_n dYs[m,n] (128 + q[k,n])  -  sum_n dYs[m,n] (128 + z[G(k),n]),   dYs = bf16(dY[m,n] * s[G(k),n])
//                 (the scale varies along the contraction, so it is folded into a per-group copy of the activation slice,
//                 rounded once to bf16 -- the same relative rounding the dequantised weight would get; the second sum is
//                 one extra MMA row per 16 columns).
//     8-bit codes take an fp32 detour (byte -> 2^23 + q -> q -> bf16, exact), offset 0 instead of 128;
//   - backward: the contraction runs across packed columns, so a fragment register needs two columns for one feature.
//     Each lane builds pairs of features of its own column and the 8 x 8 tile is transposed across the warp with
//     movmatrix: the register form of the transposition of the packed matrix (Section 3.1, "Implementation Details");
//   - the contraction is split over a cluster of up to 8 CTAs; the partial tiles are added in rank order through
//     distributed shared memory (CTA i owns a slice of the columns), so no workspace and no counters are needed and the
//     result is the same on every run;
//   - the LoRA down-projection (H = X A^T, G = dY B) over the CTA's part of the contraction comes from a few MMAs fed
//     straight from global memory (ranks up to 16), reduced with the partial tiles; the update s P L is added in the
//     epilogue in fp32 before the one rounding to bf16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "common.cuh"
#include "launch.h"

namespace qlora {
namespace {

constexpr int ST_MAX_DEVICES = 64;

template <int BITS>
struct Fmt {
    static constexpr float OFF = BITS == 8 ? 0.f : 128.f;   // what the integer operand carries on top of the code
    // forward: a ring stage = KB contraction elements x 32 columns of one warp (+ the scale / zero chunk of its group)
    static constexpr int KB = BITS == 2 ? 64 : 32;
    static constexpr int ROWS = KB * BITS / 32;              // packed rows per stage: 4, 3, 4, 8
    static constexpr int SLOT = ROWS * 128 + 128;
    static constexpr int NS = BITS == 8 ? 7 : (BITS == 3 ? 16 : 12);
    static constexpr int STEPS = KB / 16;                    // k16 MMA steps per stage
    static constexpr int NPAIR = 2 * STEPS;                  // bf16 pairs per column and lane
    static constexpr int NLD = (BITS == 3 || BITS == 8) ? 2 : 1;
    static constexpr int XPAD = BITS == 2 ? 16 : (BITS == 8 ? 32 : 64);   // pitch of an activation row = 2 xc + XPAD bytes
    // backward: a warp owns FW output features (BROWS packed rows); a ring stage = SU units of 32 columns
    static constexpr int FW = BITS == 2 ? 16 : 32;
    static constexpr int BROWS = FW * BITS / 32;             // 1, 3, 4, 8
    static constexpr int SU = BITS == 2 ? 4 : 1;
    static constexpr int BSLOT = BROWS * 128 * SU;
    static constexpr int BNS = BITS == 8 ? 8 : 16;
    static constexpr int BPAIR = BITS == 2 ? 2 : 4;          // pairs per column and lane
};

struct StreamParams {
    int M, K, N, g, r;
    int C;                       // output columns (N forward, K backward)
    int ks;                      // CTAs per cluster = ways the contraction is split
    int xc;                      // contraction elements of the activation slice staged per pass
    int copies;                  // backward: groups a CTA's features span (1 or 2)
    int fused;                   // H / G is computed here (ranks up to 16) and written to P; else P is an input
    int lup_staged;              // the epilogue's slice of the second adapter fits its shared-memory area
    float s;
    const __nv_bfloat16* In;
    const uint32_t* Q;
    const __half* scales;
    const __half* zeros;
    const __nv_bfloat16* Ldown;  // A [r, K] (forward) or B [N, r] (backward): the adapter applied first
    const __nv_bfloat16* Lup;    // B [N, r] (forward) or A [r, K] (backward): the adapter applied second
    float* P;                    // H / G fp32 [M, r]
    __nv_bfloat16* Out;
};

constexpr int ST_LUP_BYTES = 4096;

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp16(uint32_t dst, const void* src, int bytes) {   // bytes = 16, or 0 to zero-fill
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint32_t st_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t st_map(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float st_ld_cluster(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t st_movm(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t st_comp(const uint4& v, int i) { return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w)); }
__device__ __forceinline__ uint32_t ldg32(const void* p) { return *reinterpret_cast<const uint32_t*>(p); }

// A ring stage holds packed rows of 32 columns (128 bytes); row `row`, 16-byte chunk `ch` sits at a swizzled place so that
// the lanes (g, q) of a quarter-warp, which read chunk g of four different rows, hit different banks.
__device__ __forceinline__ int st_swz(int row, int ch) { return row * 128 + (((ch ^ (2 * row)) & 7) << 4); }

// The packed words a lane needs for its four columns 4g .. 4g+3: lane q takes the q-th quarter of the stage's contraction
// range (row q; 3-bit: the 24 stream bits [24 q, 24 q + 24) of the 96-bit block, which may lie in two rows; 8-bit: rows
// q and q + 4).
template <int BITS>
__device__ __forceinline__ void st_load_words(const uint8_t* slot, int g, int q, uint4 (&w)[Fmt<BITS>::NLD]) {
    if constexpr (BITS == 3) {
        w[0] = *reinterpret_cast<const uint4*>(slot + st_swz((24 * q) >> 5, g));
        w[1] = *reinterpret_cast<const uint4*>(slot + st_swz((24 * q + 23) >> 5, g));
    } else if constexpr (BITS == 8) {
        w[0] = *reinterpret_cast<const uint4*>(slot + st_swz(q, g));
        w[1] = *reinterpret_cast<const uint4*>(slot + st_swz(q + 4, g));
    } else {
        w[0] = *reinterpret_cast<const uint4*>(slot + st_swz(q, g));
    }
}

__device__ __forceinline__ uint32_t st_u8_pair(uint32_t w, int j) {   // bytes 2j, 2j+1 -> (bf16, bf16), exact
    const float f0 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7540 + 2 * j)) - 8388608.f;
    const float f1 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7541 + 2 * j)) - 8388608.f;
    const __nv_bfloat162 pr = __floats2bfloat162_rn(f0, f1);
    return *reinterpret_cast<const uint32_t*>(&pr);
}

// One column's codes of this lane -> bf16 pairs holding OFF + q.  With c_0 .. c_{n-1} the lane's codes in contraction order:
//   2-bit (16 codes): p[t] = (c_t, c_{t+8}), t < 8        3- and 4-bit (8 codes): p[t] = (c_t, c_{t+4}), t < 4
//   8-bit (row q: c_0..3, row q + 4: c_4..7): p = (c_0,c_1), (c_2,c_3), (c_4,c_5), (c_6,c_7)
template <int BITS>
__device__ __forceinline__ void st_unpack(uint32_t w0, uint32_t w1, int q, uint32_t (&p)[Fmt<BITS>::NPAIR]) {
    if constexpr (BITS == 4) {
#pragma unroll
        for (int t = 0; t < 4; ++t) p[t] = ((w0 >> (4 * t)) & 0x000F000Fu) | 0x43004300u;
    } else if constexpr (BITS == 2) {
#pragma unroll
        for (int t = 0; t < 8; ++t) p[t] = ((w0 >> (2 * t)) & 0x00030003u) | 0x43004300u;
    } else if constexpr (BITS == 3) {
        const uint32_t v = __funnelshift_r(w0, w1, (24 * q) & 31);        // codes at bits 3 j, j < 8
        const uint32_t m = (v & 0x0000FFFFu) | ((v << 4) & 0xFFFF0000u);  // codes 0..3 at bits 3 j, codes 4..7 at 16 + 3 j
#pragma unroll
        for (int t = 0; t < 4; ++t) p[t] = ((m >> (3 * t)) & 0x00070007u) | 0x43004300u;
    } else {
        p[0] = st_u8_pair(w0, 0); p[1] = st_u8_pair(w0, 1);
        p[2] = st_u8_pair(w1, 0); p[3] = st_u8_pair(w1, 1);
    }
}

// 16 bytes of activations (8 consecutive contraction elements) -> the order the lanes' pairs ask for: (x0,x4) (x1,x5)
// (x2,x6) (x3,x7); the 8-bit forward path pairs neighbours and keeps the natural order.
__device__ __forceinline__ uint4 st_permute8(const uint4& v) {
    return make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632), __byte_perm(v.y, v.w, 0x5410), __byte_perm(v.y, v.w, 0x7632));
}
__device__ __forceinline__ float st_sum8(const uint4& v) {
    return ((bf16_lo(v.x) + bf16_hi(v.x)) + (bf16_lo(v.y) + bf16_hi(v.y))) + ((bf16_lo(v.z) + bf16_hi(v.z)) + (bf16_lo(v.w) + bf16_hi(v.w)));
}

// Epilogue shared by both directions.  part: [TOKS][tile_c + 4] fp32 partial tile of this CTA; hs: [16][16] partial H / G.
// CTA `rank` adds the cluster's partial tiles in rank order for its slice of tile_c / ks columns, adds s P L and stores bf16.
template <bool TRANSPOSED, int TOKS>
__device__ __forceinline__ void st_epilogue(const StreamParams& p, float* part, float* hs, float* hfull, const __nv_bfloat16* lup,
                                            int tile_c, int rank) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int pw = tile_c + 4;
    const int sl = tile_c / p.ks;
    st_cluster_sync();                                    // every CTA's partial tile (and partial H / G) is written
    if (p.r > 0 && p.fused) {
        const uint32_t ha = s_u32(hs);
        for (int e = tid; e < 256; e += nthr) {
            float h = 0.f;
            for (int rk = 0; rk < p.ks; ++rk) h += st_ld_cluster(st_map(ha + 4u * (uint32_t)e, (uint32_t)rk));
            hfull[e] = h;
            const int j = e >> 4, tok = e & 15;
            if (blockIdx.y == 0 && rank == 0 && tok < p.M && j < p.r) p.P[(size_t)tok * p.r + j] = h;
        }
        __syncthreads();
    }
    const uint32_t pa = s_u32(part);
    for (int e = tid; e < TOKS * sl; e += nthr) {
        const int tok = e / sl, c = e % sl;
        const int cl = rank * sl + c, col = blockIdx.y * tile_c + cl;
        float v = 0.f;
        for (int rk = 0; rk < p.ks; ++rk) v += st_ld_cluster(st_map(pa + 4u * (uint32_t)(tok * pw + cl), (uint32_t)rk));
        if (tok >= p.M || col >= p.C) continue;
        if (p.r > 0) {
            float lo = 0.f;
            for (int j = 0; j < p.r; ++j) {
                float l;
                if (p.lup_staged) l = __bfloat162float(TRANSPOSED ? lup[j * sl + c] : lup[c * p.r + j]);
                else l = __bfloat162float(TRANSPOSED ? p.Lup[(size_t)j * p.K + col] : p.Lup[(size_t)col * p.r + j]);
                lo = fmaf(hfull[j * 16 + tok], l, lo);
            }
            v += p.s * lo;
        }
        p.Out[(size_t)tok * p.C + col] = __float2bfloat16_rn(v);
    }
    st_cluster_sync();                                    // nobody leaves while a peer may still read its shared memory
}

// After griddepcontrol.wait: this CTA's slice of the second adapter (the columns it will finish) and, when H / G is an
// input, the whole of it.
template <bool TRANSPOSED>
__device__ __forceinline__ void st_stage_lup(const StreamParams& p, __nv_bfloat16* lup, float* hfull, int tile_c, int rank) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    if (p.r == 0) return;
    const int sl = tile_c / p.ks;
    if (p.lup_staged) {
        for (int e = tid; e < sl * p.r; e += nthr) {
            int c, j;
            if (TRANSPOSED) { j = e / sl; c = e % sl; } else { c = e / p.r; j = e % p.r; }
            const int col = blockIdx.y * tile_c + rank * sl + c;
            __nv_bfloat16 v = __float2bfloat16_rn(0.f);
            if (col < p.C) v = TRANSPOSED ? p.Lup[(size_t)j * p.K + col] : p.Lup[(size_t)col * p.r + j];
            lup[e] = v;
        }
    }
    if (!p.fused) {
        for (int e = tid; e < 16 * p.r; e += nthr) {      // hfull[j][tok]; rows beyond M are zero
            const int j = e >> 4, tok = e & 15;
            hfull[e] = tok < p.M ? p.P[(size_t)tok * p.r + j] : 0.f;
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// Forward: Y = X W^T + s H B^T.  CTA (rank, tile): columns [32 W tile, +32 W) (warp w: 32 of them), contraction blocks
// [kb0, kb1) of KB elements, all of them taken by every warp for its own columns.
// ------------------------------------------------------------------------------------------------------------
template <int BITS, int NT>
__global__ void __launch_bounds__(256, 2) stream_fwd_kernel(const StreamParams p) {
    using F = Fmt<BITS>;
    constexpr int TOKS = 8 * NT;
    pdl_launch_dependents();
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int W = blockDim.x >> 5, tile_c = 32 * W;
    const int rank = (int)st_cluster_rank();
    const int col0 = blockIdx.y * tile_c + 32 * warp;
    const int nblk = (p.K + F::KB - 1) / F::KB;
    const int kb0 = nblk * rank / p.ks, kb1 = nblk * (rank + 1) / p.ks;
    const int nit = kb1 - kb0;
    const int total_rows = p.K * BITS / 32;
    const int xp = p.xc * 2 + F::XPAD;
    const int xcb = p.xc / F::KB;                          // blocks per staged slice
    uint8_t* ring = smem + warp * (F::NS * F::SLOT);
    uint8_t* xs = smem + W * (F::NS * F::SLOT);            // [TOKS][xp] permuted activation slice
    float* sxc = reinterpret_cast<float*>(xs + TOKS * xp); // [TOKS][xc / 8] sums of 8 activations
    float* sxs = sxc + TOKS * (p.xc / 8);                  // [xcb + 1][TOKS] sums per group segment of the slice
    float* hs = sxs + (xcb + 1) * TOKS;                    // [16][16] this CTA's part of H
    float* hfull = hs + 256;                               // [r <= 64][16] the whole of H
    __nv_bfloat16* lup = reinterpret_cast<__nv_bfloat16*>(hfull + 1024);
    float* part = reinterpret_cast<float*>(smem);          // reuses the rings after the main loop
    float* hp = reinterpret_cast<float*>(xs);              // [W][16][16], before the first slice is staged

    auto issue = [&](int it) {
        if (it < nit) {
            const int blk = kb0 + it;
            const uint32_t dst = s_u32(ring + (it % F::NS) * F::SLOT);
#pragma unroll
            for (int h = 0; h < (F::ROWS + 3) / 4; ++h) {
                const int row = 4 * h + (lane >> 3), ch = lane & 7;
                if (row < F::ROWS) {
                    const int grow = blk * F::ROWS + row, col = col0 + 4 * ch;
                    const bool ok = grow < total_rows && col < p.N;
                    cp16(dst + st_swz(row, ch), ok ? p.Q + (size_t)grow * p.N + col : p.Q, ok ? 16 : 0);
                }
            }
            const int k0 = blk * F::KB;
            if ((k0 % p.g == 0 || it == 0) && lane < 8) {  // first block of a group in this CTA's range: its scales and zeros
                const __half* base = lane < 4 ? p.scales : p.zeros;
                const int col = col0 + 8 * (lane & 3);
                const bool ok = col < p.N;
                cp16(dst + F::ROWS * 128 + lane * 16, ok ? base + (size_t)(k0 / p.g) * p.N + col : base, ok ? 16 : 0);
            }
        }
        cp_commit();
    };
    for (int it = 0; it < F::NS; ++it) issue(it);          // frozen weights only: in flight while the predecessor finishes

    pdl_wait();

    // ---- LoRA: this CTA's part of H = X A^T (k16 steps dealt to the warps, operands straight from global memory) ----
    st_stage_lup<false>(p, lup, hfull, tile_c, rank);
    if (p.r > 0 && p.fused) {
        float ah[NT][4];
#pragma unroll
        for (int tt = 0; tt < NT; ++tt) ah[tt][0] = ah[tt][1] = ah[tt][2] = ah[tt][3] = 0.f;
        const int ke = min(kb1 * F::KB, p.K);
        for (int k0 = kb0 * F::KB + 16 * warp; k0 < ke; k0 += 16 * W) {
            const __nv_bfloat16* a_lo = p.Ldown + (size_t)g * p.K + k0 + 2 * q;
            const __nv_bfloat16* a_hi = p.Ldown + (size_t)(g + 8) * p.K + k0 + 2 * q;
            const uint32_t a0 = g < p.r ? ldg32(a_lo) : 0u, a2 = g < p.r ? ldg32(a_lo + 8) : 0u;
            const uint32_t a1 = g + 8 < p.r ? ldg32(a_hi) : 0u, a3 = g + 8 < p.r ? ldg32(a_hi + 8) : 0u;
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const int tok = g + 8 * tt;
                const __nv_bfloat16* x = p.In + (size_t)tok * p.K + k0 + 2 * q;
                const uint32_t b0 = tok < p.M ? ldg32(x) : 0u, b1 = tok < p.M ? ldg32(x + 8) : 0u;
                st_mma(ah[tt], a0, a1, a2, a3, b0, b1);
            }
        }
        float* mine = hp + warp * 256;
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                mine[(g + ((e & 2) ? 8 : 0)) * 16 + 8 * tt + 2 * q + (e & 1)] = tt < NT ? ah[tt < NT ? tt : 0][e] : 0.f;
        __syncthreads();
        for (int e = threadIdx.x; e < 256; e += blockDim.x) {
            float h = 0.f;
            for (int w = 0; w < W; ++w) h += hp[w * 256 + e];
            hs[e] = h;
        }
        __syncthreads();
    }

    // ---- main loop ----
    float acc[2][NT][4], grp[2][NT][4];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[u][tt][e] = grp[u][tt][e] = 0.f;
    float sc[4] = {0.f, 0.f, 0.f, 0.f}, cz[4] = {0.f, 0.f, 0.f, 0.f};   // this lane's four columns: scale, -scale (OFF + zero)
    int it = 0;
    for (int cb = kb0; cb < kb1; cb += xcb) {
        const int ce = min(cb + xcb, kb1);
        const int k_lo = cb * F::KB, k_hi = min(ce * F::KB, p.K);
        // stage the activation slice [k_lo, k_hi): permuted for the fragment loads, plus the sums the zero-points need
        {
            constexpr int KP = BITS == 2 ? 16 : 8;
            const int per_tok = (ce - cb) * F::KB / KP;
            for (int e = threadIdx.x; e < TOKS * per_tok; e += blockDim.x) {
                const int tok = e / per_tok, ci = e % per_tok;
                const int k = k_lo + ci * KP;
                uint4 v0 = make_uint4(0, 0, 0, 0), v1 = make_uint4(0, 0, 0, 0);
                if (tok < p.M && k < p.K) {
                    v0 = *reinterpret_cast<const uint4*>(p.In + (size_t)tok * p.K + k);
                    if (KP == 16 && k + 8 < p.K) v1 = *reinterpret_cast<const uint4*>(p.In + (size_t)tok * p.K + k + 8);
                }
                uint8_t* dst = xs + tok * xp + ci * (2 * KP);
                if constexpr (BITS == 2) {                 // (x0,x8) (x1,x9) ... (x7,x15)
                    *reinterpret_cast<uint4*>(dst) = make_uint4(__byte_perm(v0.x, v1.x, 0x5410), __byte_perm(v0.x, v1.x, 0x7632),
                                                                __byte_perm(v0.y, v1.y, 0x5410), __byte_perm(v0.y, v1.y, 0x7632));
                    *reinterpret_cast<uint4*>(dst + 16) = make_uint4(__byte_perm(v0.z, v1.z, 0x5410), __byte_perm(v0.z, v1.z, 0x7632),
                                                                     __byte_perm(v0.w, v1.w, 0x5410), __byte_perm(v0.w, v1.w, 0x7632));
                    sxc[tok * (p.xc / 8) + 2 * ci] = st_sum8(v0);
                    sxc[tok * (p.xc / 8) + 2 * ci + 1] = st_sum8(v1);
                } else {
                    *reinterpret_cast<uint4*>(dst) = BITS == 8 ? v0 : st_permute8(v0);
                    sxc[tok * (p.xc / 8) + ci] = st_sum8(v0);
                }
            }
            __syncthreads();
            const int g_first = k_lo / p.g, nseg = (k_hi - 1) / p.g - g_first + 1;
            for (int e = threadIdx.x; e < nseg * TOKS; e += blockDim.x) {
                const int seg = e / TOKS, tok = e % TOKS;
                const int a = max(k_lo, (g_first + seg) * p.g), b = min(k_hi, (g_first + seg + 1) * p.g);
                float sum = 0.f;
                for (int c8 = (a - k_lo) / 8; c8 < (b - k_lo) / 8; ++c8) sum += sxc[tok * (p.xc / 8) + c8];
                sxs[seg * TOKS + tok] = sum;
            }
            __syncthreads();
        }
        for (int blk = cb; blk < ce; ++blk, ++it) {
            cp_wait<F::NS - 1>();
            __syncwarp();
            const uint8_t* slot = ring + (it % F::NS) * F::SLOT;
            const int k0 = blk * F::KB;
            if (k0 % p.g == 0 || it == 0) {                // a new group: this lane's scales and zero-points
                const uint2 s2 = *reinterpret_cast<const uint2*>(slot + F::ROWS * 128 + 8 * g);
                const uint2 z2 = *reinterpret_cast<const uint2*>(slot + F::ROWS * 128 + 64 + 8 * g);
                const float2 sa = __half22float2(*reinterpret_cast<const __half2*>(&s2.x)), sb = __half22float2(*reinterpret_cast<const __half2*>(&s2.y));
                const float2 za = __half22float2(*reinterpret_cast<const __half2*>(&z2.x)), zb = __half22float2(*reinterpret_cast<const __half2*>(&z2.y));
                sc[0] = sa.x; sc[1] = sa.y; sc[2] = sb.x; sc[3] = sb.y;
                cz[0] = -sa.x * (F::OFF + za.x); cz[1] = -sa.y * (F::OFF + za.y); cz[2] = -sb.x * (F::OFF + zb.x); cz[3] = -sb.y * (F::OFF + zb.y);
            }
            uint4 w[F::NLD];
            st_load_words<BITS>(slot, g, q, w);
            // activation fragments: token g (+ 8), this lane's quarter of the block
            uint32_t xf[NT][F::NPAIR];
            const int bl = blk - cb;
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const uint8_t* xr = xs + (g + 8 * tt) * xp;
                if constexpr (BITS == 2) {
                    const uint4 v0 = *reinterpret_cast<const uint4*>(xr + bl * 128 + 32 * q);
                    const uint4 v1 = *reinterpret_cast<const uint4*>(xr + bl * 128 + 32 * q + 16);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v0.z; xf[tt][3] = v0.w;
                    xf[tt][4] = v1.x; xf[tt][5] = v1.y; xf[tt][6] = v1.z; xf[tt][7] = v1.w;
                } else if constexpr (BITS == 8) {
                    const uint2 v0 = *reinterpret_cast<const uint2*>(xr + bl * 64 + 8 * q);
                    const uint2 v1 = *reinterpret_cast<const uint2*>(xr + bl * 64 + 32 + 8 * q);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v1.x; xf[tt][3] = v1.y;
                } else {
                    const uint4 v0 = *reinterpret_cast<const uint4*>(xr + bl * 64 + 16 * q);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v0.z; xf[tt][3] = v0.w;
                }
            }
            // two tiles of 16 columns: rows g / g + 8 of tile u are columns 4g + 2u / 4g + 2u + 1
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                uint32_t pa[F::NPAIR], pb[F::NPAIR];
                st_unpack<BITS>(st_comp(w[0], 2 * u), F::NLD > 1 ? st_comp(w[F::NLD - 1], 2 * u) : 0u, q, pa);
                st_unpack<BITS>(st_comp(w[0], 2 * u + 1), F::NLD > 1 ? st_comp(w[F::NLD - 1], 2 * u + 1) : 0u, q, pb);
#pragma unroll
                for (int s = 0; s < F::STEPS; ++s)
#pragma unroll
                    for (int tt = 0; tt < NT; ++tt)
                        st_mma(grp[u][tt], pa[2 * s], pb[2 * s], pa[2 * s + 1], pb[2 * s + 1], xf[tt][2 * s], xf[tt][2 * s + 1]);
            }
            if ((k0 + F::KB) % p.g == 0 || blk + 1 == ce) {   // end of a group segment: scale, correct, start afresh
                const int seg = k0 / p.g - k_lo / p.g;
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) {
                    const float2 sx = *reinterpret_cast<const float2*>(sxs + seg * TOKS + 8 * tt + 2 * q);
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        acc[u][tt][0] += sc[2 * u] * grp[u][tt][0] + cz[2 * u] * sx.x;
                        acc[u][tt][1] += sc[2 * u] * grp[u][tt][1] + cz[2 * u] * sx.y;
                        acc[u][tt][2] += sc[2 * u + 1] * grp[u][tt][2] + cz[2 * u + 1] * sx.x;
                        acc[u][tt][3] += sc[2 * u + 1] * grp[u][tt][3] + cz[2 * u + 1] * sx.y;
                        grp[u][tt][0] = grp[u][tt][1] = grp[u][tt][2] = grp[u][tt][3] = 0.f;
                    }
                }
            }
            __syncwarp();
            issue(it + F::NS);
        }
        __syncthreads();                                   // the slice (and, at the end, the rings) may be overwritten
    }
    cp_wait<0>();
    // accumulator element (u, tt, e): column 4g + 2u + (e >> 1) of this warp's 32, token 2q + (e & 1) + 8 tt
    {
        const int pw = tile_c + 4;
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int tt = 0; tt < NT; ++tt)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    part[(2 * q + (e & 1) + 8 * tt) * pw + 32 * warp + 4 * g + 2 * u + (e >> 1)] = acc[u][tt][e];
    }
    st_epilogue<false, TOKS>(p, part, hs, hfull, lup, tile_c, rank);
}

// ------------------------------------------------------------------------------------------------------------
// Backward: dX = dY W + s G A.  CTA (rank, tile): output features [FW W tile, + FW W) (warp w: FW of them, all inside
// one group), contraction stages [st0, st1) of 32 SU packed columns.
// ------------------------------------------------------------------------------------------------------------
template <int BITS, int NT>
__global__ void __launch_bounds__(256, 2) stream_bwd_kernel(const StreamParams p) {
    using F = Fmt<BITS>;
    constexpr int TOKS = 8 * NT;
    constexpr int NTILE = F::BPAIR / 2;                    // 16-feature MMA tiles per warp
    pdl_launch_dependents();
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int W = blockDim.x >> 5, tile_c = F::FW * W;
    const int rank = (int)st_cluster_rank();
    const int tile_f0 = blockIdx.y * tile_c, f0 = tile_f0 + F::FW * warp;
    const bool live = f0 < p.K;                            // a warp beyond the last feature only keeps the barriers company
    const int row0 = f0 * BITS / 32;
    const int sw = 32 * F::SU;                             // packed columns per stage
    const int nst = (p.N + sw - 1) / sw;
    const int st0 = nst * rank / p.ks, st1 = nst * (rank + 1) / p.ks;
    const int nit = st1 - st0;
    const int xp = p.xc * 2 + 64;
    const int xcs = p.xc / sw;                             // stages per staged slice
    const int copy = p.copies > 1 ? (f0 - tile_f0) / p.g : 0;
    uint8_t* ring = smem + warp * (F::BNS * F::BSLOT);
    uint8_t* ys = smem + W * (F::BNS * F::BSLOT);          // [copies][TOKS][xp] scaled, permuted slices of dY
    float* zp = reinterpret_cast<float*>(ys + p.copies * TOKS * xp);   // [W][2][16] zero-point sums, per warp
    float* zc = zp + W * 32;                               // [2][16] their total
    float* hs = zc + 32;
    float* hfull = hs + 256;
    __nv_bfloat16* lup = reinterpret_cast<__nv_bfloat16*>(hfull + 1024);
    float* part = reinterpret_cast<float*>(smem);
    float* hp = reinterpret_cast<float*>(ys);

    auto issue = [&](int it) {
        if (it < nit && live) {
            const int cbase = (st0 + it) * sw;
            const uint32_t dst = s_u32(ring + (it % F::BNS) * F::BSLOT);
            if constexpr (BITS == 2) {
                const int col = cbase + 32 * (lane >> 3) + 4 * (lane & 7);
                const bool ok = col < p.N;
                cp16(dst + lane * 16, ok ? p.Q + (size_t)row0 * p.N + col : p.Q, ok ? 16 : 0);
            } else {
#pragma unroll
                for (int h = 0; h < (F::BROWS + 3) / 4; ++h) {
                    const int row = 4 * h + (lane >> 3), ch = lane & 7;
                    if (row < F::BROWS) {
                        const int col = cbase + 4 * ch;
                        const bool ok = col < p.N;
                        cp16(dst + st_swz(row, ch), ok ? p.Q + (size_t)(row0 + row) * p.N + col : p.Q, ok ? 16 : 0);
                    }
                }
            }
        }
        cp_commit();
    };
    for (int it = 0; it < F::BNS; ++it) issue(it);

    pdl_wait();

    const int n_lo_cta = st0 * sw, n_hi_cta = min(st1 * sw, p.N);
    st_stage_lup<true>(p, lup, hfull, tile_c, rank);
    for (int e = threadIdx.x; e < W * 32; e += blockDim.x) zp[e] = 0.f;
    // ---- LoRA: this CTA's part of G = dY B.  B [N, r] has the ranks contiguous, so a lane loads two ranks of its own
    // contraction column and movmatrix turns them into two columns of one rank ----
    if (p.r > 0 && p.fused) {
        float ag[NT][4];
#pragma unroll
        for (int tt = 0; tt < NT; ++tt) ag[tt][0] = ag[tt][1] = ag[tt][2] = ag[tt][3] = 0.f;
        for (int nb = n_lo_cta + 16 * warp; nb < n_hi_cta; nb += 16 * W) {
            const bool v0 = nb + g < p.N, v1 = nb + 8 + g < p.N;
            const __nv_bfloat16* b_lo = p.Ldown + (size_t)(nb + g) * p.r + 2 * q;
            const __nv_bfloat16* b_hi = p.Ldown + (size_t)(nb + 8 + g) * p.r + 2 * q;
            const uint32_t a0 = st_movm(v0 ? ldg32(b_lo) : 0u), a2 = st_movm(v1 ? ldg32(b_hi) : 0u);
            const uint32_t a1 = st_movm(v0 && p.r > 8 ? ldg32(b_lo + 8) : 0u), a3 = st_movm(v1 && p.r > 8 ? ldg32(b_hi + 8) : 0u);
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const int tok = g + 8 * tt;
                const __nv_bfloat16* y = p.In + (size_t)tok * p.N + nb + 2 * q;
                const uint32_t b0 = (tok < p.M && nb + 2 * q < p.N) ? ldg32(y) : 0u;
                const uint32_t b1 = (tok < p.M && nb + 8 + 2 * q < p.N) ? ldg32(y + 8) : 0u;
                st_mma(ag[tt], a0, a1, a2, a3, b0, b1);
            }
        }
        float* mine = hp + warp * 256;
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                mine[(g + ((e & 2) ? 8 : 0)) * 16 + 8 * tt + 2 * q + (e & 1)] = tt < NT ? ag[tt < NT ? tt : 0][e] : 0.f;
        __syncthreads();
        for (int e = threadIdx.x; e < 256; e += blockDim.x) {
            float h = 0.f;
            for (int w = 0; w < W; ++w) h += hp[w * 256 + e];
            hs[e] = h;
        }
    }
    __syncthreads();

    float acc[NTILE][NT][4];
#pragma unroll
    for (int t = 0; t < NTILE; ++t)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt) acc[t][tt][0] = acc[t][tt][1] = acc[t][tt][2] = acc[t][tt][3] = 0.f;
    const int ngroups = p.K / p.g;
    int it = 0;
    for (int cs = st0; cs < st1; cs += xcs) {
        const int ce = min(cs + xcs, st1);
        const int n_lo = cs * sw, n_hi = min(ce * sw, p.N);
        // stage the slice of dY, once per group the CTA's features span, scaled by that group's scales (one rounding)
        {
            const int per_tok = (ce - cs) * sw / 8;
            for (int e = threadIdx.x; e < TOKS * per_tok; e += blockDim.x) {
                const int tok = e / per_tok, ci = e % per_tok;
                const int n = n_lo + ci * 8;
                const bool ok = tok < p.M && n < p.N;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (ok) v = *reinterpret_cast<const uint4*>(p.In + (size_t)tok * p.N + n);
                for (int c = 0; c < p.copies; ++c) {
                    const int gk = tile_f0 / p.g + c;
                    uint4 o = make_uint4(0, 0, 0, 0);
                    if (ok && gk < ngroups) {
                        const uint4 s8 = *reinterpret_cast<const uint4*>(p.scales + (size_t)gk * p.N + n);
                        const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&s8.x)), s1 = __half22float2(*reinterpret_cast<const __half2*>(&s8.y));
                        const float2 s2 = __half22float2(*reinterpret_cast<const __half2*>(&s8.z)), s3 = __half22float2(*reinterpret_cast<const __half2*>(&s8.w));
                        const __nv_bfloat162 o0 = __floats2bfloat162_rn(bf16_lo(v.x) * s0.x, bf16_hi(v.x) * s0.y);
                        const __nv_bfloat162 o1 = __floats2bfloat162_rn(bf16_lo(v.y) * s1.x, bf16_hi(v.y) * s1.y);
                        const __nv_bfloat162 o2 = __floats2bfloat162_rn(bf16_lo(v.z) * s2.x, bf16_hi(v.z) * s2.y);
                        const __nv_bfloat162 o3 = __floats2bfloat162_rn(bf16_lo(v.w) * s3.x, bf16_hi(v.w) * s3.y);
                        o = make_uint4(*reinterpret_cast<const uint32_t*>(&o0), *reinterpret_cast<const uint32_t*>(&o1),
                                       *reinterpret_cast<const uint32_t*>(&o2), *reinterpret_cast<const uint32_t*>(&o3));
                    }
                    *reinterpret_cast<uint4*>(ys + (c * TOKS + tok) * xp + ci * 16) = st_permute8(o);
                }
            }
            __syncthreads();
            // zero-point term: sum_n dYs[m, n] (OFF + z[G, n]) as one MMA row; 32-column units dealt to the warps
            for (int c = 0; c < p.copies; ++c) {
                const int gk = tile_f0 / p.g + c;
                float za[NT][4];
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) za[tt][0] = za[tt][1] = za[tt][2] = za[tt][3] = 0.f;
                for (int un = warp; un < (n_hi - n_lo + 31) / 32; un += W) {
                    const int n = n_lo + 32 * un + 8 * q;
                    uint32_t zr[4] = {0u, 0u, 0u, 0u};     // (z0,z4) (z1,z5) (z2,z6) (z3,z7) as bf16 of OFF + z
                    if (g == 0 && n < p.N && gk < ngroups) {
                        const uint4 z8 = *reinterpret_cast<const uint4*>(p.zeros + (size_t)gk * p.N + n);
                        const float2 z0 = __half22float2(*reinterpret_cast<const __half2*>(&z8.x)), z1 = __half22float2(*reinterpret_cast<const __half2*>(&z8.y));
                        const float2 z2 = __half22float2(*reinterpret_cast<const __half2*>(&z8.z)), z3 = __half22float2(*reinterpret_cast<const __half2*>(&z8.w));
                        const __nv_bfloat162 r0 = __floats2bfloat162_rn(F::OFF + z0.x, F::OFF + z2.x), r1 = __floats2bfloat162_rn(F::OFF + z0.y, F::OFF + z2.y);
                        const __nv_bfloat162 r2 = __floats2bfloat162_rn(F::OFF + z1.x, F::OFF + z3.x), r3 = __floats2bfloat162_rn(F::OFF + z1.y, F::OFF + z3.y);
                        zr[0] = *reinterpret_cast<const uint32_t*>(&r0); zr[1] = *reinterpret_cast<const uint32_t*>(&r1);
                        zr[2] = *reinterpret_cast<const uint32_t*>(&r2); zr[3] = *reinterpret_cast<const uint32_t*>(&r3);
                    }
#pragma unroll
                    for (int tt = 0; tt < NT; ++tt) {
                        const uint4 xv = *reinterpret_cast<const uint4*>(ys + (c * TOKS + g + 8 * tt) * xp + (un * 4 + q) * 16);
                        st_mma(za[tt], zr[0], 0u, zr[1], 0u, xv.x, xv.y);
                        st_mma(za[tt], zr[2], 0u, zr[3], 0u, xv.z, xv.w);
                    }
                }
                if (g == 0) {
#pragma unroll
                    for (int tt = 0; tt < NT; ++tt) {
                        zp[warp * 32 + c * 16 + 8 * tt + 2 * q] += za[tt][0];
                        zp[warp * 32 + c * 16 + 8 * tt + 2 * q + 1] += za[tt][1];
                    }
                }
            }
        }
        if (live) {
            for (int stg = cs; stg < ce; ++stg, ++it) {
                cp_wait<F::BNS - 1>();
                __syncwarp();
                const uint8_t* slot = ring + (it % F::BNS) * F::BSLOT;
#pragma unroll
                for (int su = 0; su < F::SU; ++su) {
                    const int ul = (stg - cs) * F::SU + su;    // 32-column unit inside the staged slice
                    uint32_t mx[4][F::BPAIR];                  // [column i of the lane's four][pair], transposed
                    if constexpr (BITS == 2) {
                        const uint4 w = *reinterpret_cast<const uint4*>(slot + su * 128 + g * 16);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 2; ++j)
                                mx[i][j] = st_movm(((st_comp(w, i) >> (2 * (2 * q + j))) & 0x00030003u) | 0x43004300u);
                    } else {
                        uint4 w[F::NLD];
                        st_load_words<BITS>(slot, g, q, w);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t pr[4];
                            st_unpack<BITS>(st_comp(w[0], i), F::NLD > 1 ? st_comp(w[F::NLD - 1], i) : 0u, q, pr);
#pragma unroll
                            for (int t = 0; t < 4; ++t) mx[i][t] = st_movm(pr[t]);
                        }
                    }
#pragma unroll
                    for (int tt = 0; tt < NT; ++tt) {
                        const uint4 xv = *reinterpret_cast<const uint4*>(ys + (copy * TOKS + g + 8 * tt) * xp + (ul * 4 + q) * 16);
#pragma unroll
                        for (int t = 0; t < NTILE; ++t) {
                            st_mma(acc[t][tt], mx[0][2 * t], mx[0][2 * t + 1], mx[1][2 * t], mx[1][2 * t + 1], xv.x, xv.y);
                            st_mma(acc[t][tt], mx[2][2 * t], mx[2][2 * t + 1], mx[3][2 * t], mx[3][2 * t + 1], xv.z, xv.w);
                        }
                    }
                }
                __syncwarp();
                issue(it + F::BNS);
            }
        }
        __syncthreads();
    }
    cp_wait<0>();
    for (int e = threadIdx.x; e < 32; e += blockDim.x) {   // zero-point sums of the whole range, warps added in order
        float z = 0.f;
        for (int w = 0; w < W; ++w) z += zp[w * 32 + e];
        zc[e] = z;
    }
    __syncthreads();
    // accumulator element (t, tt, e): MMA row g + 8 (e >> 1) of tile t = matrix 2t + (e >> 1), column g of it; token 2q + (e & 1) + 8 tt
    {
        const int pw = tile_c + 4;
#pragma unroll
        for (int t = 0; t < NTILE; ++t)
#pragma unroll
            for (int tt = 0; tt < NT; ++tt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int m = 2 * t + (e >> 1);        // pair index of the matrix
                    int f;                                 // feature of matrix m, column g (lane q' = g >> 1 supplied half g & 1)
                    if constexpr (BITS == 2) f = 2 * (g >> 1) + m + 8 * (g & 1);
                    else if constexpr (BITS == 8) f = 16 * (m >> 1) + 4 * (g >> 1) + 2 * (m & 1) + (g & 1);
                    else f = 8 * (g >> 1) + m + 4 * (g & 1);
                    const int tok = 2 * q + (e & 1) + 8 * tt;
                    part[tok * pw + F::FW * warp + f] = acc[t][tt][e] - zc[copy * 16 + tok];
                }
    }
    st_epilogue<true, TOKS>(p, part, hs, hfull, lup, tile_c, rank);
}

// Raising a kernel's dynamic shared-memory limit is a per-function AND per-device setting: `done` belongs to one kernel
// instantiation and holds, per device ordinal, the limit already set there.
template <typename Kern>
bool st_configure(Kern kern, size_t smem_bytes, size_t (&done)[ST_MAX_DEVICES], std::mutex& mu) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && dev < ST_MAX_DEVICES && done[dev] >= smem_bytes) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess) return false;
    if (dev >= 0 && dev < ST_MAX_DEVICES) done[dev] = smem_bytes;
    return true;
}

template <int BITS, int NT, bool TRANSPOSED>
int st_launch(const StreamParams& p, int W, int tiles, size_t smem_bytes, cudaStream_t st) {
    static std::mutex mu;
    static size_t done[ST_MAX_DEVICES] = {};
    cudaError_t err;
    const dim3 grid((unsigned)p.ks, (unsigned)tiles), block((unsigned)(32 * W));
    if (TRANSPOSED) {
        auto kern = stream_bwd_kernel<BITS, NT>;
        if (!st_configure(kern, smem_bytes, done, mu)) return QLORA_ERR_CUDA;
        err = launch_pdl(kern, grid, block, smem_bytes, st, (unsigned)p.ks, p);
    } else {
        auto kern = stream_fwd_kernel<BITS, NT>;
        if (!st_configure(kern, smem_bytes, done, mu)) return QLORA_ERR_CUDA;
        err = launch_pdl(kern, grid, block, smem_bytes, st, (unsigned)p.ks, p);
    }
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// Warps per CTA of the backward kernel: the features of a CTA must lie in one group or span exactly two.
int bwd_warps(int bits, int g) {
    const int fw = bits == 2 ? 16 : 32;
    for (int W = 8; W >= 1; W /= 2)
        if (g % (W * fw) == 0 || W * fw == 2 * g) return W;
    return 0;
}

int fwd_kb(int bits) { return bits == 2 ? 64 : 32; }

}  // namespace

bool stream_supported(const qlora_desc& d, int M, bool transposed) {
    if (M < 1 || M > 16) return false;
    if (d.K < 32 || d.N < 8) return false;
    if (transposed) return bwd_warps(d.bits, d.group_size) > 0;
    return d.group_size % fwd_kb(d.bits) == 0;
}

int launch_stream_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q, const void* scales,
                       const void* zeros, const void* Ldown, const void* Lup, float* P, bool p_is_input, void* Out,
                       cudaStream_t st) {
    StreamParams p{};
    p.M = M; p.K = d.K; p.N = d.N; p.g = d.group_size; p.r = d.r;
    p.C = transposed ? d.K : d.N;
    p.s = d.r > 0 ? d.alpha / (float)d.r : 0.f;
    p.In = (const __nv_bfloat16*)In; p.Q = (const uint32_t*)Q; p.scales = (const __half*)scales; p.zeros = (const __half*)zeros;
    p.Ldown = (const __nv_bfloat16*)Ldown; p.Lup = (const __nv_bfloat16*)Lup; p.P = P; p.Out = (__nv_bfloat16*)Out;
    p.fused = (d.r > 0 && !p_is_input) ? 1 : 0;
    if (p.fused && d.r > 16) return QLORA_ERR_INVALID_ARG;
    const int nt = M > 8 ? 2 : 1, toks = 8 * nt;
    int W, tile_c, units;                                  // warps per CTA, output columns per CTA, contraction stages
    if (transposed) {
        W = bwd_warps(d.bits, d.group_size);
        if (W == 0) return QLORA_ERR_UNSUPPORTED;
        tile_c = W * (d.bits == 2 ? 16 : 32);
        p.copies = tile_c > d.group_size ? 2 : 1;
        units = (d.N + (d.bits == 2 ? 128 : 32) - 1) / (d.bits == 2 ? 128 : 32);
    } else {
        if (d.group_size % fwd_kb(d.bits) != 0) return QLORA_ERR_UNSUPPORTED;
        W = d.N >= 256 ? 8 : (d.N >= 128 ? 4 : (d.N >= 64 ? 2 : 1));
        tile_c = 32 * W;
        p.copies = 1;
        units = (d.K + fwd_kb(d.bits) - 1) / fwd_kb(d.bits);
    }
    const int tiles = (p.C + tile_c - 1) / tile_c;
    // split the contraction until the grid covers the GPU (about one CTA per SM), keeping a few stages per CTA
    int ks = 1;
    while (ks < 8 && tiles * ks < 120 && units / (2 * ks) >= 4 && tile_c / (2 * ks) >= 1) ks *= 2;
    p.ks = ks;
    p.xc = (transposed && p.copies * toks > 16) ? 256 : 512;
    const int sl = tile_c / ks;
    p.lup_staged = (sl * d.r * 2 <= ST_LUP_BYTES) ? 1 : 0;
    size_t smem;
    if (transposed) {
        const int bslot = (d.bits == 2 ? 1 : d.bits) * 128 * (d.bits == 2 ? 4 : 1), bns = d.bits == 8 ? 8 : 16;
        smem = (size_t)W * bns * bslot + (size_t)p.copies * toks * (p.xc * 2 + 64) + (size_t)(W * 32 + 32 + 256 + 1024) * 4 + ST_LUP_BYTES;
    } else {
        const int kb = fwd_kb(d.bits), rows = kb * d.bits / 32, slot = rows * 128 + 128;
        const int ns = d.bits == 8 ? 7 : (d.bits == 3 ? 16 : 12);
        const int xpad = d.bits == 2 ? 16 : (d.bits == 8 ? 32 : 64);
        smem = (size_t)W * ns * slot + (size_t)toks * (p.xc * 2 + xpad) + (size_t)(toks * (p.xc / 8) + (p.xc / kb + 1) * toks + 256 + 1024) * 4 + ST_LUP_BYTES;
    }
    // the partial tile [toks][tile_c + 4] fp32 reuses the rings
    const size_t part = (size_t)16 * (tile_c + 4) * 4;
    if (smem < part + 4096) smem = part + 4096;
#define QLORA_ST(B, NT)                                                                                   \
    return transposed ? st_launch<B, NT, true>(p, W, tiles, smem, st) : st_launch<B, NT, false>(p, W, tiles, smem, st)
#define QLORA_ST_BITS(NT)           \
    switch (d.bits) {               \
        case 2: QLORA_ST(2, NT);    \
        case 3: QLORA_ST(3, NT);    \
        case 4: QLORA_ST(4, NT);    \
        case 8: QLORA_ST(8, NT);    \
    }
    if (nt == 1) { QLORA_ST_BITS(1) } else { QLORA_ST_BITS(2) }
#undef QLORA_ST_BITS
#undef QLORA_ST
    return QLORA_ERR_UNSUPPORTED;
}

}  // namespace qlora
