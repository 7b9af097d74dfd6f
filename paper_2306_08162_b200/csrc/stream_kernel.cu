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
//   - the contraction is split over a cluster of up to 8 CTAs, and inside a CTA over up to four sets of warps (sixteen
//     warps per SM keep the schedulers busy).  CTA i of a cluster finishes a slice of the columns: every CTA stores its
//     partial sums for that slice straight into i's shared memory (distributed shared memory; nothing waits on a remote
//     store), one cluster barrier later i adds them in a fixed order.  No workspace, no counters, and the result is the
//     same on every run;
//   - the LoRA down-projection (H = X A^T, G = dY B) over the CTA's part of the contraction comes from a few MMAs fed
//     straight from global memory (ranks up to 16), reduced with the partial tiles; the update s P L is added in the
//     epilogue in fp32 before the one rounding to bf16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "common.cuh"
#include "device_state.h"
#include "launch.h"

namespace qlora {
namespace {

constexpr int ST_MAX_DEVICES = kMaxDevices;

template <int BITS>
struct Fmt {
    static constexpr float OFF = BITS == 8 ? 0.f : 128.f;   // what the integer operand carries on top of the code
    // forward: a ring stage = KB contraction elements x 32 columns of one warp (+ the scale / zero chunk of its group)
    static constexpr int KB = BITS == 2 ? 64 : 32;
    static constexpr int ROWS = KB * BITS / 32;              // packed rows per stage: 4, 3, 4, 8
    static constexpr int SLOT = ROWS * 128 + 128;
    static constexpr int NS = BITS == 8 ? 5 : 8;            // ring stages per warp: 4 - 5.6 KB in flight per warp
    static constexpr int STEPS = KB / 16;                    // k16 MMA steps per stage
    static constexpr int NPAIR = 2 * STEPS;                  // bf16 pairs per column and lane
    static constexpr int NLD = (BITS == 3 || BITS == 8) ? 2 : 1;
    static constexpr int XPAD = BITS == 2 ? 16 : (BITS == 8 ? 32 : 64);   // pitch of an activation row = 2 xc + XPAD bytes
    // backward: a warp owns FW output features (BROWS packed rows); a ring stage = SU units of 32 columns
    static constexpr int FW = BITS == 2 ? 16 : 32;
    static constexpr int BROWS = FW * BITS / 32;             // 1, 3, 4, 8
    static constexpr int SU = BITS == 2 ? 4 : 1;
    static constexpr int BSLOT = BROWS * 128 * SU;
    static constexpr int BNS = BITS == 8 ? 4 : 8;
    static constexpr int BPAIR = BITS == 2 ? 2 : 4;          // pairs per column and lane
};

struct StreamParams {
    int M, K, N, g, r;
    int C;                       // output columns (N forward, K backward)
    int ks;                      // CTAs per cluster = ways the contraction is split
    int wc;                      // warps side by side in a CTA (32 columns forward, FW features backward each)
    int khs;                     // log2 of the parts the warps of a CTA split each staged slice of the contraction into
    int sls;                     // log2 of the columns a CTA of the cluster finishes (32 wc / ks or FW wc / ks)
    int lwc, lks;                // log2 of wc and of ks
    int xc;                      // contraction elements of the activations staged per pass (a power of two, all parts together)
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

// ---- reduction across the cluster: push, barrier, add locally -------------------------------------------------------
// The CTAs of a cluster hold partial tiles of the same output columns.  CTA `o` finishes the slice of tile_c / ks columns
// [o sl, o sl + sl): every CTA stores its partial sums for those columns straight into o's shared memory (remote stores,
// nothing waits on them), one cluster barrier later o adds what it received in a fixed order.  recv layout in the owner:
//   recv_part [ks][KH][sl][16 tokens] fp32      recv_h [ks][16 ranks][16 tokens] fp32
// Nobody reads a peer's shared memory, so a CTA may leave as soon as it has stored its own outputs.
struct RecvLayout {
    uint32_t part_addr, h_addr;   // shared-space addresses (the same in every CTA of the cluster)
    int sls, khs;                 // log2 of the slice width and of the parts per CTA
};

__device__ __forceinline__ void st_push2(const RecvLayout& rl, int src_rank, int kh, int cl, int tok, float v0, float v1) {
    const int owner = cl >> rl.sls, c = cl & ((1 << rl.sls) - 1);
    const uint32_t off = (uint32_t)(((((src_rank << rl.khs) + kh) << rl.sls) + c) * 16 + tok) * 4u;
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(st_map(rl.part_addr + off, (uint32_t)owner)), "f"(v0), "f"(v1) : "memory");
}

// This CTA's part of H / G (hs [16][16]) goes to every CTA of the cluster.
__device__ __forceinline__ void st_push_h(const RecvLayout& rl, const float* hs, int src_rank, int ks) {
    for (int e = threadIdx.x; e < 256 * ks; e += blockDim.x) {
        const int peer = e >> 8, i = e & 255;
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(st_map(rl.h_addr + (uint32_t)(src_rank * 256 + i) * 4u, (uint32_t)peer)), "f"(hs[i]) : "memory");
    }
}

__device__ __forceinline__ void st_cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void st_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// After the pushes: one cluster barrier, then the owner adds (source rank, part) in order, adds s P L, stores bf16.
template <bool TRANSPOSED, int TOKS>
__device__ __forceinline__ void st_finish(const StreamParams& p, const float* recv_part, const float* recv_h, float* hfull,
                                          const __nv_bfloat16* lup, int tile_c, int rank) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int sl = tile_c / p.ks, KH = 1 << p.khs;
    st_cluster_sync();                                    // every CTA's stores into this CTA's shared memory are visible
    if (p.r > 0 && p.fused) {
        for (int e = tid; e < 256; e += nthr) {
            float h = 0.f;
            for (int rk = 0; rk < p.ks; ++rk) h += recv_h[rk * 256 + e];
            hfull[e] = h;
            const int j = e >> 4, tok = e & 15;
            if (blockIdx.y == 0 && rank == 0 && tok < p.M && j < p.r) p.P[(size_t)tok * p.r + j] = h;
        }
        __syncthreads();
    }
    for (int e = tid; e < sl * TOKS; e += nthr) {
        const int tok = e % TOKS, c = e / TOKS;           // TOKS is a power of two
        const int col = blockIdx.y * tile_c + rank * sl + c;
        float v = 0.f;
        for (int i = 0; i < p.ks * KH; ++i) v += recv_part[(i * sl + c) * 16 + tok];
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

// Before griddepcontrol.wait nothing but the frozen weights may be READ, but lines can be asked into L2 (the point of
// coherence: a line the predecessor rewrites afterwards is simply updated there); the kernels do that for the slices of
// the activations and adapters they load right after the wait.

// A warp's partial H / G tile ([16 ranks][16 tokens], MMA accumulator layout) -> its slot of hp.
template <int NT>
__device__ __forceinline__ void st_store_hp(float (&ah)[NT][4], float* hp, int warp, int g, int q) {
    float* mine = hp + warp * 256;
#pragma unroll
    for (int tt = 0; tt < 2; ++tt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            mine[(g + ((e & 2) ? 8 : 0)) * 16 + 8 * tt + 2 * q + (e & 1)] = tt < NT ? ah[tt < NT ? tt : 0][e] : 0.f;
}

// ------------------------------------------------------------------------------------------------------------
// Forward: Y = X W^T + s H B^T.  CTA (rank, tile): columns [32 wc tile, + 32 wc), contraction blocks [kb0, kb1) of KB
// elements.  Warp (cg, kh): 32 columns and the kh-th of KH consecutive parts of [kb0, kb1).  The activations of the
// parts are staged side by side, xpb blocks of every part per pass (one pass when the CTA's range fits the buffer).
// ------------------------------------------------------------------------------------------------------------
constexpr int ST_HSTEPS = 4;   // k16 steps of the fused down-projection whose operands a warp loads in one go

struct PartInfo { int k0, k1, gf, nseg; };   // a part's share of the current pass: contraction range, first group, segments

template <int BITS, int NT>
__global__ void __launch_bounds__(512, 1) stream_fwd_kernel(const StreamParams p) {
    using F = Fmt<BITS>;
    constexpr int TOKS = 8 * NT, LTOKS = NT == 1 ? 3 : 4;
    constexpr int KP = BITS == 2 ? 16 : 8;                 // contraction elements per staged item
    constexpr int LKB = BITS == 2 ? 6 : 5;
    pdl_launch_dependents();
    st_cluster_arrive_relaxed();                           // waited for before the first store into a peer's shared memory
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ PartInfo tab[4];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, q = lane & 3;
    const int nthr = blockDim.x, nw = nthr >> 5, tile_c = 32 * p.wc, KH = 1 << p.khs;
    const int cg = warp & (p.wc - 1), kh = warp >> p.lwc;
    const int rank = (int)st_cluster_rank();
    const int col0 = blockIdx.y * tile_c + 32 * cg;
    const int nblk = (p.K + F::KB - 1) >> LKB;
    const int kb0 = (nblk * rank) >> p.lks, kb1 = (nblk * (rank + 1)) >> p.lks, nb = kb1 - kb0;
    const int wb0 = kb0 + ((nb * kh) >> p.khs), wb1 = kb0 + ((nb * (kh + 1)) >> p.khs);
    const int xp = p.xc * 2 + F::XPAD;
    const int xpb = (p.xc >> LKB) >> p.khs;                // blocks of a part staged per pass
    const int bpg = p.g >> LKB;                            // blocks per group
    const int sl = tile_c >> p.lks;
    uint8_t* ring = smem + warp * (F::NS * F::SLOT);
    uint8_t* xs = smem + nw * (F::NS * F::SLOT);           // [TOKS][xp] permuted activations: KH parts side by side
    float* sxc = reinterpret_cast<float*>(xs + TOKS * xp); // [TOKS][xc / 8] sums of 8 activations
    float* sxs = sxc + TOKS * (p.xc >> 3);                 // [KH][xpb + 1][TOKS] sums per (part, group) segment of the pass
    float* hs = sxs + KH * (xpb + 1) * TOKS;               // [16][16] this CTA's part of H
    float* hfull = hs + 256;                               // [r <= 64][16] the whole of H
    __nv_bfloat16* lup = reinterpret_cast<__nv_bfloat16*>(hfull + 1024);
    float* hp = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(lup) + ST_LUP_BYTES);   // [nw][16][16]
    float* recv_h = hp + nw * 256;                         // [ks][16][16]
    float* recv_part = recv_h + p.ks * 256;                // [ks][KH][sl][16]
    RecvLayout rl;
    rl.part_addr = s_u32(recv_part); rl.h_addr = s_u32(recv_h); rl.sls = p.sls; rl.khs = p.khs;

    // ---- the copy side of this warp: blocks wb0 .. wb1 - 1 in order, NS ahead of the arithmetic ----
    const int i_row = lane >> 3, i_ch = lane & 7;
    const bool i_col_ok = col0 + 4 * i_ch < p.N;
    const uint32_t* i_src = p.Q + (size_t)(wb0 * F::ROWS + i_row) * p.N + col0 + 4 * i_ch;   // row i_row of block wb0
    const size_t i_stride = (size_t)F::ROWS * p.N;
    const uint32_t i_dst = s_u32(ring) + st_swz(i_row, i_ch);
    const bool i_sz_lane = lane < 8 && col0 + 8 * (lane & 3) < p.N;
    const __half* i_sz = (lane < 4 ? p.scales : p.zeros) + col0 + 8 * (lane & 3);
    int i_blk = wb0, i_gpos = wb0 % bpg, i_slot = 0;
    bool i_first = true;
    auto issue = [&]() {
        if (i_blk < wb1) {
            const uint32_t dst = i_dst + i_slot * F::SLOT;
            if (BITS != 3 || i_row < 3) {
                const bool ok = i_col_ok && (BITS != 2 || i_blk * F::ROWS + i_row < (p.K >> 4));
                cp16(dst, ok ? i_src : p.Q, ok ? 16 : 0);
                if (BITS == 8) cp16(dst + 512, i_col_ok ? i_src + 4 * (size_t)p.N : p.Q, i_col_ok ? 16 : 0);
            }
            if ((i_gpos == 0 || i_first) && lane < 8)      // first block of a group in this part: its scales and zeros
                cp16(s_u32(ring) + i_slot * F::SLOT + F::ROWS * 128 + lane * 16, i_sz_lane ? i_sz + (size_t)(i_blk / bpg) * p.N : p.scales,
                     i_sz_lane ? 16 : 0);
            i_first = false;
            i_src += i_stride;
            ++i_blk;
            if (++i_gpos == bpg) i_gpos = 0;
        }
        if (++i_slot == F::NS) i_slot = 0;
        cp_commit();
    };
#pragma unroll 1
    for (int it = 0; it < F::NS; ++it) issue();            // frozen weights only: in flight while the predecessor finishes
    {   // ask the lines this CTA will read right after the wait into L2: its slices of X, A and B
        const int k_lo = kb0 << LKB, kbytes = (min(kb1 << LKB, p.K) - k_lo) * 2;
        const int lines = (kbytes + 127) >> 7, rows = p.M + ((p.r > 0 && p.fused) ? p.r : 0);
        for (int e = tid; e < rows * lines; e += nthr) {
            const int rr = e / lines, i = e - rr * lines;
            const __nv_bfloat16* base = rr < p.M ? p.In + (size_t)rr * p.K : p.Ldown + (size_t)(rr - p.M) * p.K;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(base + k_lo) + (size_t)i * 128));
        }
        const int c_lo = blockIdx.y * tile_c + rank * sl;
        if (p.r > 0 && c_lo < p.N && tid * 64 < min(sl, p.N - c_lo) * p.r)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.Lup + (size_t)c_lo * p.r + tid * 64));
    }

    pdl_wait();

    // ---- LoRA: this CTA's part of H = X A^T (k16 steps dealt to the warps, operands straight from global memory); the
    // loads of the first ST_HSTEPS steps are issued here and used once the activation slice is on its way too ----
    const bool fused = p.r > 0 && p.fused;
    const int h_k0 = (kb0 << LKB) + 16 * warp, h_ke = min(kb1 << LKB, p.K);
    uint32_t ha[ST_HSTEPS][4], hb[ST_HSTEPS][NT][2];
    auto h_load = [&](int kk) {
        const __nv_bfloat16* a_lo = p.Ldown + (size_t)g * p.K + 2 * q;
        const __nv_bfloat16* a_hi = a_lo + 8 * (size_t)p.K;
        const __nv_bfloat16* x_lo = p.In + (size_t)g * p.K + 2 * q;
#pragma unroll
        for (int h = 0; h < ST_HSTEPS; ++h) {
            const int k0 = kk + 16 * nw * h;
            const bool in = k0 < h_ke;
            ha[h][0] = (in && g < p.r) ? ldg32(a_lo + k0) : 0u; ha[h][2] = (in && g < p.r) ? ldg32(a_lo + k0 + 8) : 0u;
            ha[h][1] = (in && g + 8 < p.r) ? ldg32(a_hi + k0) : 0u; ha[h][3] = (in && g + 8 < p.r) ? ldg32(a_hi + k0 + 8) : 0u;
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const bool tin = in && g + 8 * tt < p.M;
                hb[h][tt][0] = tin ? ldg32(x_lo + 8 * tt * (size_t)p.K + k0) : 0u;
                hb[h][tt][1] = tin ? ldg32(x_lo + 8 * tt * (size_t)p.K + k0 + 8) : 0u;
            }
        }
    };
    if (fused) h_load(h_k0);
    st_stage_lup<false>(p, lup, hfull, tile_c, rank);

    // ---- main loop ----
    float acc[2][NT][4], grp[2][NT][4];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[u][tt][e] = grp[u][tt][e] = 0.f;
    float sc[4] = {0.f, 0.f, 0.f, 0.f}, cz[4] = {0.f, 0.f, 0.f, 0.f};   // this lane's four columns: scale, -scale (OFF + zero)
    int c_slot = 0;
    const int lcpt = 31 - __clz(p.xc / KP), lcpp = lcpt - p.khs;          // log2: items per token row, per part of it
    const int npass = (((nb + KH - 1) >> p.khs) + xpb - 1) / xpb;
    if (npass == 0) st_cluster_wait();                     // (an empty range: the wait below is never reached)
    for (int ps = 0; ps < npass; ++ps) {
        // this warp's blocks of the pass, and what the staging needs to know about every part
        const int pb0 = min(wb0 + ps * xpb, wb1), pb1 = min(wb1, pb0 + xpb);
        const int wk0 = pb0 << LKB, wk1 = min(pb1 << LKB, p.K);
        const int gf = wk0 / p.g;
        if (cg == 0 && lane == 0) { tab[kh].k0 = wk0; tab[kh].k1 = wk1; tab[kh].gf = gf; tab[kh].nseg = wk1 > wk0 ? (wk1 - 1) / p.g - gf + 1 : 0; }
        // stage the activations: permuted for the fragment loads, plus the sums the zero-points need
        {
            constexpr int NB = BITS == 2 ? 2 : 4;          // items per round, their loads issued together
            const int n_items = TOKS << lcpt;
            for (int e0 = tid; e0 < n_items; e0 += NB * nthr) {
                uint4 v0[NB], v1[NB];
                int tk[NB], ci[NB];
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    const int e = e0 + j * nthr;
                    tk[j] = e >> lcpt; ci[j] = e & ((1 << lcpt) - 1);
                    const int h = ci[j] >> lcpp, cl = ci[j] & ((1 << lcpp) - 1);
                    const int hb0 = kb0 + ((nb * h) >> p.khs), hb1 = kb0 + ((nb * (h + 1)) >> p.khs);
                    const int k = (min(hb0 + ps * xpb, hb1) << LKB) + cl * KP, kend = min(min(hb1, hb0 + (ps + 1) * xpb) << LKB, p.K);
                    v0[j] = make_uint4(0, 0, 0, 0); v1[j] = make_uint4(0, 0, 0, 0);
                    if (e < n_items && tk[j] < p.M && k < kend) {
                        v0[j] = *reinterpret_cast<const uint4*>(p.In + (size_t)tk[j] * p.K + k);
                        if (KP == 16 && k + 8 < kend) v1[j] = *reinterpret_cast<const uint4*>(p.In + (size_t)tk[j] * p.K + k + 8);
                    }
                }
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    if (e0 + j * nthr >= n_items) break;
                    uint8_t* dst = xs + tk[j] * xp + ci[j] * (2 * KP);
                    if constexpr (BITS == 2) {             // (x0,x8) (x1,x9) ... (x7,x15)
                        *reinterpret_cast<uint4*>(dst) = make_uint4(__byte_perm(v0[j].x, v1[j].x, 0x5410), __byte_perm(v0[j].x, v1[j].x, 0x7632),
                                                                    __byte_perm(v0[j].y, v1[j].y, 0x5410), __byte_perm(v0[j].y, v1[j].y, 0x7632));
                        *reinterpret_cast<uint4*>(dst + 16) = make_uint4(__byte_perm(v0[j].z, v1[j].z, 0x5410), __byte_perm(v0[j].z, v1[j].z, 0x7632),
                                                                         __byte_perm(v0[j].w, v1[j].w, 0x5410), __byte_perm(v0[j].w, v1[j].w, 0x7632));
                        sxc[tk[j] * (p.xc >> 3) + 2 * ci[j]] = st_sum8(v0[j]);
                        sxc[tk[j] * (p.xc >> 3) + 2 * ci[j] + 1] = st_sum8(v1[j]);
                    } else {
                        *reinterpret_cast<uint4*>(dst) = BITS == 8 ? v0[j] : st_permute8(v0[j]);
                        sxc[tk[j] * (p.xc >> 3) + ci[j]] = st_sum8(v0[j]);
                    }
                }
            }
            if (ps == 0 && fused) {                        // the down-projection's MMAs, with the activations' loads behind them
                float ah[NT][4];
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) ah[tt][0] = ah[tt][1] = ah[tt][2] = ah[tt][3] = 0.f;
                for (int kk = h_k0;;) {
#pragma unroll
                    for (int h = 0; h < ST_HSTEPS; ++h)
#pragma unroll
                        for (int tt = 0; tt < NT; ++tt) st_mma(ah[tt], ha[h][0], ha[h][1], ha[h][2], ha[h][3], hb[h][tt][0], hb[h][tt][1]);
                    kk += 16 * nw * ST_HSTEPS;
                    if (kk >= h_ke) break;
                    h_load(kk);
                }
                st_store_hp<NT>(ah, hp, warp, g, q);
            }
            __syncthreads();
            {   // sums per (part, group segment): four lanes per (token, segment), segments numbered through the parts
                int n_all = 0;
                for (int h = 0; h < KH; ++h) n_all += tab[h].nseg;
                const int total = n_all << LTOKS;
                for (int base = 0; base < total; base += nthr >> 2) {      // the same trip count for every thread
                    const int task = base + (tid >> 2), sub = tid & 3;
                    const bool on = task < total;
                    const int tok = task & (TOKS - 1);
                    int h = 0, sg = on ? task >> LTOKS : 0;
                    while (on && sg >= tab[h].nseg) { sg -= tab[h].nseg; ++h; }
                    const PartInfo pi = tab[h];
                    const int a = max(pi.k0, (pi.gf + sg) * p.g), b = min(pi.k1, (pi.gf + sg + 1) * p.g);
                    const float* src = sxc + tok * (p.xc >> 3) + ((h << lcpp) * KP + (a - pi.k0)) / 8;
                    float sum = 0.f;
                    if (on)
                        for (int c8 = sub; c8 < (b - a) >> 3; c8 += 4) sum += src[c8];
                    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                    if (on && sub == 0) sxs[(h * (xpb + 1) + sg) * TOKS + tok] = sum;
                }
            }
            if (ps == 0 && fused) {
                for (int e = tid; e < 256; e += nthr) {
                    float h = 0.f;
                    for (int w = 0; w < nw; ++w) h += hp[w * 256 + e];
                    hs[e] = h;
                }
            }
            __syncthreads();
            if (ps == 0) {
                st_cluster_wait();                         // every CTA of the cluster is running: its shared memory may be written
                if (fused) st_push_h(rl, hs, rank, p.ks);
            }
        }
        int gpos = pb0 - gf * bpg, grpi = gf;
        const uint8_t* xw = xs + (kh * xpb << (LKB + 1)) + (BITS == 2 ? 32 * q : (BITS == 8 ? 8 * q : 16 * q)) + g * xp;
#pragma unroll 2
        for (int blk = pb0; blk < pb1; ++blk) {
            cp_wait<F::NS - 1>();
            __syncwarp();
            const uint8_t* slot = ring + c_slot * F::SLOT;
            if (gpos == 0 || blk == wb0) {                 // a new group: this lane's scales and zero-points
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
            const uint8_t* xb = xw + ((blk - pb0) << (LKB + 1));
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const uint8_t* xr = xb + 8 * tt * xp;
                if constexpr (BITS == 2) {
                    const uint4 v0 = *reinterpret_cast<const uint4*>(xr);
                    const uint4 v1 = *reinterpret_cast<const uint4*>(xr + 16);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v0.z; xf[tt][3] = v0.w;
                    xf[tt][4] = v1.x; xf[tt][5] = v1.y; xf[tt][6] = v1.z; xf[tt][7] = v1.w;
                } else if constexpr (BITS == 8) {
                    const uint2 v0 = *reinterpret_cast<const uint2*>(xr);
                    const uint2 v1 = *reinterpret_cast<const uint2*>(xr + 32);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v1.x; xf[tt][3] = v1.y;
                } else {
                    const uint4 v0 = *reinterpret_cast<const uint4*>(xr);
                    xf[tt][0] = v0.x; xf[tt][1] = v0.y; xf[tt][2] = v0.z; xf[tt][3] = v0.w;
                }
            }
            // two tiles of 16 columns: rows g / g + 8 of tile u are columns 4g + 2u / 4g + 2u + 1
            uint32_t pc[4][F::NPAIR];                      // [column i of the lane's four][pair]
#pragma unroll
            for (int i = 0; i < 4; ++i) st_unpack<BITS>(st_comp(w[0], i), F::NLD > 1 ? st_comp(w[F::NLD - 1], i) : 0u, q, pc[i]);
#pragma unroll
            for (int s = 0; s < F::STEPS; ++s)             // MMAs into the same accumulator are 2 NT instructions apart
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int tt = 0; tt < NT; ++tt)
                        st_mma(grp[u][tt], pc[2 * u][2 * s], pc[2 * u + 1][2 * s], pc[2 * u][2 * s + 1], pc[2 * u + 1][2 * s + 1], xf[tt][2 * s], xf[tt][2 * s + 1]);
            if (gpos == bpg - 1 || blk + 1 == pb1) {       // end of a group segment: scale, correct, start afresh
                const float* sxr = sxs + (kh * (xpb + 1) + grpi - gf) * TOKS + 2 * q;
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) {
                    const float2 sx = *reinterpret_cast<const float2*>(sxr + 8 * tt);
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
            if (++gpos == bpg) { gpos = 0; ++grpi; }
            if (++c_slot == F::NS) c_slot = 0;
            __syncwarp();
            issue();
        }
        if (ps + 1 < npass) __syncthreads();               // the staged activations may be overwritten
    }
    // accumulator element (u, tt, e): column 4g + 2u + (e >> 1) of this warp's 32, token 2q + (e & 1) + 8 tt; sent to the
    // CTA that finishes that column
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt) {
            st_push2(rl, rank, kh, 32 * cg + 4 * g + 2 * u, 2 * q + 8 * tt, acc[u][tt][0], acc[u][tt][1]);
            st_push2(rl, rank, kh, 32 * cg + 4 * g + 2 * u + 1, 2 * q + 8 * tt, acc[u][tt][2], acc[u][tt][3]);
        }
    st_finish<false, TOKS>(p, recv_part, recv_h, hfull, lup, tile_c, rank);
}

// ------------------------------------------------------------------------------------------------------------
// Backward: dX = dY W + s G A.  CTA (rank, tile): output features [FW wc tile, + FW wc), contraction stages [st0, st1)
// of 32 SU packed columns.  Warp (fw, kh): FW features (all inside one group) and the kh-th of KH consecutive parts of
// [st0, st1).  The slices of dY of the parts are staged side by side, xps stages of every part per pass.
// ------------------------------------------------------------------------------------------------------------
template <int BITS, int NT>
__global__ void __launch_bounds__(512, 1) stream_bwd_kernel(const StreamParams p) {
    using F = Fmt<BITS>;
    constexpr int TOKS = 8 * NT;
    constexpr int NTILE = F::BPAIR / 2;                    // 16-feature MMA tiles per warp
    constexpr int LSW = BITS == 2 ? 7 : 5;                 // log2 of the packed columns per stage
    pdl_launch_dependents();
    st_cluster_arrive_relaxed();                           // waited for before the first store into a peer's shared memory
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, q = lane & 3;
    const int nthr = blockDim.x, nw = nthr >> 5, tile_c = F::FW * p.wc, sl = tile_c >> p.lks, KH = 1 << p.khs;
    const int fw = warp & (p.wc - 1), kh = warp >> p.lwc;
    const int rank = (int)st_cluster_rank();
    const int tile_f0 = blockIdx.y * tile_c, f0 = tile_f0 + F::FW * fw;
    const bool live = f0 < p.K;                            // a warp beyond the last feature only keeps the barriers company
    const int row0 = f0 * BITS / 32;
    const int nst = (p.N + (1 << LSW) - 1) >> LSW;
    const int st0 = (nst * rank) >> p.lks, st1 = (nst * (rank + 1)) >> p.lks, ns = st1 - st0;
    const int ws0 = st0 + ((ns * kh) >> p.khs), ws1 = st0 + ((ns * (kh + 1)) >> p.khs);
    const int xp = p.xc * 2 + 64;
    const int xps = (p.xc >> LSW) >> p.khs;                // stages of a part staged per pass
    const int gk0 = tile_f0 / p.g;                         // group of the CTA's first feature
    const int ngroups = p.K / p.g;
    const int copy = p.copies > 1 ? (f0 - tile_f0) / p.g : 0;
    uint8_t* ring = smem + warp * (F::BNS * F::BSLOT);
    uint8_t* ys = smem + nw * (F::BNS * F::BSLOT);         // [copies][TOKS][xp] scaled, permuted slices of dY
    float* zp = reinterpret_cast<float*>(ys + p.copies * TOKS * xp);   // [nw][2][16] zero-point sums, per warp
    float* zc = zp + nw * 32;                              // [2][16] their total
    float* hs = zc + 32;
    float* hfull = hs + 256;
    __nv_bfloat16* lup = reinterpret_cast<__nv_bfloat16*>(hfull + 1024);
    float* hp = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(lup) + ST_LUP_BYTES);   // [nw][16][16]
    float* recv_h = hp + nw * 256;                         // [ks][16][16]
    float* recv_part = recv_h + p.ks * 256;                // [ks][KH][sl][16]
    RecvLayout rl;
    rl.part_addr = s_u32(recv_part); rl.h_addr = s_u32(recv_h); rl.sls = p.sls; rl.khs = p.khs;

    // ---- the copy side of this warp: stages ws0 .. ws1 - 1 in order, BNS ahead of the arithmetic ----
    const int i_row = BITS == 2 ? 0 : lane >> 3;
    const int i_coff = BITS == 2 ? 32 * (lane >> 3) + 4 * (lane & 7) : 4 * (lane & 7);   // column inside the stage
    const uint32_t* i_src = p.Q + (size_t)(row0 + i_row) * p.N;
    const uint32_t i_dst = s_u32(ring) + (BITS == 2 ? lane * 16 : st_swz(i_row, lane & 7));
    int i_stg = ws0, i_slot = 0;
    auto issue = [&]() {
        if (i_stg < ws1 && live) {
            const uint32_t dst = i_dst + i_slot * F::BSLOT;
            const int col = (i_stg << LSW) + i_coff;
            const bool ok = col < p.N;
            if (BITS != 3 || i_row < 3) {
                cp16(dst, ok ? i_src + col : p.Q, ok ? 16 : 0);
                if (BITS == 8) cp16(dst + 512, ok ? i_src + 4 * (size_t)p.N + col : p.Q, ok ? 16 : 0);
            }
            ++i_stg;
        }
        if (++i_slot == F::BNS) i_slot = 0;
        cp_commit();
    };
#pragma unroll 1
    for (int it = 0; it < F::BNS; ++it) issue();

    const int n_lo_cta = st0 << LSW, n_hi_cta = min(st1 << LSW, p.N);
    {   // ask the lines this CTA will read right after the wait into L2: its slices of dY, B, A and of the group parameters
        const int nbytes = (n_hi_cta - n_lo_cta) * 2, lines = (nbytes + 127) >> 7;
        const int rows = p.M + 2 * p.copies;
        for (int e = tid; e < rows * lines; e += nthr) {
            const int rr = e / lines, i = e - rr * lines;
            const char* base;
            if (rr < p.M) base = reinterpret_cast<const char*>(p.In + (size_t)rr * p.N + n_lo_cta);
            else {
                const int c = (rr - p.M) >> 1, gk = min(gk0 + c, ngroups - 1);
                base = reinterpret_cast<const char*>(((rr - p.M) & 1 ? p.zeros : p.scales) + (size_t)gk * p.N + n_lo_cta);
            }
            asm volatile("prefetch.global.L2 [%0];" ::"l"(base + (size_t)i * 128));
        }
        if (p.r > 0 && p.fused)
            for (int e = tid; e * 64 < (n_hi_cta - n_lo_cta) * p.r; e += nthr)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p.Ldown + (size_t)n_lo_cta * p.r + (size_t)e * 64));
        const int c_lo = tile_f0 + rank * sl;
        if (p.r > 0 && c_lo < p.K && tid < p.r) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.Lup + (size_t)tid * p.K + c_lo));
    }

    pdl_wait();

    // ---- LoRA: this CTA's part of G = dY B.  B [N, r] has the ranks contiguous, so a lane loads two ranks of its own
    // contraction column and movmatrix turns them into two columns of one rank.  The loads of the first ST_HSTEPS steps are
    // issued here and used once the slice of dY is on its way too ----
    const bool fused = p.r > 0 && p.fused;
    const int h_n0 = n_lo_cta + 16 * warp;
    uint32_t ha[ST_HSTEPS][4], hb[ST_HSTEPS][NT][2];
    auto h_load = [&](int nn) {
#pragma unroll
        for (int h = 0; h < ST_HSTEPS; ++h) {
            const int nb = nn + 16 * nw * h;
            const bool in = nb < n_hi_cta;
            const bool v0 = in && nb + g < p.N, v1 = in && nb + 8 + g < p.N;
            const __nv_bfloat16* b_lo = p.Ldown + (size_t)(nb + g) * p.r + 2 * q;
            const __nv_bfloat16* b_hi = b_lo + 8 * p.r;
            ha[h][0] = v0 ? ldg32(b_lo) : 0u; ha[h][2] = v1 ? ldg32(b_hi) : 0u;
            ha[h][1] = (v0 && p.r > 8) ? ldg32(b_lo + 8) : 0u; ha[h][3] = (v1 && p.r > 8) ? ldg32(b_hi + 8) : 0u;
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) {
                const int tok = g + 8 * tt;
                const __nv_bfloat16* y = p.In + (size_t)tok * p.N + nb + 2 * q;
                hb[h][tt][0] = (in && tok < p.M && nb + 2 * q < p.N) ? ldg32(y) : 0u;
                hb[h][tt][1] = (in && tok < p.M && nb + 8 + 2 * q < p.N) ? ldg32(y + 8) : 0u;
            }
        }
    };
    if (fused) h_load(h_n0);
    st_stage_lup<true>(p, lup, hfull, tile_c, rank);
    for (int e = tid; e < nw * 32; e += nthr) zp[e] = 0.f;

    float acc[NTILE][NT][4];
#pragma unroll
    for (int t = 0; t < NTILE; ++t)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt) acc[t][tt][0] = acc[t][tt][1] = acc[t][tt][2] = acc[t][tt][3] = 0.f;
    int c_slot = 0;
    const int lcpt = 31 - __clz(p.xc >> 3), lcpp = lcpt - p.khs;          // log2: 8-column items per token row, per part of it
    const int npass = (((ns + KH - 1) >> p.khs) + xps - 1) / xps;
    if (npass == 0) st_cluster_wait();                     // (an empty range: the wait below is never reached)
    for (int ps = 0; ps < npass; ++ps) {
        const int pb0 = min(ws0 + ps * xps, ws1), pb1 = min(ws1, pb0 + xps);     // this warp's stages of the pass
        // stage the slices of dY, once per group the CTA's features span, scaled by that group's scales (one rounding)
        {
            const int n_items = TOKS << lcpt;
            for (int e0 = tid; e0 < n_items; e0 += 2 * nthr) {                   // two items per round, loads first
                uint4 v[2], s8[2][2];
                int tk[2], ci[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int e = e0 + j * nthr;
                    tk[j] = e >> lcpt; ci[j] = e & ((1 << lcpt) - 1);
                    const int h = ci[j] >> lcpp, cl = ci[j] & ((1 << lcpp) - 1);
                    const int hs0 = st0 + ((ns * h) >> p.khs), hs1 = st0 + ((ns * (h + 1)) >> p.khs);
                    const int n = (min(hs0 + ps * xps, hs1) << LSW) + cl * 8, nend = min(min(hs1, hs0 + (ps + 1) * xps) << LSW, p.N);
                    v[j] = s8[j][0] = s8[j][1] = make_uint4(0, 0, 0, 0);
                    if (e < n_items && tk[j] < p.M && n < nend) {
                        v[j] = *reinterpret_cast<const uint4*>(p.In + (size_t)tk[j] * p.N + n);
#pragma unroll
                        for (int c = 0; c < 2; ++c)
                            if (c < p.copies && gk0 + c < ngroups) s8[j][c] = *reinterpret_cast<const uint4*>(p.scales + (size_t)(gk0 + c) * p.N + n);
                    }
                }
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if (e0 + j * nthr >= n_items) break;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        if (c >= p.copies) break;
                        const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&s8[j][c].x)), s1 = __half22float2(*reinterpret_cast<const __half2*>(&s8[j][c].y));
                        const float2 s2 = __half22float2(*reinterpret_cast<const __half2*>(&s8[j][c].z)), s3 = __half22float2(*reinterpret_cast<const __half2*>(&s8[j][c].w));
                        const __nv_bfloat162 o0 = __floats2bfloat162_rn(bf16_lo(v[j].x) * s0.x, bf16_hi(v[j].x) * s0.y);
                        const __nv_bfloat162 o1 = __floats2bfloat162_rn(bf16_lo(v[j].y) * s1.x, bf16_hi(v[j].y) * s1.y);
                        const __nv_bfloat162 o2 = __floats2bfloat162_rn(bf16_lo(v[j].z) * s2.x, bf16_hi(v[j].z) * s2.y);
                        const __nv_bfloat162 o3 = __floats2bfloat162_rn(bf16_lo(v[j].w) * s3.x, bf16_hi(v[j].w) * s3.y);
                        const uint4 o = make_uint4(*reinterpret_cast<const uint32_t*>(&o0), *reinterpret_cast<const uint32_t*>(&o1),
                                                   *reinterpret_cast<const uint32_t*>(&o2), *reinterpret_cast<const uint32_t*>(&o3));
                        *reinterpret_cast<uint4*>(ys + (c * TOKS + tk[j]) * xp + ci[j] * 16) = st_permute8(o);
                    }
                }
            }
            if (ps == 0 && fused) {                        // the down-projection's MMAs, with the slice's loads behind them
                float ag[NT][4];
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) ag[tt][0] = ag[tt][1] = ag[tt][2] = ag[tt][3] = 0.f;
                for (int nn = h_n0;;) {
#pragma unroll
                    for (int h = 0; h < ST_HSTEPS; ++h) {
                        const uint32_t a0 = st_movm(ha[h][0]), a1 = st_movm(ha[h][1]), a2 = st_movm(ha[h][2]), a3 = st_movm(ha[h][3]);
#pragma unroll
                        for (int tt = 0; tt < NT; ++tt) st_mma(ag[tt], a0, a1, a2, a3, hb[h][tt][0], hb[h][tt][1]);
                    }
                    nn += 16 * nw * ST_HSTEPS;
                    if (nn >= n_hi_cta) break;
                    h_load(nn);
                }
                st_store_hp<NT>(ag, hp, warp, g, q);
            }
            __syncthreads();
            if (ps == 0 && fused) {
                for (int e = tid; e < 256; e += nthr) {
                    float h = 0.f;
                    for (int w = 0; w < nw; ++w) h += hp[w * 256 + e];
                    hs[e] = h;
                }
            }
            // zero-point term: sum_n dYs[m, n] (OFF + z[G, n]) as one MMA row; the warps of a part share its 32-column units
            const int un_end = ((min(pb1 << LSW, p.N) - (pb0 << LSW)) + 31) >> 5;
            for (int c = 0; c < p.copies; ++c) {
                const int gk = gk0 + c;
                float za[NT][4];
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) za[tt][0] = za[tt][1] = za[tt][2] = za[tt][3] = 0.f;
                for (int un = fw; un < un_end; un += p.wc) {
                    const int n = (pb0 << LSW) + 32 * un + 8 * q;
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
                        const uint4 xv = *reinterpret_cast<const uint4*>(ys + (c * TOKS + g + 8 * tt) * xp + (((kh << lcpp) + un * 4 + q) << 4));
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
            if (ps == 0) {
                st_cluster_wait();                         // every CTA of the cluster is running: its shared memory may be written
                if (fused) {
                    __syncthreads();                       // hs is complete
                    st_push_h(rl, hs, rank, p.ks);
                }
            }
        }
        if (live) {
            const uint8_t* yw = ys + (copy * TOKS + g) * xp + (((kh << lcpp) + q) << 4);
#pragma unroll 2
            for (int stg = pb0; stg < pb1; ++stg) {
                cp_wait<F::BNS - 1>();
                __syncwarp();
                const uint8_t* slot = ring + c_slot * F::BSLOT;
#pragma unroll
                for (int su = 0; su < F::SU; ++su) {
                    const int ul = (stg - pb0) * F::SU + su;   // 32-column unit inside this part's staged slice
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
                        const uint4 xv = *reinterpret_cast<const uint4*>(yw + 8 * tt * xp + (ul << 6));
#pragma unroll
                        for (int t = 0; t < NTILE; ++t) {
                            st_mma(acc[t][tt], mx[0][2 * t], mx[0][2 * t + 1], mx[1][2 * t], mx[1][2 * t + 1], xv.x, xv.y);
                            st_mma(acc[t][tt], mx[2][2 * t], mx[2][2 * t + 1], mx[3][2 * t], mx[3][2 * t + 1], xv.z, xv.w);
                        }
                    }
                }
                if (++c_slot == F::BNS) c_slot = 0;
                __syncwarp();
                issue();
            }
        }
        __syncthreads();
    }
    if (tid < 32) {                                        // zero-point sums of the whole range, warps added in order
        float z = 0.f;
        for (int w = 0; w < nw; ++w) z += zp[w * 32 + tid];
        zc[tid] = z;
    }
    __syncthreads();
    // accumulator element (t, tt, e): MMA row g + 8 (e >> 1) of tile t = matrix 2t + (e >> 1), column g of it; token
    // 2q + (e & 1) + 8 tt.  The zero-point sum covers the CTA's whole range, so part 0 alone subtracts it.  Each pair of
    // tokens goes to the CTA that finishes that feature.
#pragma unroll
    for (int t = 0; t < NTILE; ++t)
#pragma unroll
        for (int tt = 0; tt < NT; ++tt)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int m = 2 * t + hh;                  // pair index of the matrix
                int f;                                     // feature of matrix m, column g (lane q' = g >> 1 supplied half g & 1)
                if constexpr (BITS == 2) f = 2 * (g >> 1) + m + 8 * (g & 1);
                else if constexpr (BITS == 8) f = 16 * (m >> 1) + 4 * (g >> 1) + 2 * (m & 1) + (g & 1);
                else f = 8 * (g >> 1) + m + 4 * (g & 1);
                const int tok = 2 * q + 8 * tt;
                const float z0 = kh == 0 ? zc[copy * 16 + tok] : 0.f, z1 = kh == 0 ? zc[copy * 16 + tok + 1] : 0.f;
                st_push2(rl, rank, kh, F::FW * fw + f, tok, acc[t][tt][2 * hh] - z0, acc[t][tt][2 * hh + 1] - z1);
            }
    st_finish<true, TOKS>(p, recv_part, recv_h, hfull, lup, tile_c, rank);
}

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

// Dynamic shared memory of a launch: the carve-up at the top of the two kernels, in the same order.
template <int BITS>
size_t st_smem_bytes(bool transposed, int nw, int toks, int xc, int copies, int KH, int ks, int tile_c) {
    using F = Fmt<BITS>;
    const size_t tail = (size_t)(256 + 1024) * 4 + ST_LUP_BYTES + (size_t)nw * 1024 + (size_t)ks * 1024 + (size_t)KH * tile_c * 64;
    if (transposed)
        return (size_t)nw * F::BNS * F::BSLOT + (size_t)copies * toks * (xc * 2 + 64) + (size_t)(nw * 32 + 32) * 4 + tail;
    return (size_t)nw * F::NS * F::SLOT + (size_t)toks * (xc * 2 + F::XPAD) + (size_t)(toks * (xc / 8) + KH * (xc / F::KB / KH + 1) * toks) * 4 + tail;
}

// Warps per CTA of the backward kernel: the features of a CTA must lie in one group or span exactly two.
int bwd_warps(int bits, int g) {
    const int fw = bits == 2 ? 16 : 32;
    const int order[4] = {4, 8, 2, 1};                     // four side by side leave room for four parts of the contraction
    for (int i = 0; i < 4; ++i)
        if (g % (order[i] * fw) == 0 || order[i] * fw == 2 * g) return order[i];
    return 0;
}

int fwd_kb(int bits) { return bits == 2 ? 64 : 32; }

__global__ void __launch_bounds__(512, 1) st_probe_kernel() {}

struct DeviceFacts { int sms = 0; int clusters[9] = {}; };

// SM count and how many clusters of 2 / 4 / 8 CTAs that own an SM each can run at once, per device ordinal.
const DeviceFacts& device_facts() {
    static std::mutex mu;
    static DeviceFacts facts[ST_MAX_DEVICES];
    static DeviceFacts fallback;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= ST_MAX_DEVICES) { fallback.sms = 148; fallback.clusters[2] = 74; fallback.clusters[4] = 32; fallback.clusters[8] = 14; return fallback; }
    std::lock_guard<std::mutex> lock(mu);
    DeviceFacts& f = facts[dev];
    if (f.sms == 0) {
        int v = 0;
        f.sms = (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) ? v : 148;
        (void)cudaFuncSetAttribute(st_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        for (int cs = 2; cs <= 8; cs *= 2) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)cs, (unsigned)f.sms);
            cfg.blockDim = dim3(512);
            cfg.dynamicSmemBytes = 200 * 1024;         // one CTA per SM, as the streaming kernels are
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = (unsigned)cs; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, st_probe_kernel, &cfg) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = f.sms / cs * 3 / 4; }
            f.clusters[cs] = n;
        }
    }
    return f;
}
int max_clusters(int cs) { return cs <= 1 ? device_facts().sms : device_facts().clusters[cs > 8 ? 8 : cs]; }
int sm_count_here() { return device_facts().sms; }

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
    int wc, tile_c, units;                                 // warps side by side, output columns per CTA, contraction stages
    if (transposed) {
        wc = bwd_warps(d.bits, d.group_size);
        if (wc == 0) return QLORA_ERR_UNSUPPORTED;
        tile_c = wc * (d.bits == 2 ? 16 : 32);
        p.copies = tile_c > d.group_size ? 2 : 1;
        units = (d.N + (d.bits == 2 ? 128 : 32) - 1) / (d.bits == 2 ? 128 : 32);
    } else {
        if (d.group_size % fwd_kb(d.bits) != 0) return QLORA_ERR_UNSUPPORTED;
        wc = d.N >= 128 ? 4 : (d.N >= 64 ? 2 : 1);
        tile_c = 32 * wc;
        p.copies = 1;
        units = (d.K + fwd_kb(d.bits) - 1) / fwd_kb(d.bits);
    }
    p.wc = wc;
    p.lwc = 0;
    while ((1 << p.lwc) < wc) ++p.lwc;
    const int tiles = (p.C + tile_c - 1) / tile_c;
    // split the contraction over a cluster until the grid covers the GPU: one CTA per SM, and no more clusters than can
    // run at once (the clusters of a launch that come later would wait for whole earlier ones to finish)
    int ks = 1;
    while (ks < 8 && tiles * 2 * ks <= max_clusters(2 * ks) * 2 * ks && tiles * 2 * ks <= sm_count_here() && units / (2 * ks) >= 4 &&
           tile_c / (2 * ks) >= 1)
        ks *= 2;
    p.ks = ks;
    p.lks = 0;
    while ((1 << p.lks) < ks) ++p.lks;
    // ... and inside a CTA until it has sixteen warps, while a warp keeps at least two stages
    p.khs = 0;
    while ((wc << (p.khs + 1)) <= 16 && p.khs < 2 && units / (ks << (p.khs + 1)) >= 2) ++p.khs;
    const int nw = wc << p.khs, KH = 1 << p.khs;
    const int sl = tile_c / ks;
    p.sls = 0;
    while ((1 << p.sls) < sl) ++p.sls;
    // the activations staged per pass (all parts of a CTA together): the CTA's whole range when that fits (one pass, two
    // barriers), else 512 at a time; a power of two, and at least one stage per part
    {
        const int unit = transposed ? (d.bits == 2 ? 128 : 32) : fwd_kb(d.bits);
        const int range = ((units + ks - 1) / ks + KH - 1) / KH * KH * unit;
        const int cap = (transposed && p.copies * toks > 16) ? 512 : 1024;
        p.xc = 128;
        while (p.xc < range && p.xc < cap) p.xc *= 2;
        if (p.xc < unit * KH) p.xc = unit * KH;
    }
    p.lup_staged = (sl * d.r * 2 <= ST_LUP_BYTES) ? 1 : 0;
    size_t smem = 0;
    switch (d.bits) {
        case 2: smem = st_smem_bytes<2>(transposed, nw, toks, p.xc, p.copies, KH, ks, tile_c); break;
        case 3: smem = st_smem_bytes<3>(transposed, nw, toks, p.xc, p.copies, KH, ks, tile_c); break;
        case 4: smem = st_smem_bytes<4>(transposed, nw, toks, p.xc, p.copies, KH, ks, tile_c); break;
        case 8: smem = st_smem_bytes<8>(transposed, nw, toks, p.xc, p.copies, KH, ks, tile_c); break;
    }
    if (smem > 227 * 1024) return QLORA_ERR_UNSUPPORTED;
#define QLORA_ST(B, NT)                                                                                   \
    return transposed ? st_launch<B, NT, true>(p, nw, tiles, smem, st) : st_launch<B, NT, false>(p, nw, tiles, smem, st)
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
