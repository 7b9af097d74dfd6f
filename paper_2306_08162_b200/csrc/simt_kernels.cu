// CUDA-core kernels of the quantized-linear + LoRA layer.  They are correct for every shape the library accepts
// and serve (a) shapes the tensor-core kernels do not tile, and (b) the skinny LoRA products, which are bound by
// HBM traffic rather than by arithmetic (Figure 1 of the paper: the green "MM" blocks and their gradients).
#include "common.cuh"
#include "device_state.h"
#include "launch.h"
#include "lora_down.cuh"

namespace qlora {

// ------------------------------------------------------------------------------------------------------------
// Generic tiled product with on-the-fly dequantisation.
//   forward        : Out[m, n] = sum_k In[m, k] W[n, k] + s sum_j P[m, j] B[n, j]        (T = K, C = N)
//   backward-input : Out[m, k] = sum_n In[m, n] W[n, k] + s sum_j P[m, j] A[j, k]        (T = N, C = K)
// 64 x 64 output tile, contraction step 16, 256 threads, 4 x 4 outputs per thread, fp32 accumulation.
// ------------------------------------------------------------------------------------------------------------
constexpr int SG_BM = 64, SG_BC = 64, SG_BT = 16;

template <bool TRANSPOSED>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(int bits, int g, int K, int N, int r, float s, int M, const __nv_bfloat16* __restrict__ In,
                 const uint32_t* __restrict__ Q, const __half* __restrict__ scales, const __half* __restrict__ zeros,
                 const __nv_bfloat16* __restrict__ L, const float* __restrict__ P, __nv_bfloat16* __restrict__ Out) {
    pdl_launch_dependents();
    pdl_wait();
    const int T = TRANSPOSED ? N : K;   // contraction length
    const int C = TRANSPOSED ? K : N;   // output columns
    __shared__ float sIn[SG_BT][SG_BM + 4];
    __shared__ float sW[SG_BT][SG_BC + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * SG_BM, c0 = blockIdx.x * SG_BC;
    const int ty = tid / 16, tx = tid % 16;
    float acc[4][4] = {};

    for (int t0 = 0; t0 < T; t0 += SG_BT) {
        {   // activations: 64 rows x 16 contraction values, 4 consecutive t per thread
            const int mi = tid / 4, tq = (tid % 4) * 4;
            const int m = m0 + mi;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (m < M && t0 + tq < T) {   // T is a multiple of 8, so a group of 4 is all-in or all-out
                const uint2 raw = *reinterpret_cast<const uint2*>(In + (size_t)m * T + t0 + tq);
                v[0] = bf16_lo(raw.x); v[1] = bf16_hi(raw.x); v[2] = bf16_lo(raw.y); v[3] = bf16_hi(raw.y);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) sIn[tq + i][mi] = v[i];
        }
        {   // weights: 16 contraction values x 64 output columns, 4 per thread
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int e = tid + i * 256;
                const int ti = e / 64, ci = e % 64;   // ti: contraction offset, ci: output offset (fastest across threads)
                const int t = t0 + ti, c = c0 + ci;
                float w = 0.f;
                if (t < T && c < C) {
                    const int k = TRANSPOSED ? c : t, n = TRANSPOSED ? t : c;
                    const size_t gi = (size_t)(k / g) * N + n;
                    w = __bfloat162float(dequant_one(load_code(Q, N, bits, k, n), scales[gi], zeros[gi]));
                }
                sW[ti][ci] = w;
            }
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < SG_BT; ++t) {
            const float4 a = *reinterpret_cast<const float4*>(&sIn[t][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&sW[t][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + tx * 4 + j;
            if (c >= C) continue;
            float lo = 0.f;
            for (int q = 0; q < r; ++q) {
                const float l = TRANSPOSED ? __bfloat162float(L[(size_t)q * K + c])    // A[j, k]
                                           : __bfloat162float(L[(size_t)c * r + q]);   // B[n, j]
                lo = fmaf(P[(size_t)m * r + q], l, lo);
            }
            Out[(size_t)m * C + c] = __float2bfloat16_rn(acc[i][j] + s * lo);
        }
    }
}

int launch_simt_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q,
                     const void* scales, const void* zeros, const void* L, const float* P, void* Out,
                     cudaStream_t st) {
    const int C = transposed ? d.K : d.N;
    if (M == 0 || C == 0) return QLORA_OK;
    const float s = d.r > 0 ? d.alpha / (float)d.r : 0.f;
    dim3 grid((C + SG_BC - 1) / SG_BC, (M + SG_BM - 1) / SG_BM);
    cudaError_t err;
    if (transposed)
        err = launch_pdl(simt_gemm_kernel<true>, grid, dim3(256), 0, st, 1, d.bits, d.group_size, d.K, d.N, d.r, s, M,
            (const __nv_bfloat16*)In, (const uint32_t*)Q, (const __half*)scales, (const __half*)zeros,
            (const __nv_bfloat16*)L, P, (__nv_bfloat16*)Out);
    else
        err = launch_pdl(simt_gemm_kernel<false>, grid, dim3(256), 0, st, 1, d.bits, d.group_size, d.K, d.N, d.r, s, M,
            (const __nv_bfloat16*)In, (const uint32_t*)Q, (const __half*)scales, (const __half*)zeros,
            (const __nv_bfloat16*)L, P, (__nv_bfloat16*)Out);
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA down-projections: H = X A^T (contraction over K) and G = dY B (contraction over N), fp32 [M, r].
// Skinny products bound by reading the activations once: a block owns 16 token rows (lora_down.cuh has the method).
// ------------------------------------------------------------------------------------------------------------
template <bool L_IS_A, int NT, int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
lora_down_kernel(int M, int T, int r, const __nv_bfloat16* __restrict__ In, const __nv_bfloat16* __restrict__ L,
                 float* __restrict__ P, const uint8_t* __restrict__ mask, float out_scale) {
    __shared__ float red[WARPS * NT * 128];
    pdl_launch_dependents();
    pdl_wait();
    lora_down_rows<L_IS_A, NT>(M, T, r, In, L, P, mask, out_scale, (int)blockIdx.x * 16, WARPS, red);
}

int launch_lora_down(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st,
                     const uint8_t* mask, float out_scale) {
    if (M == 0 || r == 0) return QLORA_OK;
    // Many rows, low rank: the streaming kernel (also the form that runs inside the CTA-pair kernel, so H / G have the
    // same bits whichever call produced them).
    if (mask == nullptr && out_scale == 1.0f && M > 256 && r <= 16) return launch_lora_down_stream(M, T, r, l_is_A, In, L, P, st);
    const unsigned grid = (unsigned)((M + 15) / 16);
    const __nv_bfloat16* in = (const __nv_bfloat16*)In;
    const __nv_bfloat16* l = (const __nv_bfloat16*)L;
    const int nt = (r + 7) / 8;
    cudaError_t err = cudaSuccess;
#define QLORA_LD(NTV, W)                                                                              \
    do {                                                                                              \
        if (l_is_A) err = launch_pdl(lora_down_kernel<true, NTV, W>, dim3(grid), dim3(W * 32), 0, st, 1, M, T, r, in, l, P, mask, out_scale);   \
        else        err = launch_pdl(lora_down_kernel<false, NTV, W>, dim3(grid), dim3(W * 32), 0, st, 1, M, T, r, in, l, P, mask, out_scale);  \
    } while (0)
    if (nt <= 1) QLORA_LD(1, 32);
    else if (nt <= 2) QLORA_LD(2, 32);
    else if (nt <= 4) QLORA_LD(4, 8);
    else QLORA_LD(8, 8);
#undef QLORA_LD
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA gradients: Out(c, j) = s * sum_m In[m, c] * P[m, j]   (dB: In = dY, P = H, C = N;  dA: In = X, P = G, C = K).
// Bound by reading X and dY once.  Pass 1 (one launch for both gradients): a block owns 256 columns and one slice of
// the token rows; a warp owns 32 of the columns and runs mma.sync m16n8k16 with the ranks as the MMA's M side:
//   D[j, c] += sum_m P^T[j, m] In[m, c]
// The P^T fragments come from a bf16 copy of the slice's P rows staged (transposed) in shared memory; the In fragments
// need pairs of consecutive m for a fixed column, so the 16-byte row loads (8 columns per lane) are transposed across
// the warp with movmatrix.  This permutes which column each accumulator element belongs to (lane (g, q), tile c,
// element e  <->  column 8q + 2c + e of the warp's 32), which the write-out undoes.  The block writes its tile to
// scratch[slice]; pass 2 adds the slices in index order, scales by s and writes (or adds to) dA / dB.
// Nothing depends on scheduling: the result is bitwise reproducible.
// ------------------------------------------------------------------------------------------------------------
constexpr int LG_COLS = 256;          // columns per block (32 per warp)
constexpr int LG_WARPS = 8;
constexpr int LG_UNROLL = 4;          // 16-row steps whose loads are issued together
constexpr int LG_MAX_SLICES = 64;

struct GradPlan { int slices, rows_per_slice; };

static GradPlan lora_grad_plan(int M, int K, int N) {
    const int col_blocks = (K + LG_COLS - 1) / LG_COLS + (N + LG_COLS - 1) / LG_COLS;
    int slices = (2 * 148) / col_blocks;                         // two blocks fit an SM (registers): aim for one wave of a 148-SM part
    if (slices > LG_MAX_SLICES) slices = LG_MAX_SLICES;
    if (slices < 1) slices = 1;
    int rows = (M + slices - 1) / slices;
    rows = (rows + 63) / 64 * 64;                                // whole 16-row MMA steps; keeps the staged P^T conflict-free
    if (rows < 64) rows = 64;
    if (rows > 1024) rows = 1024;                                // bounds the staged P^T (64 ranks x 1032 x 2 B = 129 KiB at most)
    GradPlan g;
    g.rows_per_slice = rows;
    g.slices = M > 0 ? (M + rows - 1) / rows : 1;
    return g;
}

size_t lora_grad_scratch_bytes(int M, int K, int N, int r) {
    return (size_t)lora_grad_plan(M, K, N).slices * (size_t)(K + N) * (size_t)r * sizeof(float);
}

struct GradSide {
    const __nv_bfloat16* In;   // [M, C]
    const float* P;            // [M, r]
    float* partial;            // [slices][C][r]
    float* Out;
    int C;
    const uint8_t* mask;       // [M, C] dropout mask on In (non-zero = keep), or NULL
    float scale;               // s (times the dropout keep scale on the masked side)
    int out_is_dB;             // Out is dB [C, r] (else dA [r, C])
};

// thread-block cluster helpers of the one-launch form below
__device__ __forceinline__ uint32_t lg_map_to_cta(const void* smem_ptr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((uint32_t)__cvta_generic_to_shared(smem_ptr)), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 lg_ld_cluster_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ void lg_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// CL == 0: grid (column blocks, slices, 2 sides); the block writes its partial tile to scratch for lora_grad_reduce_kernel.
// CL >= 1: one launch does it all.  grid (column blocks * CL, 1, 2 sides) in clusters of CL CTAs along x; the CTAs of a
//   cluster take the CL row slices of one column block, leave their partial tiles in shared memory, and after a cluster
//   barrier CTA i adds them in slice order (distributed shared memory, fixed order) for its 256 / CL columns, scales
//   and writes (or adds to) dA / dB.
template <int RT, int CL>   // rank tiles of 16; cluster width (0 = two-launch form)
__global__ void __launch_bounds__(LG_WARPS * 32)
lora_grad_partial_kernel(int M, int r, int rows_per_slice, GradSide side0, GradSide side1, int accumulate) {
    extern __shared__ __align__(16) uint8_t lg_smem[];
    pdl_launch_dependents();
    pdl_wait();
    __nv_bfloat16* Pt = reinterpret_cast<__nv_bfloat16*>(lg_smem);   // [RT * 16][rows_per_slice + 8]
    const GradSide& sd = blockIdx.z == 0 ? side0 : side1;
    const int C = sd.C;
    const int cb = (CL > 0 ? (int)blockIdx.x / CL : (int)blockIdx.x) * LG_COLS;
    if (cb >= C) return;                                       // (the whole cluster returns: same column block)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const int slice = CL > 0 ? (int)blockIdx.x % CL : (int)blockIdx.y;
    const int m_begin = slice * rows_per_slice;
    const int stride = rows_per_slice + 8;                     // in bf16: (stride / 2) % 32 == 4 -> conflict-free fragment loads
    constexpr int RP = RT * 16;
    // stage P^T (bf16) of this slice: rows beyond M and ranks beyond r are zero
    for (int e = threadIdx.x; e < rows_per_slice * RP; e += LG_WARPS * 32) {
        const int ml = e / RP, j = e % RP;
        const int m = m_begin + ml;
        const float v = (m < M && j < r) ? __ldg(sd.P + (size_t)m * r + j) : 0.f;
        Pt[j * stride + ml] = __float2bfloat16_rn(v);
    }
    __syncthreads();

    const int c0 = cb + warp * 32 + q * 8;                     // this lane loads columns c0 .. c0 + 7
    const bool live = c0 < C;                                  // C is a multiple of 8
    const __nv_bfloat16* src = sd.In + c0;
    float acc[RT][4][4];
#pragma unroll
    for (int rt = 0; rt < RT; ++rt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[rt][c][0] = acc[rt][c][1] = acc[rt][c][2] = acc[rt][c][3] = 0.f;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    const int m_stop = min(M, m_begin + rows_per_slice);
    // two register sets: the loads of the next round of 16-row steps are in flight while this round is transposed and multiplied
    uint4 n0[LG_UNROLL], n1[LG_UNROLL];
    auto load_round = [&](int mm) {
#pragma unroll
        for (int u = 0; u < LG_UNROLL; ++u) {
            const int ma = mm + 16 * u + g, mb = ma + 8;
            n0[u] = (live && ma < m_stop) ? *reinterpret_cast<const uint4*>(src + (size_t)ma * C) : zero4;
            n1[u] = (live && mb < m_stop) ? *reinterpret_cast<const uint4*>(src + (size_t)mb * C) : zero4;
            if (sd.mask != nullptr) {
                if (live && ma < m_stop) n0[u] = mask_eight(n0[u], __ldg(reinterpret_cast<const uint2*>(sd.mask + (size_t)ma * C + c0)));
                if (live && mb < m_stop) n1[u] = mask_eight(n1[u], __ldg(reinterpret_cast<const uint2*>(sd.mask + (size_t)mb * C + c0)));
            }
        }
    };
    load_round(m_begin);
    for (int mm = m_begin; mm < m_stop; mm += 16 * LG_UNROLL) {
        uint4 x0[LG_UNROLL], x1[LG_UNROLL];
#pragma unroll
        for (int u = 0; u < LG_UNROLL; ++u) { x0[u] = n0[u]; x1[u] = n1[u]; }
        if (mm + 16 * LG_UNROLL < m_stop) load_round(mm + 16 * LG_UNROLL);
#pragma unroll
        for (int u = 0; u < LG_UNROLL; ++u) {
            const int ml = mm + 16 * u - m_begin;              // warp-uniform
            if (ml >= rows_per_slice || mm + 16 * u >= m_stop) break;
            uint32_t b0[4], b1[4];
            b0[0] = movmatrix_trans(x0[u].x); b0[1] = movmatrix_trans(x0[u].y);
            b0[2] = movmatrix_trans(x0[u].z); b0[3] = movmatrix_trans(x0[u].w);
            b1[0] = movmatrix_trans(x1[u].x); b1[1] = movmatrix_trans(x1[u].y);
            b1[2] = movmatrix_trans(x1[u].z); b1[3] = movmatrix_trans(x1[u].w);
#pragma unroll
            for (int rt = 0; rt < RT; ++rt) {
                const __nv_bfloat16* pa = Pt + (rt * 16 + g) * stride + ml + 2 * q;
                const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa);
                const uint32_t a1 = *reinterpret_cast<const uint32_t*>(pa + 8 * stride);
                const uint32_t a2 = *reinterpret_cast<const uint32_t*>(pa + 8);
                const uint32_t a3 = *reinterpret_cast<const uint32_t*>(pa + 8 * stride + 8);
#pragma unroll
                for (int c = 0; c < 4; ++c) mma_bf16_16816(acc[rt][c], a0, a1, a2, a3, b0[c], b1[c]);
            }
        }
    }
    // accumulator element (rt, c, i): rank rt*16 + g (+8 for i >= 2), column 8q + 2c + (i & 1) of the warp's 32
    if constexpr (CL > 0) {
        __syncthreads();                                       // every warp is done with the staged P^T: the tile takes its place
        float* tile = reinterpret_cast<float*>(lg_smem);       // [256 columns][RP] fp32
#pragma unroll
        for (int rt = 0; rt < RT; ++rt)
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    tile[(warp * 32 + q * 8 + 2 * c + (i & 1)) * RP + rt * 16 + g + ((i & 2) ? 8 : 0)] = acc[rt][c][i];
        __syncthreads();
        lg_cluster_sync();                                     // all CL partial tiles are written
        constexpr int COLS_PER = LG_COLS / CL;
        uint32_t peer[CL];
#pragma unroll
        for (int k = 0; k < CL; ++k) peer[k] = lg_map_to_cta(tile, (uint32_t)k);
        const bool is_dB = sd.out_is_dB != 0;
        for (int e = threadIdx.x; e < COLS_PER * (RP / 4); e += LG_WARPS * 32) {
            const int cl = slice * COLS_PER + e / (RP / 4), j = (e % (RP / 4)) * 4;     // column inside the block, first of four ranks
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < CL; ++k) {                     // slice order
                const float4 x = lg_ld_cluster_f32x4(peer[k] + (uint32_t)((cl * RP + j) * 4));
                v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
            }
            const int col = cb + cl;
            if (col >= C || j >= r) continue;                  // r is a multiple of 8: four ranks are all-in or all-out
            v.x *= sd.scale; v.y *= sd.scale; v.z *= sd.scale; v.w *= sd.scale;
            if (is_dB) {                                       // dB [C, r]
                float4* dst = reinterpret_cast<float4*>(sd.Out + (size_t)col * r + j);
                if (accumulate) { const float4 o = *dst; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
                *dst = v;
            } else {                                           // dA [r, C]
                float* dst = sd.Out + (size_t)j * C + col;
                if (accumulate) { v.x += dst[0]; v.y += dst[C]; v.z += dst[2 * (size_t)C]; v.w += dst[3 * (size_t)C]; }
                dst[0] = v.x; dst[C] = v.y; dst[2 * (size_t)C] = v.z; dst[3 * (size_t)C] = v.w;
            }
        }
        lg_cluster_sync();                                     // nobody leaves while a peer may still read its tile
        return;
    }
    float* part = sd.partial + (size_t)slice * C * r;
#pragma unroll
    for (int rt = 0; rt < RT; ++rt)
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = rt * 16 + g + ((i & 2) ? 8 : 0);
                const int col = cb + warp * 32 + q * 8 + 2 * c + (i & 1);
                if (col < C && j < r) part[(size_t)col * r + j] = acc[rt][c][i];
            }
}

__global__ void lora_grad_reduce_kernel(int r, int slices, int accumulate, GradSide dB_side, GradSide dA_side) {
    // elements [0, N*r): dB[n, j]; elements [N*r, N*r + K*r): dA (stored [r, K])
    pdl_launch_dependents();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t nb = (size_t)dB_side.C * r, na = (size_t)dA_side.C * r;
    if (idx >= nb + na) return;
    const bool is_dB = idx < nb;
    const GradSide& sd = is_dB ? dB_side : dA_side;
    const size_t e = is_dB ? idx : idx - nb;          // index into [C][r]
    const size_t step = (size_t)sd.C * r;
    float v = 0.f;
    int sl = 0;
    for (; sl + 4 <= slices; sl += 4) {               // four independent loads in flight, added in slice order
        const float p0 = sd.partial[(size_t)sl * step + e], p1 = sd.partial[(size_t)(sl + 1) * step + e];
        const float p2 = sd.partial[(size_t)(sl + 2) * step + e], p3 = sd.partial[(size_t)(sl + 3) * step + e];
        v = (((v + p0) + p1) + p2) + p3;
    }
    for (; sl < slices; ++sl) v += sd.partial[(size_t)sl * step + e];
    v *= sd.scale;
    const int c = (int)(e / r), j = (int)(e % r);
    float* dst = is_dB ? sd.Out + e : sd.Out + (size_t)j * sd.C + c;
    *dst = accumulate ? (*dst + v) : v;
}

int launch_lora_grads(int M, int K, int N, int r, float s, const void* X, const void* dY, const float* H, const float* G,
                      float* dA, float* dB, int accumulate, void* scratch, cudaStream_t st, const uint8_t* x_mask, float keep_scale,
                      int sides) {
    if (r == 0) return QLORA_OK;
    const bool want_dB = (sides & 1) != 0, want_dA = (sides & 2) != 0;
    if (!want_dB && !want_dA) return QLORA_OK;
    if (M == 0) {   // empty sums: dA = dB = 0 unless accumulating
        if (!accumulate) {
            if (want_dA && cudaMemsetAsync(dA, 0, (size_t)r * K * sizeof(float), st) != cudaSuccess) return QLORA_ERR_CUDA;
            if (want_dB && cudaMemsetAsync(dB, 0, (size_t)N * r * sizeof(float), st) != cudaSuccess) return QLORA_ERR_CUDA;
        }
        return QLORA_OK;
    }
    const int n_sides = (want_dB ? 1 : 0) + (want_dA ? 1 : 0);
    const int cols = want_dB && want_dA ? (N > K ? N : K) : (want_dB ? N : K);
    const int col_blocks = (cols + LG_COLS - 1) / LG_COLS;
    const int rt = (r + 15) / 16;
    cudaError_t err = cudaSuccess;
    // Up to 256 tokens: one launch; the (at most four) 64-row slices of a column block form a cluster and reduce through
    // distributed shared memory.  (With more tokens, clusters of eight slices measured slower than free-floating blocks
    // plus a reduction launch: 19.6 against 13.4 us at 2048 tokens.)
    int cl = 4;
    while (cl > 1 && M <= 64 * (cl / 2)) cl /= 2;
    const int rows_cl = ((M + cl - 1) / cl + 63) / 64 * 64;
    if (M <= 256) {
        GradSide sB{(const __nv_bfloat16*)dY, H, nullptr, dB, N, nullptr, s, 1};
        GradSide sA{(const __nv_bfloat16*)X, G, nullptr, dA, K, x_mask, x_mask ? s * keep_scale : s, 0};
        if (!want_dB) sB = sA;                                  // one side only: it is the first (and only) z-slice of the grid
        const size_t pt_bytes = (size_t)rt * 16 * (rows_cl + 8) * sizeof(__nv_bfloat16), tile_bytes = (size_t)LG_COLS * rt * 16 * sizeof(float);
        const size_t smem = pt_bytes > tile_bytes ? pt_bytes : tile_bytes;
        const dim3 grid((unsigned)(col_blocks * cl), 1, (unsigned)n_sides);
#define QLORA_LGC(RTV, CLV)                                                                                    \
    do {                                                                                                       \
        static SmemLimit limit;                                                                                \
        if (!limit.raise(lora_grad_partial_kernel<RTV, CLV>, (size_t)RTV * 16 * (1024 + 8) * 2)) return QLORA_ERR_CUDA; \
        err = launch_pdl(lora_grad_partial_kernel<RTV, CLV>, grid, dim3(LG_WARPS * 32), smem, st, CLV, M, r, rows_cl, sB, sA, accumulate); \
    } while (0)
#define QLORA_LGC_RT(CLV)                                                                                      \
    switch (rt) {                                                                                              \
        case 1: QLORA_LGC(1, CLV); break;                                                                      \
        case 2: QLORA_LGC(2, CLV); break;                                                                      \
        case 3: QLORA_LGC(3, CLV); break;                                                                      \
        default: QLORA_LGC(4, CLV); break;                                                                     \
    }
        switch (cl) {
            case 4: QLORA_LGC_RT(4); break;
            case 2: QLORA_LGC_RT(2); break;
            default: QLORA_LGC_RT(1); break;
        }
#undef QLORA_LGC_RT
#undef QLORA_LGC
        return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
    }
    // More tokens: partial sums per row slice to scratch, then a reduction launch.
    GradPlan plan = lora_grad_plan(M, K, N);
    if (n_sides == 1) {
        // one gradient only: its column blocks alone would leave most SMs without a block, so the rows are cut finer -- as
        // fine as the scratch sized for both gradients allows
        const size_t room = (size_t)plan.slices * (size_t)(K + N);
        const int C1 = want_dB ? N : K;
        GradPlan one = lora_grad_plan(M, want_dB ? 0 : K, want_dB ? N : 0);
        while ((size_t)one.slices * C1 > room && one.rows_per_slice < 1024) {
            one.rows_per_slice += 64;
            one.slices = (M + one.rows_per_slice - 1) / one.rows_per_slice;
        }
        if ((size_t)one.slices * C1 <= room) plan = one;
    }
    float* part_dB = (float*)scratch;
    float* part_dA = n_sides == 1 ? part_dB : part_dB + (size_t)plan.slices * N * r;   // (alone, it starts at the base)
    GradSide sB{(const __nv_bfloat16*)dY, H, part_dB, dB, N, nullptr, s, 1};
    GradSide sA{(const __nv_bfloat16*)X, G, part_dA, dA, K, x_mask, x_mask ? s * keep_scale : s, 0};
    GradSide none{};                                         // C = 0: no elements for the reduction
    if (!want_dB) sB = sA;
    dim3 grid(col_blocks, plan.slices, (unsigned)n_sides);
    const size_t smem = (size_t)rt * 16 * (plan.rows_per_slice + 8) * sizeof(__nv_bfloat16);
#define QLORA_LG(RTV)                                                                                          \
    do {                                                                                                       \
        static SmemLimit limit;                                                                                \
        if (!limit.raise(lora_grad_partial_kernel<RTV, 0>, (size_t)RTV * 16 * (1024 + 8) * 2)) return QLORA_ERR_CUDA; \
        err = launch_pdl(lora_grad_partial_kernel<RTV, 0>, grid, dim3(LG_WARPS * 32), smem, st, 1, M, r, plan.rows_per_slice, sB, sA, accumulate); \
    } while (0)
    switch (rt) {
        case 1: QLORA_LG(1); break;
        case 2: QLORA_LG(2); break;
        case 3: QLORA_LG(3); break;
        default: QLORA_LG(4); break;
    }
#undef QLORA_LG
    if (err != cudaSuccess) return QLORA_ERR_CUDA;
    const GradSide& rB = want_dB ? sB : none;
    const GradSide& rA = want_dA ? sA : none;
    const size_t total = (size_t)(rB.C + rA.C) * r;
    err = launch_pdl(lora_grad_reduce_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, 1, r, plan.slices, accumulate, rB, rA);
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA dropout, backward through the branch input: dX[m, k] += mask[m, k] * c * sum_j G[m, j] A[j, k]   (c = s * keep scale).
// The tensor-core kernels add the LoRA term inside the accumulator, where a per-element mask cannot be applied, so with
// dropout they run without the branch and this elementwise pass adds the masked term (dX is read and rounded once more).
// One thread = 8 consecutive k of one token row.
// ------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
lora_masked_update_kernel(int M, int K, int r, float c, const float* __restrict__ G, const __nv_bfloat16* __restrict__ A,
                          const uint8_t* __restrict__ mask, __nv_bfloat16* __restrict__ dX) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int kchunks = K / 8;
    if (idx >= (size_t)M * kchunks) return;
    const int m = (int)(idx / kchunks), k = (int)(idx % kchunks) * 8;
    const uint2 mb = __ldg(reinterpret_cast<const uint2*>(mask + (size_t)m * K + k));
    if ((mb.x | mb.y) == 0u) return;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int j = 0; j < r; ++j) {
        const float gj = __ldg(G + (size_t)m * r + j);
        const uint4 av = __ldg(reinterpret_cast<const uint4*>(A + (size_t)j * K + k));
        acc[0] = fmaf(gj, bf16_lo(av.x), acc[0]); acc[1] = fmaf(gj, bf16_hi(av.x), acc[1]);
        acc[2] = fmaf(gj, bf16_lo(av.y), acc[2]); acc[3] = fmaf(gj, bf16_hi(av.y), acc[3]);
        acc[4] = fmaf(gj, bf16_lo(av.z), acc[4]); acc[5] = fmaf(gj, bf16_hi(av.z), acc[5]);
        acc[6] = fmaf(gj, bf16_lo(av.w), acc[6]); acc[7] = fmaf(gj, bf16_hi(av.w), acc[7]);
    }
    uint4* px = reinterpret_cast<uint4*>(dX + (size_t)m * K + k);
    const uint4 xv = *px;
    const uint32_t xin[4] = {xv.x, xv.y, xv.z, xv.w};
    const uint32_t mbytes[2] = {mb.x, mb.y};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t m2 = mbytes[i >> 1] >> (16 * (i & 1));
        const float lo = bf16_lo(xin[i]) + ((m2 & 0xFFu) ? c * acc[2 * i] : 0.f);
        const float hi = bf16_hi(xin[i]) + ((m2 & 0xFF00u) ? c * acc[2 * i + 1] : 0.f);
        const __nv_bfloat162 pr = __floats2bfloat162_rn(lo, hi);
        o[i] = *reinterpret_cast<const uint32_t*>(&pr);
    }
    *px = make_uint4(o[0], o[1], o[2], o[3]);
}

int launch_lora_masked_update(int M, int K, int r, float c, const float* G, const void* A, const uint8_t* mask, void* dX,
                              cudaStream_t st) {
    if (M == 0 || K == 0 || r == 0) return QLORA_OK;
    const size_t total = (size_t)M * (K / 8);
    const cudaError_t err = launch_pdl(lora_masked_update_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, 1, M, K, r,
                                       c, G, (const __nv_bfloat16*)A, mask, (__nv_bfloat16*)dX);
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
