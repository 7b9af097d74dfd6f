// CUDA-core kernels of the quantized-linear + LoRA layer.  They are correct for every shape the library accepts
// and serve (a) shapes the tensor-core kernels do not tile, and (b) the skinny LoRA products, which are bound by
// HBM traffic rather than by arithmetic (Figure 1 of the paper: the green "MM" blocks and their gradients).
#include "common.cuh"
#include "launch.h"

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
                int ti, ci;
                if (TRANSPOSED) { ti = e / 64; ci = e % 64; }   // ti: n offset, ci: k offset (k fastest: same word for 8 lanes)
                else            { ti = e / 64; ci = e % 64; }   // ti: k offset, ci: n offset (n fastest: coalesced words)
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
    if (transposed)
        simt_gemm_kernel<true><<<grid, 256, 0, st>>>(d.bits, d.group_size, d.K, d.N, d.r, s, M,
            (const __nv_bfloat16*)In, (const uint32_t*)Q, (const __half*)scales, (const __half*)zeros,
            (const __nv_bfloat16*)L, P, (__nv_bfloat16*)Out);
    else
        simt_gemm_kernel<false><<<grid, 256, 0, st>>>(d.bits, d.group_size, d.K, d.N, d.r, s, M,
            (const __nv_bfloat16*)In, (const uint32_t*)Q, (const __half*)scales, (const __half*)zeros,
            (const __nv_bfloat16*)L, P, (__nv_bfloat16*)Out);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA down-projections: H = X A^T (contraction over K) and G = dY B (contraction over N), fp32 [M, r].
// Skinny products bound by reading the activations once, so they use the warp-level mma.sync (m16n8k16, bf16 in,
// fp32 accumulate): a block owns 16 token rows, its 8 warps stride over the contraction in steps of 32, and every lane
// feeds the tensor core straight from two 16-byte row loads.  The 32 contraction indices of a step are assigned to the
// fragments in a permuted order (lane q of a quad owns indices 8q..8q+7); activation and adapter fragments use the same
// permutation, so the sum is unchanged.  The 8 per-warp partial tiles are added in warp order through shared memory
// (fixed order: deterministic).
// ------------------------------------------------------------------------------------------------------------
constexpr int LD_WARPS = 8;
constexpr int LD_MAX_NT = 8;   // rank tiles of 8 (r <= 64)

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <bool L_IS_A, int NT>
__global__ void __launch_bounds__(LD_WARPS * 32)
lora_down_kernel(int M, int T, int r, const __nv_bfloat16* __restrict__ In, const __nv_bfloat16* __restrict__ L,
                 float* __restrict__ P) {
    __shared__ float red[LD_WARPS][NT][4][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const int m_base = blockIdx.x * 16;
    const int r0 = m_base + g, r1 = r0 + 8;
    const __nv_bfloat16* row0 = In + (size_t)r0 * T;
    const __nv_bfloat16* row1 = In + (size_t)r1 * T;
    const bool v0 = r0 < M, v1 = r1 < M;
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll 2
    for (int k0 = warp * 32; k0 < T; k0 += LD_WARPS * 32) {
        const int k = k0 + q * 8;
        const bool kin = k < T;                     // T is a multiple of 8
        const uint4 xlo = (v0 && kin) ? *reinterpret_cast<const uint4*>(row0 + k) : zero4;
        const uint4 xhi = (v1 && kin) ? *reinterpret_cast<const uint4*>(row1 + k) : zero4;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int j = nt * 8 + g;               // rank index of this lane's adapter fragment
            uint4 lv = zero4;
            if (kin && j < r) {
                if (L_IS_A) {
                    lv = __ldg(reinterpret_cast<const uint4*>(L + (size_t)j * T + k));            // A[j, k..k+7]
                } else {
                    uint32_t e[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) e[i] = __bfloat16_as_ushort(__ldg(L + (size_t)(k + i) * r + j));   // B[k+i, j]
                    lv = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
                }
            }
            mma_bf16_16816(acc[nt], xlo.x, xhi.x, xlo.y, xhi.y, lv.x, lv.y);
            mma_bf16_16816(acc[nt], xlo.z, xhi.z, xlo.w, xhi.w, lv.z, lv.w);
        }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[warp][nt][c][lane] = acc[nt][c];
    __syncthreads();
    for (int idx = threadIdx.x; idx < NT * 128; idx += LD_WARPS * 32) {
        const int nt = idx >> 7, c = (idx >> 5) & 3, ln = idx & 31;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < LD_WARPS; ++w) v += red[w][nt][c][ln];
        const int row = m_base + (ln >> 2) + ((c & 2) ? 8 : 0);
        const int col = nt * 8 + (ln & 3) * 2 + (c & 1);
        if (row < M && col < r) P[(size_t)row * r + col] = v;
    }
}

int launch_lora_down(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st) {
    if (M == 0 || r == 0) return QLORA_OK;
    const unsigned grid = (unsigned)((M + 15) / 16);
    const __nv_bfloat16* in = (const __nv_bfloat16*)In;
    const __nv_bfloat16* l = (const __nv_bfloat16*)L;
    const int nt = (r + 7) / 8;
#define QLORA_LD(NTV)                                                                                  \
    do {                                                                                               \
        if (l_is_A) lora_down_kernel<true, NTV><<<grid, LD_WARPS * 32, 0, st>>>(M, T, r, in, l, P);   \
        else        lora_down_kernel<false, NTV><<<grid, LD_WARPS * 32, 0, st>>>(M, T, r, in, l, P);  \
    } while (0)
    if (nt <= 1) QLORA_LD(1);
    else if (nt <= 2) QLORA_LD(2);
    else if (nt <= 4) QLORA_LD(4);
    else QLORA_LD(8);
#undef QLORA_LD
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA gradients: Out(c, j) = s * sum_m In[m, c] * P[m, j]   (dB: In = dY, P = H, C = N;  dA: In = X, P = G, C = K).
// Bound by reading X and dY once.  Pass 1 (one launch for both gradients): a block owns 256 columns and one slice of
// the token rows; each lane keeps an 8-column x 8-rank tile of fp32 sums, the block's four warps take interleaved rows
// and are added in warp order through shared memory; the block writes its tile to scratch[slice].  Pass 2 adds the
// slices in index order, scales by s and writes (or adds to) dA / dB.  Nothing depends on scheduling.
// ------------------------------------------------------------------------------------------------------------
constexpr int LG_COLS = 256;          // columns per block (8 per lane)
constexpr int LG_MAX_SLICES = 64;

static int lora_grad_slices(int M, int K, int N) {
    const int col_blocks = (K + LG_COLS - 1) / LG_COLS + (N + LG_COLS - 1) / LG_COLS;
    int slices = (4 * 148 + col_blocks - 1) / col_blocks;        // aim for ~4 blocks per SM
    const int max_by_rows = (M + 31) / 32;                       // at least 32 rows per slice
    if (slices > max_by_rows) slices = max_by_rows;
    if (slices > LG_MAX_SLICES) slices = LG_MAX_SLICES;
    if (slices < 1) slices = 1;
    return slices;
}

size_t lora_grad_scratch_bytes(int M, int K, int N, int r) {
    return (size_t)lora_grad_slices(M, K, N) * (size_t)(K + N) * (size_t)r * sizeof(float);
}

struct GradSide {
    const __nv_bfloat16* In;   // [M, C]
    const float* P;            // [M, r]
    float* partial;            // [slices][C][r]
    float* Out;
    int C;
};

__global__ void __launch_bounds__(128)
lora_grad_partial_kernel(int M, int r, int rows_per_slice, GradSide side0, GradSide side1) {
    __shared__ float red[4][64][32];
    const GradSide& sd = blockIdx.z == 0 ? side0 : side1;
    const int C = sd.C;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cb = blockIdx.x * LG_COLS;
    if (cb >= C) return;
    const int c0 = cb + lane * 8;
    const bool live = c0 < C;                                       // C is a multiple of 8
    const int slice = blockIdx.y;
    const int m_begin = slice * rows_per_slice;
    const int m_end = min(M, m_begin + rows_per_slice);
    for (int j0 = 0; j0 < r; j0 += 8) {
        float acc[8][8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
        if (live) {
#pragma unroll 2
            for (int m = m_begin + warp; m < m_end; m += 4) {
                const uint4 xv = *reinterpret_cast<const uint4*>(sd.In + (size_t)m * C + c0);
                const float4 p0 = __ldg(reinterpret_cast<const float4*>(sd.P + (size_t)m * r + j0));
                const float4 p1 = __ldg(reinterpret_cast<const float4*>(sd.P + (size_t)m * r + j0 + 4));
                const float x[8] = {bf16_lo(xv.x), bf16_hi(xv.x), bf16_lo(xv.y), bf16_hi(xv.y),
                                    bf16_lo(xv.z), bf16_hi(xv.z), bf16_lo(xv.w), bf16_hi(xv.w)};
                const float pj[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(x[i], pj[j], acc[i][j]);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) red[warp][i * 8 + j][lane] = acc[i][j];
        __syncthreads();
        // 64 x 32 sums; thread t adds the four warps' values for 16 of them and writes partial[slice][c][j0 + j]
        for (int e = threadIdx.x; e < 64 * 32; e += 128) {
            const int ij = e >> 5, ln = e & 31;
            const float v = ((red[0][ij][ln] + red[1][ij][ln]) + red[2][ij][ln]) + red[3][ij][ln];
            const int c = cb + ln * 8 + (ij >> 3);
            if (c < C) sd.partial[((size_t)slice * C + c) * r + j0 + (ij & 7)] = v;
        }
        __syncthreads();
    }
}

__global__ void lora_grad_reduce_kernel(int r, int slices, float s, int accumulate, GradSide dB_side, GradSide dA_side) {
    // elements [0, N*r): dB[n, j]; elements [N*r, N*r + K*r): dA (stored [r, K])
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t nb = (size_t)dB_side.C * r, na = (size_t)dA_side.C * r;
    if (idx >= nb + na) return;
    const bool is_dB = idx < nb;
    const GradSide& sd = is_dB ? dB_side : dA_side;
    const size_t e = is_dB ? idx : idx - nb;          // index into [C][r]
    float v = 0.f;
    for (int sl = 0; sl < slices; ++sl) v += sd.partial[(size_t)sl * sd.C * r + e];
    v *= s;
    const int c = (int)(e / r), j = (int)(e % r);
    float* dst = is_dB ? sd.Out + e : sd.Out + (size_t)j * sd.C + c;
    *dst = accumulate ? (*dst + v) : v;
}

int launch_lora_grads(int M, int K, int N, int r, float s, const void* X, const void* dY, const float* H, const float* G,
                      float* dA, float* dB, int accumulate, void* scratch, cudaStream_t st) {
    if (r == 0) return QLORA_OK;
    if (M == 0) {   // empty sums: dA = dB = 0 unless accumulating
        if (!accumulate) {
            if (cudaMemsetAsync(dA, 0, (size_t)r * K * sizeof(float), st) != cudaSuccess) return QLORA_ERR_CUDA;
            if (cudaMemsetAsync(dB, 0, (size_t)N * r * sizeof(float), st) != cudaSuccess) return QLORA_ERR_CUDA;
        }
        return QLORA_OK;
    }
    const int slices = lora_grad_slices(M, K, N);
    const int rows_per_slice = (M + slices - 1) / slices;
    float* part_dB = (float*)scratch;
    float* part_dA = part_dB + (size_t)slices * N * r;
    GradSide sB{(const __nv_bfloat16*)dY, H, part_dB, dB, N};
    GradSide sA{(const __nv_bfloat16*)X, G, part_dA, dA, K};
    const int cols = (N > K ? N : K);
    dim3 grid((cols + LG_COLS - 1) / LG_COLS, slices, 2);
    lora_grad_partial_kernel<<<grid, 128, 0, st>>>(M, r, rows_per_slice, sB, sA);
    if (cudaGetLastError() != cudaSuccess) return QLORA_ERR_CUDA;
    const size_t total = (size_t)(N + K) * r;
    lora_grad_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(r, slices, s, accumulate, sB, sA);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
