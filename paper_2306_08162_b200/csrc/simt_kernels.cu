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
// LoRA down-projections: H = X A^T (contraction over K) and G = dY B (contraction over N).  One warp per token row;
// lanes stride over the contraction in 8-element (16-byte) vectors; 8 ranks at a time; warp-shuffle reduction.
// ------------------------------------------------------------------------------------------------------------
template <bool L_IS_A>
__global__ void __launch_bounds__(128)
lora_down_kernel(int M, int T, int r, const __nv_bfloat16* __restrict__ In, const __nv_bfloat16* __restrict__ L,
                 float* __restrict__ P) {
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int m = blockIdx.x * 4 + warp;
    if (m >= M) return;
    const __nv_bfloat16* row = In + (size_t)m * T;
    for (int j0 = 0; j0 < r; j0 += 8) {
        float acc[8] = {};
        for (int t = lane * 8; t < T; t += 256) {
            const uint4 xv = *reinterpret_cast<const uint4*>(row + t);
            const float x[8] = {bf16_lo(xv.x), bf16_hi(xv.x), bf16_lo(xv.y), bf16_hi(xv.y),
                                bf16_lo(xv.z), bf16_hi(xv.z), bf16_lo(xv.w), bf16_hi(xv.w)};
            if (L_IS_A) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {   // A[j0 + j, t .. t+7]
                    const uint4 lv = __ldg(reinterpret_cast<const uint4*>(L + (size_t)(j0 + j) * T + t));
                    acc[j] += x[0] * bf16_lo(lv.x) + x[1] * bf16_hi(lv.x) + x[2] * bf16_lo(lv.y) + x[3] * bf16_hi(lv.y) +
                              x[4] * bf16_lo(lv.z) + x[5] * bf16_hi(lv.z) + x[6] * bf16_lo(lv.w) + x[7] * bf16_hi(lv.w);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {   // B[t + i, j0 .. j0+7]
                    const uint4 lv = __ldg(reinterpret_cast<const uint4*>(L + (size_t)(t + i) * r + j0));
                    acc[0] = fmaf(x[i], bf16_lo(lv.x), acc[0]); acc[1] = fmaf(x[i], bf16_hi(lv.x), acc[1]);
                    acc[2] = fmaf(x[i], bf16_lo(lv.y), acc[2]); acc[3] = fmaf(x[i], bf16_hi(lv.y), acc[3]);
                    acc[4] = fmaf(x[i], bf16_lo(lv.z), acc[4]); acc[5] = fmaf(x[i], bf16_hi(lv.z), acc[5]);
                    acc[6] = fmaf(x[i], bf16_lo(lv.w), acc[6]); acc[7] = fmaf(x[i], bf16_hi(lv.w), acc[7]);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float v = acc[j];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
            acc[j] = v;
        }
        if (lane < 8) {
            float v = acc[0];
#pragma unroll
            for (int j = 1; j < 8; ++j) v = (lane == j) ? acc[j] : v;
            P[(size_t)m * r + j0 + lane] = v;
        }
    }
}

int launch_lora_down(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st) {
    if (M == 0 || r == 0) return QLORA_OK;
    const unsigned grid = (unsigned)((M + 3) / 4);
    if (l_is_A) lora_down_kernel<true><<<grid, 128, 0, st>>>(M, T, r, (const __nv_bfloat16*)In, (const __nv_bfloat16*)L, P);
    else        lora_down_kernel<false><<<grid, 128, 0, st>>>(M, T, r, (const __nv_bfloat16*)In, (const __nv_bfloat16*)L, P);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------
// LoRA gradients: Out(c, j) = s * sum_m In[m, c] * P[m, j]   (dB: In = dY, P = H;  dA: In = X, P = G).
// Pass 1: each block owns 256 columns (2 per thread) and one slice of the token rows, keeps 2 x 8 fp32 sums per
// thread per rank chunk and writes them to scratch[slice].  Pass 2 adds the slices in index order, so the result
// does not depend on scheduling.
// ------------------------------------------------------------------------------------------------------------
constexpr int LG_COLS = 256;          // columns per block
constexpr int LG_MAX_SLICES = 64;

static int lora_grad_slices(int M, int C) {
    const int col_blocks = (C + LG_COLS - 1) / LG_COLS;
    int slices = (4 * 148 + col_blocks - 1) / col_blocks;        // aim for ~4 blocks per SM
    const int max_by_rows = (M + 31) / 32;                       // at least 32 rows per slice
    if (slices > max_by_rows) slices = max_by_rows;
    if (slices > LG_MAX_SLICES) slices = LG_MAX_SLICES;
    if (slices < 1) slices = 1;
    return slices;
}

size_t lora_grad_scratch_bytes(int M, int C, int r) {
    return (size_t)lora_grad_slices(M, C) * (size_t)C * (size_t)r * sizeof(float);
}

__global__ void __launch_bounds__(128)
lora_grad_partial_kernel(int M, int C, int r, int rows_per_slice, const __nv_bfloat16* __restrict__ In,
                         const float* __restrict__ P, float* __restrict__ partial) {
    const int c = blockIdx.x * LG_COLS + threadIdx.x * 2;
    const int slice = blockIdx.y;
    const int m_begin = slice * rows_per_slice;
    const int m_end = min(M, m_begin + rows_per_slice);
    const bool live = c < C;                                       // C is even
    float* out = partial + ((size_t)slice * C + c) * r;            // [slice][c][j]
    for (int j0 = 0; j0 < r; j0 += 8) {
        float a0[8] = {}, a1[8] = {};
        if (live) {
            for (int m = m_begin; m < m_end; ++m) {
                const uint32_t xv = *reinterpret_cast<const uint32_t*>(In + (size_t)m * C + c);
                const float x0 = bf16_lo(xv), x1 = bf16_hi(xv);
                const float4 p0 = __ldg(reinterpret_cast<const float4*>(P + (size_t)m * r + j0));
                const float4 p1 = __ldg(reinterpret_cast<const float4*>(P + (size_t)m * r + j0 + 4));
                const float p[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) { a0[j] = fmaf(x0, p[j], a0[j]); a1[j] = fmaf(x1, p[j], a1[j]); }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) { out[j0 + j] = a0[j]; out[r + j0 + j] = a1[j]; }
        }
    }
}

__global__ void lora_grad_reduce_kernel(int C, int r, int slices, float s, int out_is_dB, int accumulate,
                                        const float* __restrict__ partial, float* __restrict__ Out) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // index into [C][r]
    if (idx >= (size_t)C * r) return;
    float v = 0.f;
    for (int sl = 0; sl < slices; ++sl) v += partial[(size_t)sl * C * r + idx];
    v *= s;
    const int c = (int)(idx / r), j = (int)(idx % r);
    float* dst = out_is_dB ? Out + idx : Out + (size_t)j * C + c;
    *dst = accumulate ? (*dst + v) : v;
}

int launch_lora_grad(int M, int C, int r, float s, bool out_is_dB, const void* In, const float* P, float* Out,
                     int accumulate, void* scratch, cudaStream_t st) {
    if (r == 0 || C == 0) return QLORA_OK;
    const size_t total = (size_t)C * r;
    if (M == 0) {   // empty sum: dA = dB = 0 unless accumulating
        if (!accumulate && cudaMemsetAsync(Out, 0, total * sizeof(float), st) != cudaSuccess) return QLORA_ERR_CUDA;
        return QLORA_OK;
    }
    const int slices = lora_grad_slices(M, C);
    const int rows_per_slice = (M + slices - 1) / slices;
    dim3 grid((C + LG_COLS - 1) / LG_COLS, slices);
    lora_grad_partial_kernel<<<grid, 128, 0, st>>>(M, C, r, rows_per_slice, (const __nv_bfloat16*)In, P, (float*)scratch);
    if (cudaGetLastError() != cudaSuccess) return QLORA_ERR_CUDA;
    lora_grad_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(C, r, slices, s, out_is_dB ? 1 : 0,
                                                                              accumulate, (const float*)scratch, Out);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
