// LoRA down-projection of one block of 16 token rows, as a device function shared by the stand-alone kernel
// (simt_kernels.cu) and by the CTA-pair tensor-core kernel, whose idle SM pairs run it beside the main tiles.
//   P[m, j] = out_scale * sum_t In[m, t] * L(j, t)     l_is_A: L = A [r, T] (contraction-contiguous), else L = B [T, r].
// mma.sync m16n8k16 (bf16 in, fp32 accumulate) fed straight from 16-byte row loads: the warps of the block stride over
// the contraction in steps of 32 and keep LD_UNROLL steps of loads in flight.  The 32 contraction indices of a step are
// assigned to the fragments in a permuted order (lane q of a quad owns indices 8q..8q+7); activation and adapter fragments
// use the same permutation, so the sum is unchanged.  A is contraction-contiguous and loads directly; B is rank-contiguous,
// so its 8 x 8 fragment tiles are loaded row-wise and transposed across the warp with movmatrix.  The per-warp partial
// tiles are added in warp order through shared memory (fixed order: deterministic for a given number of warps).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace qlora {

constexpr int LD_UNROLL = 4;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// LoRA dropout: keep the bf16 pair elements whose mask byte is non-zero (mask bytes m0, m1 in the low two bytes of `mb`).
__device__ __forceinline__ uint32_t mask_pair(uint32_t pair, uint32_t mb) {
    return pair & (((mb & 0xFFu) ? 0x0000FFFFu : 0u) | ((mb & 0xFF00u) ? 0xFFFF0000u : 0u));
}
// Eight bf16 (uint4) against eight mask bytes (uint2).
__device__ __forceinline__ uint4 mask_eight(uint4 x, uint2 m) {
    return make_uint4(mask_pair(x.x, m.x), mask_pair(x.y, m.x >> 16), mask_pair(x.z, m.y), mask_pair(x.w, m.y >> 16));
}
// Transpose an 8 x 8 matrix of 16-bit elements held across the warp (lane l: row l / 4, elements 2 (l % 4), +1).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// Rows m_base .. m_base + 15.  Called by all `nwarps` warps of a block (it synchronises the block twice);
// `red` is shared memory for nwarps * NT * 128 floats.  In and L are read through the read-only path.
template <bool L_IS_A, int NT>
__device__ __forceinline__ void lora_down_rows(int M, int T, int r, const __nv_bfloat16* __restrict__ In,
                                               const __nv_bfloat16* __restrict__ L, float* __restrict__ P,
                                               const uint8_t* __restrict__ mask, float out_scale, int m_base, int nwarps,
                                               float* red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const int r0 = m_base + g, r1 = r0 + 8;
    const __nv_bfloat16* row0 = In + (size_t)r0 * T;
    const __nv_bfloat16* row1 = In + (size_t)r1 * T;
    const bool v0 = r0 < M, v1 = r1 < M;
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    const int wstride = nwarps * 32;
    for (int kk = warp * 32; kk < T; kk += wstride * LD_UNROLL) {
        uint4 xlo[LD_UNROLL], xhi[LD_UNROLL];
#pragma unroll
        for (int u = 0; u < LD_UNROLL; ++u) {                 // all activation loads of the unrolled steps first
            const int k = kk + u * wstride + q * 8;            // T is a multiple of 8: 8 elements are all-in or all-out
            xlo[u] = (v0 && k < T) ? __ldg(reinterpret_cast<const uint4*>(row0 + k)) : zero4;
            xhi[u] = (v1 && k < T) ? __ldg(reinterpret_cast<const uint4*>(row1 + k)) : zero4;
            if (mask != nullptr) {   // dropout on the branch input: dropped elements contribute nothing
                if (v0 && k < T) xlo[u] = mask_eight(xlo[u], __ldg(reinterpret_cast<const uint2*>(mask + (size_t)r0 * T + k)));
                if (v1 && k < T) xhi[u] = mask_eight(xhi[u], __ldg(reinterpret_cast<const uint2*>(mask + (size_t)r1 * T + k)));
            }
        }
#pragma unroll
        for (int u = 0; u < LD_UNROLL; ++u) {
            const int k0 = kk + u * wstride;                   // warp-uniform
            if (k0 >= T) break;
            const int k = k0 + q * 8;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                uint4 lv = zero4;
                if (L_IS_A) {
                    const int j = nt * 8 + g;                  // rank index of this lane's adapter fragment
                    if (k < T && j < r) lv = __ldg(reinterpret_cast<const uint4*>(L + (size_t)j * T + k));   // A[j, k..k+7]
                } else {
                    // tile t: row rho (0..7) <-> n = k0 + 8 (rho / 2) + (rho % 2) + 2 t, columns = ranks 8 nt .. 8 nt + 7;
                    // after the transpose lane (g, q) holds B[k0 + 8q + 2t, 8nt + g], B[k0 + 8q + 2t + 1, 8nt + g]
                    uint32_t w[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int n = k0 + 8 * (g >> 1) + (g & 1) + 2 * t;
                        uint32_t v = 0;
                        if (n < T && nt * 8 < r) v = __ldg(reinterpret_cast<const uint32_t*>(L + (size_t)n * r + nt * 8 + 2 * q));
                        w[t] = movmatrix_trans(v);
                    }
                    lv = make_uint4(w[0], w[1], w[2], w[3]);
                }
                mma_bf16_16816(acc[nt], xlo[u].x, xhi[u].x, xlo[u].y, xhi[u].y, lv.x, lv.y);
                mma_bf16_16816(acc[nt], xlo[u].z, xhi[u].z, xlo[u].w, xhi[u].w, lv.z, lv.w);
            }
        }
    }
    // red[warp][nt][c][lane]
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[((warp * NT + nt) * 4 + c) * 32 + lane] = acc[nt][c];
    __syncthreads();
    for (int idx = threadIdx.x; idx < NT * 128; idx += wstride) {
        const int nt = idx >> 7, c = (idx >> 5) & 3, ln = idx & 31;
        float v = 0.f;
        for (int w = 0; w < nwarps; ++w) v += red[((w * NT + nt) * 4 + c) * 32 + ln];
        const int row = m_base + (ln >> 2) + ((c & 2) ? 8 : 0);
        const int col = nt * 8 + (ln & 3) * 2 + (c & 1);
        if (row < M && col < r) P[(size_t)row * r + col] = v * out_scale;
    }
    __syncthreads();   // `red` may be rewritten by the next call
}

}  // namespace qlora
