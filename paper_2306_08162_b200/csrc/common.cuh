// Device-side helpers shared by the kernels of the quantized-linear + LoRA library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qlora.h"

namespace qlora {

// One code of the packed matrix, read through the bit-stream definition of the format: code k of column n sits at
// stream bits [k*bits, k*bits+bits); only the 3-bit format can straddle two words (codes 10 and 21 of a block).
__device__ __forceinline__ uint32_t load_code(const uint32_t* __restrict__ Q, int N, int bits, int k, int n) {
    const uint32_t bitpos = (uint32_t)k * (uint32_t)bits;
    const uint32_t row = bitpos >> 5, sh = bitpos & 31u;
    uint32_t v = __ldg(Q + (size_t)row * N + n) >> sh;
    if (sh + (uint32_t)bits > 32u) v |= __ldg(Q + (size_t)(row + 1) * N + n) << (32u - sh);
    return v & ((1u << bits) - 1u);
}

// Canonical weight: one nearest-even rounding to bf16 of the exact fp32 product scale * (q - zero).
__device__ __forceinline__ __nv_bfloat16 dequant_one(uint32_t q, __half scale, __half zero) {
    const float d = (float)((int)q - (int)__half2float(zero));
    return __float2bfloat16_rn(__half2float(scale) * d);
}

// Programmatic dependent launch.  Every layer kernel is launched with the programmatic-stream-serialization attribute:
// it may be scheduled while its predecessor in the stream is still running, does its own set-up (barriers, tensor memory,
// descriptor fetches), and then blocks in pdl_wait() until the predecessor has completed and its writes are visible.
// Nothing may read or write global memory before pdl_wait().  pdl_launch_dependents() at the top lets the successor be
// scheduled as soon as every CTA of this grid has started.  This hides the launch latency between the kernels of a step.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

// ------------------------------------------------------------------------------------------------------------
// dequant32: 32 consecutive-k codes of one output column (BITS packed words) -> 16 registers of bf16 pairs
// (register i holds k = 2i in its low half and k = 2i+1 in its high half), each value the canonical
// bf16_rne(fp32(scale) * (q - zero)).  Used by the tensor-core kernel and by the qlora_dequant utility, so the
// bit-exact check of the utility covers what the tensor cores are fed.
//
// 2- and 4-bit path (packed bf16x2 arithmetic, about 3 instructions per weight).  Write the fp16 scale as
// s = s_hi + s_lo with s_hi its top 8 significant bits (a bf16) and s_lo the remaining <= 3 bits (also a bf16).
// The code is ORed into the mantissa of the bf16 constant 128 (ulp 1), so u = 128 + q and d = u - (128 + zero) = q - zero
// exactly.  |d| <= 15 has <= 4 significant bits, hence p = s_lo * d (<= 7 bits) is exact in bf16, s_hi * d (<= 12 bits)
// is exact inside the fused multiply-add, and fma(s_hi, d, p) rounds the exact value s * d once, to nearest even.
// 3- and 8-bit path: the code is ORed into the mantissa of the fp32 constant 2^23, 2^23 + zero is subtracted (exact),
// the fp32 product with the scale is exact and the pair is rounded once by the packed convert.
// ------------------------------------------------------------------------------------------------------------
struct GroupParams {
    uint32_t s_hi2, s_lo2, c2;   // bf16x2 constants of the 2/4-bit path
    float scale, bias;           // fp32 constants of the 3/8-bit path: scale, 2^23 + zero
};

__device__ __forceinline__ GroupParams group_params(__half scale, __half zero) {
    GroupParams gp;
    const float sf = __half2float(scale);
    const uint32_t hi = __float_as_uint(sf) & 0xFFFF0000u;
    const uint32_t lo = __float_as_uint(sf - __uint_as_float(hi)) >> 16;      // exact: at most 3 significant bits
    gp.s_hi2 = hi | (hi >> 16);
    gp.s_lo2 = lo | (lo << 16);
    const uint32_t c = 0x4300u | (uint32_t)(int)__half2float(zero);            // bf16(128 + zero), zero < 128
    gp.c2 = c | (c << 16);
    gp.scale = sf;
    gp.bias = 8388608.0f + __half2float(zero);
    return gp;
}

__device__ __forceinline__ uint32_t bf16x2_scale(uint32_t u, const GroupParams& gp) {
    const __nv_bfloat162 d = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&u), *reinterpret_cast<const __nv_bfloat162*>(&gp.c2));
    const __nv_bfloat162 p = __hmul2(d, *reinterpret_cast<const __nv_bfloat162*>(&gp.s_lo2));
    const __nv_bfloat162 v = __hfma2(d, *reinterpret_cast<const __nv_bfloat162*>(&gp.s_hi2), p);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int BITS>
__device__ __forceinline__ void dequant32(const uint32_t (&w)[BITS], const GroupParams& gp, uint32_t (&out)[16]) {
    if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {            // word i: codes k = 8i .. 8i+7
            uint32_t v[4];
#pragma unroll
            for (int t = 0; t < 4; ++t)          // v[t] = (code t, code t+4)
                v[t] = bf16x2_scale(((w[i] >> (4 * t)) & 0x000F000Fu) | 0x43004300u, gp);
            out[4 * i + 0] = __byte_perm(v[0], v[1], 0x5410);   // (c0, c1)
            out[4 * i + 1] = __byte_perm(v[2], v[3], 0x5410);   // (c2, c3)
            out[4 * i + 2] = __byte_perm(v[0], v[1], 0x7632);   // (c4, c5)
            out[4 * i + 3] = __byte_perm(v[2], v[3], 0x7632);   // (c6, c7)
        }
    } else if constexpr (BITS == 2) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {            // word i: codes k = 16i .. 16i+15
            uint32_t v[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)          // v[t] = (code t, code t+8)
                v[t] = bf16x2_scale(((w[i] >> (2 * t)) & 0x00030003u) | 0x43004300u, gp);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                out[8 * i + t] = __byte_perm(v[2 * t], v[2 * t + 1], 0x5410);       // (c_2t, c_2t+1)
                out[8 * i + 4 + t] = __byte_perm(v[2 * t], v[2 * t + 1], 0x7632);   // (c_2t+8, c_2t+9)
            }
        }
    } else {
        constexpr uint32_t mask = (1u << BITS) - 1u;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            float f[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int bitpos = (j + h) * BITS, wi = bitpos >> 5, sh = bitpos & 31;
                uint32_t q = w[wi] >> sh;
                if (sh + BITS > 32) q |= w[(wi + 1) % BITS] << (32 - sh);   // only the 3-bit format straddles words
                q = (q & mask) | 0x4B000000u;
                f[h] = (__uint_as_float(q) - gp.bias) * gp.scale;
            }
            const __nv_bfloat162 pr = __floats2bfloat162_rn(f[0], f[1]);
            out[j / 2] = *reinterpret_cast<const uint32_t*>(&pr);
        }
    }
}

// Host side: launch with the programmatic-stream-serialization attribute (and an optional cluster width).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, unsigned cluster_x,
                              Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    unsigned n = 0;
    attrs[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attrs[n].id = cudaLaunchAttributeClusterDimension;
        attrs[n].val.clusterDim.x = cluster_x; attrs[n].val.clusterDim.y = 1; attrs[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace qlora
