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

__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

}  // namespace qlora
