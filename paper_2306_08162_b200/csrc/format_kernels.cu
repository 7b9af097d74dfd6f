// Pack / unpack / full dequantisation of the bit-packed INT32 weight matrix (Section 3.1 of the paper:
// "bit-packed, compact INT32 datatype matrix").  Integer work, bit-exact by construction.
#include "common.cuh"
#include "launch.h"

namespace qlora {

// One thread builds one packed word: it gathers the (up to 17) codes whose bits fall into stream bits
// [32*row, 32*row+32) of column n.  Consecutive threads own consecutive n, so both the byte reads of codes[k, n]
// and the word writes are coalesced.
__global__ void pack_kernel(int bits, int rows, int N, const uint8_t* __restrict__ codes, uint32_t* __restrict__ Q) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)rows * N) return;
    const int row = (int)(idx / N), n = (int)(idx % N);
    const uint32_t mask = (1u << bits) - 1u;
    const int first_bit = row * 32;
    const int k_first = first_bit / bits;                 // first code with bits in this word
    const int k_last = (first_bit + 31) / bits;           // last one
    uint32_t word = 0;
    for (int k = k_first; k <= k_last; ++k) {
        const uint32_t q = codes[(size_t)k * N + n] & mask;
        const int pos = k * bits - first_bit;             // may be negative (code started in the previous word)
        word |= (pos >= 0) ? (q << pos) : (q >> (-pos));  // bits shifted past 31 fall off
    }
    Q[idx] = word;
}

__global__ void unpack_kernel(int bits, int K, int N, const uint32_t* __restrict__ Q, uint8_t* __restrict__ codes) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    const int k = (int)(idx / N), n = (int)(idx % N);
    codes[idx] = (uint8_t)load_code(Q, N, bits, k, n);
}

// Full dequantisation.  One thread turns the 32 consecutive-k codes of one column (BITS words) into 32 bf16 with the same
// routine the tensor-core kernel uses, and writes them as 64 contiguous bytes of row n of W.
template <int BITS>
__global__ void dequant_kernel(int g, int K, int N, const uint32_t* __restrict__ Q, const __half* __restrict__ scales,
                               const __half* __restrict__ zeros, __nv_bfloat16* __restrict__ W) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int blocks = K / 32;
    if (idx >= (size_t)blocks * N) return;
    const int kb = (int)(idx / N), n = (int)(idx % N);
    uint32_t w[BITS];
#pragma unroll
    for (int i = 0; i < BITS; ++i) w[i] = __ldg(Q + (size_t)(kb * BITS + i) * N + n);
    const size_t gi = (size_t)((kb * 32) / g) * N + n;
    const GroupParams gp = group_params(scales[gi], zeros[gi]);
    uint32_t out[16];
    dequant32<BITS>(w, gp, out);
    uint4* dst = reinterpret_cast<uint4*>(W + (size_t)n * K + (size_t)kb * 32);
#pragma unroll
    for (int c = 0; c < 4; ++c) dst[c] = make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
}

// Column gather out[m, j] = in[m, perm[j]] for 2- or 4-byte elements: the per-call step of the activation-order format
// (Appendix A: GPTQ "activation order" leaves the input features of a group scattered; permuting the packed rows once so
// that groups become contiguous, and gathering the activation columns with the same permutation, gives the same layer).
template <typename T>
__global__ void gather_columns_kernel(int rows, int cols, const T* __restrict__ in, const int32_t* __restrict__ perm, T* __restrict__ out) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)rows * cols) return;
    const int m = (int)(idx / cols), j = (int)(idx % cols);
    out[idx] = in[(size_t)m * cols + __ldg(perm + j)];
}

// Asymmetric min-max round-to-nearest quantizer (the "RTN" of the paper's comparisons, and how the benchmark layers get
// their codes).  A block of 8 warps owns one group index and 32 consecutive output rows n of W [N, K]:
//   1. warp w takes rows 4w .. 4w+3 in turn: its lanes read the group's g weights (coalesced along k), min and max go
//      through shuffles, and every lane derives the same scale / zero-point -- in float32, with IEEE division, the scale
//      rounded to fp16 first and halves rounded to even, so the integers are those of the CPU statement of the method;
//   2. per 32 consecutive k: each warp quantizes its four rows (lane = k) into shared memory, then thread (word i, row n)
//      assembles word i of the 32-code block of row n from the bit-stream definition of the format and stores it;
//      neighbouring threads own neighbouring n, so the word stores are coalesced.
// Integer results: bit-exact by construction.
constexpr int QZ_ROWS = 32;

template <int BITS>
__global__ void __launch_bounds__(256) quantize_rtn_kernel(int g, int K, int N, const float* __restrict__ W, uint32_t* __restrict__ Q,
                                                            __half* __restrict__ scales, __half* __restrict__ zeros) {
    __shared__ float s_scale[QZ_ROWS], s_zero[QZ_ROWS];
    __shared__ uint8_t s_code[QZ_ROWS][36];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gi = blockIdx.y, n0 = blockIdx.x * QZ_ROWS;
    const float qmax = (float)((1 << BITS) - 1);
    for (int j = 0; j < 4; ++j) {
        const int n = n0 + 4 * warp + j;
        float lo = 0.f, hi = 0.f;
        if (n < N) {
            const float* row = W + (size_t)n * K + (size_t)gi * g;
            for (int k = lane; k < g; k += 32) { const float w = row[k]; lo = fminf(lo, w); hi = fmaxf(hi, w); }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o)); hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o)); }
        __half sc16 = __float2half_rn(__fdiv_rn(hi - lo, qmax));
        if (__half2float(sc16) == 0.f) sc16 = __float2half_rn(1.f);
        const float sc = __half2float(sc16);
        const float z = fminf(fmaxf(rintf(__fdiv_rn(-lo, sc)), 0.f), qmax) + 0.f;
        if (lane == 0 && n < N) {
            s_scale[4 * warp + j] = sc; s_zero[4 * warp + j] = z;
            scales[(size_t)gi * N + n] = sc16;
            zeros[(size_t)gi * N + n] = __float2half_rn(z);
        }
    }
    __syncthreads();
    for (int kb = 0; kb < g / 32; ++kb) {
        const int k0 = gi * g + kb * 32;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int r = 4 * warp + j, n = n0 + r;
            uint8_t c = 0;
            if (n < N) {
                const float w = W[(size_t)n * K + k0 + lane];
                c = (uint8_t)fminf(fmaxf(rintf(__fdiv_rn(w, s_scale[r])) + s_zero[r], 0.f), qmax);
            }
            s_code[r][lane] = c;
        }
        __syncthreads();
        if (threadIdx.x < BITS * QZ_ROWS) {
            const int i = threadIdx.x / QZ_ROWS, r = threadIdx.x % QZ_ROWS;   // word i of the block's BITS words, row r
            const int k_first = (32 * i) / BITS, k_last = (32 * i + 31) / BITS;
            uint32_t word = 0;
            for (int k = k_first; k <= k_last; ++k) {
                const uint32_t q = s_code[r][k];
                const int pos = k * BITS - 32 * i;                        // negative: the code started in the previous word
                word |= pos >= 0 ? (q << pos) : (q >> (-pos));
            }
            if (n0 + r < N) Q[(size_t)((k0 / 32) * BITS + i) * N + n0 + r] = word;
        }
        __syncthreads();
    }
}

int launch_quantize_rtn(const qlora_desc& d, const float* W, int32_t* Q, void* scales, void* zeros, cudaStream_t st) {
    if (d.K == 0 || d.N == 0) return QLORA_OK;
    const dim3 grid((unsigned)((d.N + QZ_ROWS - 1) / QZ_ROWS), (unsigned)(d.K / d.group_size));
    uint32_t* q = (uint32_t*)Q;
    __half* s = (__half*)scales;
    __half* z = (__half*)zeros;
    switch (d.bits) {
        case 2: quantize_rtn_kernel<2><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, W, q, s, z); break;
        case 3: quantize_rtn_kernel<3><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, W, q, s, z); break;
        case 4: quantize_rtn_kernel<4><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, W, q, s, z); break;
        case 8: quantize_rtn_kernel<8><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, W, q, s, z); break;
        default: return QLORA_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

int launch_gather_columns(int elem_bytes, int rows, int cols, const void* in, const int32_t* perm, void* out, cudaStream_t st) {
    const size_t total = (size_t)rows * cols;
    if (total == 0) return QLORA_OK;
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (elem_bytes == 2) gather_columns_kernel<uint16_t><<<grid, 256, 0, st>>>(rows, cols, (const uint16_t*)in, perm, (uint16_t*)out);
    else if (elem_bytes == 4) gather_columns_kernel<uint32_t><<<grid, 256, 0, st>>>(rows, cols, (const uint32_t*)in, perm, (uint32_t*)out);
    else return QLORA_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

int launch_pack(int bits, int K, int N, const uint8_t* codes, int32_t* Q, cudaStream_t st) {
    const int rows = K * bits / 32;
    const size_t total = (size_t)rows * N;
    if (total == 0) return QLORA_OK;
    pack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(bits, rows, N, codes, (uint32_t*)Q);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

int launch_unpack(int bits, int K, int N, const int32_t* Q, uint8_t* codes, cudaStream_t st) {
    const size_t total = (size_t)K * N;
    if (total == 0) return QLORA_OK;
    unpack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(bits, K, N, (const uint32_t*)Q, codes);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

int launch_dequant(const qlora_desc& d, const int32_t* Q, const void* scales, const void* zeros, void* W,
                   cudaStream_t st) {
    if (d.K == 0 || d.N == 0) return QLORA_OK;
    const size_t total = (size_t)(d.K / 32) * d.N;
    const unsigned grid = (unsigned)((total + 255) / 256);
    const uint32_t* q = (const uint32_t*)Q;
    const __half* s = (const __half*)scales;
    const __half* z = (const __half*)zeros;
    __nv_bfloat16* w = (__nv_bfloat16*)W;
    switch (d.bits) {
        case 2: dequant_kernel<2><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, q, s, z, w); break;
        case 3: dequant_kernel<3><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, q, s, z, w); break;
        case 4: dequant_kernel<4><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, q, s, z, w); break;
        case 8: dequant_kernel<8><<<grid, 256, 0, st>>>(d.group_size, d.K, d.N, q, s, z, w); break;
        default: return QLORA_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
