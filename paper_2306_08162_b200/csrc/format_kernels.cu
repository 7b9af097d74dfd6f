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

// W[n, k] for a 32(k) x 32(n) tile per block: reads are coalesced along n, the tile is transposed through shared
// memory so that the bf16 writes are coalesced along k.
__global__ void dequant_kernel(int bits, int g, int K, int N, const uint32_t* __restrict__ Q,
                               const __half* __restrict__ scales, const __half* __restrict__ zeros,
                               __nv_bfloat16* __restrict__ W) {
    __shared__ __nv_bfloat16 tile[32][33];
    const int n0 = blockIdx.x * 32, k0 = blockIdx.y * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;          // 32 x 8
    for (int i = ty; i < 32; i += 8) {
        const int k = k0 + i, n = n0 + tx;
        if (n < N) {
            const size_t gi = (size_t)(k / g) * N + n;
            tile[i][tx] = dequant_one(load_code(Q, N, bits, k, n), scales[gi], zeros[gi]);
        }
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int n = n0 + i, k = k0 + tx;
        if (n < N) W[(size_t)n * K + k] = tile[tx][i];
    }
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
    dim3 grid((d.N + 31) / 32, d.K / 32), block(32, 8);
    dequant_kernel<<<grid, block, 0, st>>>(d.bits, d.group_size, d.K, d.N, (const uint32_t*)Q, (const __half*)scales,
                                           (const __half*)zeros, (__nv_bfloat16*)W);
    return cudaGetLastError() == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
