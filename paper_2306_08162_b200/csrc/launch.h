// Host-side launch functions of the individual kernels (internal; the public boundary is include/qlora.h).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "qlora.h"

namespace qlora {

// format_kernels.cu
int launch_pack(int bits, int K, int N, const uint8_t* codes, int32_t* Q, cudaStream_t st);
int launch_unpack(int bits, int K, int N, const int32_t* Q, uint8_t* codes, cudaStream_t st);
int launch_gather_columns(int elem_bytes, int rows, int cols, const void* in, const int32_t* perm, void* out, cudaStream_t st);
int launch_dequant(const qlora_desc& d, const int32_t* Q, const void* scales, const void* zeros, void* W,
                   cudaStream_t st);
int launch_quantize_rtn(const qlora_desc& d, const float* W, int32_t* Q, void* scales, void* zeros, cudaStream_t st);

// loss_kernel.cu -- fused KL + cross-entropy loss and its gradient over [T, V] logits (V % 8 == 0, V <= 32768)
int launch_lrec_loss(int T, int V, const void* Z, const void* Tt, const int32_t* labels, float lambda_kl, float lambda_ce,
                     float grad_scale, float* loss_tokens, void* dZ, cudaStream_t st);

// simt_kernels.cu -- CUDA-core kernels, correct for every supported shape
// In [M, T] bf16 times the dequantised weight, plus s * P L.  transposed = false: forward (T = K, C = N);
// true: backward-input (T = N, C = K).  P fp32 [M, r] (H or G) may be NULL when r == 0.
int launch_simt_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q,
                     const void* scales, const void* zeros, const void* L, const float* P, void* Out,
                     cudaStream_t st);
// P[m, j] = sum_t In[m, t] * L(j, t);  l_is_A: L = A [r, K] (t = k) else L = B [N, r] (t = n).
// mask (optional, only with l_is_A): uint8 [M, T] dropout mask on In, non-zero = keep; the result is multiplied by out_scale.
int launch_lora_down(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st,
                     const uint8_t* mask = nullptr, float out_scale = 1.0f);
// umma_kernel.cu -- the same product for many rows and r <= 16: activations streamed through shared memory by bulk
// copies (launch_lora_down routes there above 256 rows; the CTA-pair kernel runs the same code on idle SM pairs).
int launch_lora_down_stream(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st);
// dB = s dY^T H [N, r] and dA = s G^T X [r, K] in one pair of launches (partial sums per row slice, then a fixed-order
// reduction); scratch needs lora_grad_scratch_bytes().
size_t lora_grad_scratch_bytes(int M, int K, int N, int r);
// sides: 1 = dB only, 2 = dA only, 3 = both (the tensors of a side that is left out may be NULL)
int launch_lora_grads(int M, int K, int N, int r, float s, const void* X, const void* dY, const float* H, const float* G,
                      float* dA, float* dB, int accumulate, void* scratch, cudaStream_t st, const uint8_t* x_mask = nullptr,
                      float keep_scale = 1.0f, int sides = 3);
// dX[m, k] += mask[m, k] * c * sum_j G[m, j] A[j, k]: the LoRA term of the backward pass under dropout.
int launch_lora_masked_update(int M, int K, int r, float c, const float* G, const void* A, const uint8_t* mask, void* dX,
                              cudaStream_t st);

// umma_kernel.cu -- tcgen05 tensor-core kernel (both directions); same contract as launch_simt_gemm
// Ldown == NULL: P is an input.  Ldown != NULL (the adapter applied first: A forward, B backward): P is an output,
// computed on the way -- by SM pairs the tiles of the CTA-pair kernel leave idle when there are some (they signal the
// tiles through the two counters at `sync`, device memory the caller owns: the layer calls carve them out of their
// workspace, so calls that may overlap in time have different ones), otherwise by a down-projection launch ahead of it.
bool umma_supported(const qlora_desc& d, int M);
// dB = s dY^T H as a by-product of the backward call: the producer clusters of the CTA-pair kernel stream every row of dY
// to form G, and the same pass gives dB (ranks up to 8).  `part`: workspace for one [N, r] fp32 part per producer CTA.
// `done` is set when the launch took it on; otherwise dB is still to be computed by the caller.
struct DbFuse {
    const float* H;
    float* dB;
    int accumulate;
    float* part;
    size_t part_bytes;
    bool done;
};
// Workspace bytes with which any backward call of this shape can take dB on (0: none can).
size_t umma_db_part_bytes(const qlora_desc& d, int M);
// The number of producer pairs on which such a call, given its whole workspace, forms dB on the current device; else 0.
int umma_db_on_producers(const qlora_desc& d, int M);
int launch_umma_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q,
                     const void* scales, const void* zeros, const void* L, float* P, void* Out,
                     cudaStream_t st, const void* Ldown = nullptr, unsigned int* sync = nullptr, void* split_buf = nullptr,
                     size_t split_bytes = 0, DbFuse* db = nullptr);
// Bytes of workspace (`split_buf`) with which the CTA-pair kernel splits the tiles of a partly filled last wave along the
// contraction (two SM pairs per tile, exchanging halves of the result); 0 when it would not.  Needs `sync` as well.
size_t umma_split_scratch_bytes(const qlora_desc& d, int M);
// api.cu -- the workspace a layer call needs at least (qlora_workspace_bytes less the optional exchange area above)
size_t required_workspace_bytes(const qlora_desc& d, int M);
// stream_kernel.cu -- few tokens (M <= 16): cp.async-fed mma.sync kernels on raw codes, the contraction split over a
// cluster.  Ldown / Lup: the adapter applied first / second (forward A, B; backward B, A).  P = H or G, fp32 [M, r]: read
// when p_is_input, otherwise computed inside the kernel (ranks up to 16) and written out.
bool stream_supported(const qlora_desc& d, int M, bool transposed);
int launch_stream_gemm(const qlora_desc& d, int M, bool transposed, const void* In, const int32_t* Q, const void* scales,
                       const void* zeros, const void* Ldown, const void* Lup, float* P, bool p_is_input, void* Out,
                       cudaStream_t st);
int read_device_status(unsigned int* out, int clear);
int launch_wait_probe(int limit_us, cudaStream_t st);   // a wait that is known to run out after limit_us (self-test)

}  // namespace qlora
