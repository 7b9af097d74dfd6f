// Fused LREC training loss (Section 3.2, Eq. 1-2 of the paper): per token, with student logits z (the quantized model with
// its LoRA pairs) and cached teacher logits t (the frozen full-precision model),
//     loss = lambda_KL * KL(softmax(z) || softmax(t)) + lambda_CE * ( -log softmax(z)[label] )
// and its gradient with respect to z, in one pass over the two [T, V] logit matrices:
//     d KL / d z_j = p_j * ((log p_j - log q_j) - KL),      d CE / d z_j = p_j - [j == label]        (p = softmax(z), q = softmax(t))
// Bound by HBM traffic (read 2 * V * 2 bytes, write V * 2 bytes per token), so a token row is read once: a block of 512
// threads holds both rows entirely in registers (up to 8 chunks of 8 bf16 per thread and matrix, V <= 32768), three block-wide
// reductions give the two maxima, the two exp-sums and the KL sum, and the gradient is written from the same registers.
// Exponentials use the hardware ex2 path (relative error ~2^-22 on the arguments <= 0 that occur here) and the KL sum
// shares the exp-sum pass (3 exponentials per logit pair instead of 5): the special-function unit, not memory, was the bound.
// One row fills half an SM's register file, so only one block fits per SM; to keep HBM busy while a row is being reduced,
// every thread prefetches ITS OWN chunks of the block's next row into shared memory with cp.async (thread-private slots:
// no barrier is involved, the thread just waits for its own copies) and moves them to registers when the row's turn comes.
#include "common.cuh"
#include "device_state.h"
#include "launch.h"

namespace qlora {

constexpr int LL_THREADS = 512;

// 2^x on the special-function unit (relative error about 2^-22; results below the normal range flush to zero).
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float u = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = is_max ? fmaxf(v, u) : v + u;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                       // scratch free again
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float r = scratch[0];                  // every thread combines the 16 warp values in the same order: deterministic
#pragma unroll
    for (int w = 1; w < LL_THREADS / 32; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];
    return r;
}

template <int CH>   // 16-byte chunks (8 bf16) per thread and matrix
__global__ void __launch_bounds__(LL_THREADS)
lrec_loss_kernel(int T, int V, const __nv_bfloat16* __restrict__ Z, const __nv_bfloat16* __restrict__ Tt,
                 const int32_t* __restrict__ labels, float lambda_kl, float lambda_ce, float grad_scale,
                 float* __restrict__ loss_tokens, __nv_bfloat16* __restrict__ dZ) {
    __shared__ float scratch[LL_THREADS / 32];
    extern __shared__ __align__(16) uint8_t ll_smem[];          // [2][CH][LL_THREADS] uint4: next row of Z and of Tt
    uint4* stage_z = reinterpret_cast<uint4*>(ll_smem);
    uint4* stage_t = stage_z + CH * LL_THREADS;
    pdl_launch_dependents();
    pdl_wait();
    const int chunks = V / 8;
    auto prefetch = [&](int row) {                              // this thread's chunks of `row` -> its shared-memory slots
        const uint4* zr = reinterpret_cast<const uint4*>(Z + (size_t)row * V);
        const uint4* tr = reinterpret_cast<const uint4*>(Tt + (size_t)row * V);
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int ci = c * LL_THREADS + threadIdx.x;
            if (ci < chunks) {
                const uint32_t dz = (uint32_t)__cvta_generic_to_shared(stage_z + ci), dt = (uint32_t)__cvta_generic_to_shared(stage_t + ci);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dz), "l"(zr + ci) : "memory");
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dt), "l"(tr + ci) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if ((int)blockIdx.x < T) prefetch(blockIdx.x);
    for (int row = blockIdx.x; row < T; row += gridDim.x) {
        uint4 zc[CH], tc[CH];
        const uint4 neg = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // bf16 -inf pairs: padding
        asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int ci = c * LL_THREADS + threadIdx.x;
            zc[c] = ci < chunks ? stage_z[ci] : neg;
            tc[c] = ci < chunks ? stage_t[ci] : neg;
        }
        if (row + (int)gridDim.x < T) prefetch(row + gridDim.x);   // overlaps the reductions and the stores below
        float mz = -INFINITY, mt = -INFINITY;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const uint32_t zw[4] = {zc[c].x, zc[c].y, zc[c].z, zc[c].w}, tw[4] = {tc[c].x, tc[c].y, tc[c].z, tc[c].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                mz = fmaxf(mz, fmaxf(bf16_lo(zw[i]), bf16_hi(zw[i])));
                mt = fmaxf(mt, fmaxf(bf16_lo(tw[i]), bf16_hi(tw[i])));
            }
        }
        mz = block_reduce(mz, true, scratch);
        mt = block_reduce(mt, true, scratch);
        // One pass gives both exp-sums and the KL numerator: with e_j = exp(z_j - mz) and sz = sum e_j,
        //   KL = sum_j (e_j / sz) ((z_j - lz) - (t_j - lt)) = (sum_j e_j (z_j - t_j)) / sz - lz + lt        (lz = mz + log sz, ...)
        // (padding: z = t = -inf would give 0 * nan, so padded chunks are skipped rather than relied on to vanish)
        constexpr float kLog2e = 1.4426950408889634f;
        const float mz2 = mz * kLog2e, mt2 = mt * kLog2e;
        float sz = 0.f, st = 0.f, az = 0.f;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int ci = c * LL_THREADS + threadIdx.x;
            if (ci < chunks) {
                const uint32_t zw[4] = {zc[c].x, zc[c].y, zc[c].z, zc[c].w}, tw[4] = {tc[c].x, tc[c].y, tc[c].z, tc[c].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float z0 = bf16_lo(zw[i]), z1 = bf16_hi(zw[i]), t0 = bf16_lo(tw[i]), t1 = bf16_hi(tw[i]);
                    const float e0 = fast_exp2(fmaf(z0, kLog2e, -mz2)), e1 = fast_exp2(fmaf(z1, kLog2e, -mz2));
                    sz += e0 + e1;
                    az = fmaf(e0, z0 - t0, fmaf(e1, z1 - t1, az));
                    st += fast_exp2(fmaf(t0, kLog2e, -mt2)) + fast_exp2(fmaf(t1, kLog2e, -mt2));
                }
            }
        }
        sz = block_reduce(sz, false, scratch);
        st = block_reduce(st, false, scratch);
        az = block_reduce(az, false, scratch);
        const float lz = mz + logf(sz), lt = mt + logf(st);       // log-partition functions: log p_j = z_j - lz
        const float kl = az / sz - lz + lt;
        const int label = labels != nullptr ? __ldg(labels + row) : -1;
        const bool has_label = label >= 0 && label < V;
        if (threadIdx.x == 0) {
            float ce = 0.f;
            if (has_label) ce = lz - __bfloat162float(Z[(size_t)row * V + label]);   // -log p_label
            loss_tokens[row] = lambda_kl * kl + lambda_ce * ce;
        }
        if (dZ != nullptr) {
            uint4* dr = reinterpret_cast<uint4*>(dZ + (size_t)row * V);
            const float shift = (lz - lt) + kl, ce_w = has_label ? lambda_ce : 0.f;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int ci = c * LL_THREADS + threadIdx.x;
                if (ci < chunks) {
                    const uint32_t zw[4] = {zc[c].x, zc[c].y, zc[c].z, zc[c].w}, tw[4] = {tc[c].x, tc[c].y, tc[c].z, tc[c].w};
                    uint32_t o[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float gsum[2];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            // g_j = p_j (lambda_kl ((z_j - t_j) - (lz - lt) - KL) + lambda_ce) - lambda_ce [j == label]
                            const float z = h ? bf16_hi(zw[i]) : bf16_lo(zw[i]), t = h ? bf16_hi(tw[i]) : bf16_lo(tw[i]);
                            const float pj = fast_exp2(fmaf(z, kLog2e, -lz * kLog2e));
                            float gr = pj * fmaf(lambda_kl, (z - t) - shift, ce_w);
                            if (has_label && (ci * 8 + 2 * i + h) == label) gr -= lambda_ce;
                            gsum[h] = grad_scale * gr;
                        }
                        const __nv_bfloat162 pr = __floats2bfloat162_rn(gsum[0], gsum[1]);
                        o[i] = *reinterpret_cast<const uint32_t*>(&pr);
                    }
                    dr[ci] = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    }
}

int launch_lrec_loss(int T, int V, const void* Z, const void* Tt, const int32_t* labels, float lambda_kl, float lambda_ce,
                     float grad_scale, float* loss_tokens, void* dZ, cudaStream_t st) {
    if (T == 0) return QLORA_OK;
    const int chunks = V / 8;
    const int ch = (chunks + LL_THREADS - 1) / LL_THREADS;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(T < sms ? T : sms);   // one block per SM (registers), persistent over the rows
    cudaError_t err;
#define QLORA_LL(CHV)                                                                                                  \
    {                                                                                                                  \
        static SmemLimit limit;                                                                                        \
        if (!limit.raise(lrec_loss_kernel<CHV>, (size_t)2 * CHV * LL_THREADS * 16)) return QLORA_ERR_CUDA;             \
    }                                                                                                                  \
    err = launch_pdl(lrec_loss_kernel<CHV>, dim3(grid), dim3(LL_THREADS), (size_t)2 * CHV * LL_THREADS * 16, st, 1, T, V, (const __nv_bfloat16*)Z, \
                     (const __nv_bfloat16*)Tt, labels, lambda_kl, lambda_ce, grad_scale, loss_tokens, (__nv_bfloat16*)dZ)
    if (ch <= 1) { QLORA_LL(1); }
    else if (ch <= 2) { QLORA_LL(2); }
    else if (ch <= 4) { QLORA_LL(4); }
    else if (ch <= 8) { QLORA_LL(8); }
    else return QLORA_ERR_UNSUPPORTED;
#undef QLORA_LL
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}

}  // namespace qlora
