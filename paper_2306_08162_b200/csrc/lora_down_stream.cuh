// Streaming form of the LoRA down-projection for many token rows (included by umma_kernel.cu, inside its anonymous
// namespace, after the mbarrier helpers):
//   P[m, j] = sum_t In[m, t] * L(j, t)      L_IS_A: L = A [r, T] (contraction-contiguous), else L = B [T, r].
// A CTA of 15 warps owns up to LDS_MAXB blocks of 16 token rows.  The last warp streams the activation rows
// into a deep shared-memory ring with bulk copies (one per row and chunk of LDS_TC contraction elements, ~200 KB in
// flight per SM: the product is bound by the latency of cold reads, not by arithmetic); 14 consumer warps run
// mma.sync m16n8k16 on them.  The chunks are visited chunk-major, so a warp loads its adapter fragments once per chunk
// (from L2) and reuses them for all of the CTA's row blocks, whose accumulators it keeps in registers until the end;
// then the warps' partial tiles are added in warp order through shared memory.  The summation order of a row block
// depends on nothing but T, so every launch shape gives the same bits.
// Used (a) by the producer clusters of the CTA-pair kernel and (b) by lora_down_stream_kernel, the stand-alone launch
// ahead of the tensor-core kernels when they cannot host it.

constexpr int LDS_TC = 1024;                              // contraction elements per ring stage
constexpr int LDS_ROW_BYTES = LDS_TC * 2 + 64;            // padded: rows 16 words apart (mod 32) -> conflict-free 16-byte fragment loads
constexpr int LDS_STAGE_BYTES = 16 * LDS_ROW_BYTES;       // 33 KiB
constexpr int LDS_MAXB = 8;                               // row blocks per CTA
constexpr int LDS_CWARPS = 14;                            // consumer warps (warp 14 issues the copies)
constexpr int LDS_STEPS = (LDS_TC / 32 + LDS_CWARPS - 1) / LDS_CWARPS;   // 32-wide contraction steps per warp and chunk
constexpr int LDS_BAR_BYTES = 256;                        // full[S] + empty[S] barriers behind the ring (S <= 16)

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Shared memory needed for `stages` ring stages (the cross-warp reduction reuses the ring).
constexpr size_t lds_smem_bytes(int stages) { return (size_t)stages * LDS_STAGE_BYTES + LDS_BAR_BYTES; }
constexpr int LDS_MIN_STAGES = (LDS_CWARPS * LDS_MAXB * 2 * 128 * 4 + LDS_STAGE_BYTES - 1) / LDS_STAGE_BYTES;   // room for the reduction

// Row blocks first_block, first_block + block_stride, ... (at most LDS_MAXB of them below ceil(M / 16)).
// Called by all threads of the CTA (15 warps or more; the first 15 work); `smem` is 128-byte aligned with room for lds_smem_bytes(stages), stages >=
// LDS_MIN_STAGES.  Returns with no copy in flight (every issued stage has been waited for) unless the kernel is aborting.
// WITH_DB (backward only: In = dY [M, T = N], L = B): the rows that pass through for G = dY B also give this CTA's part of
//   dB[n, j] = sum_m dY[m, n] H[m, j]   (H fp32 [M, r], the forward's down-projection; the scale s is applied by whoever adds the parts up)
// as a second product per fragment: the tokens are now the contraction, so the 8 x 8 blocks of the dY fragments are
// transposed across the warp (movmatrix) into the 16-row operand and H supplies the 8-column one.  A warp owns the columns
// n of its own contraction steps, so nothing is summed across warps; its accumulators live for one chunk and are then
// written to dBpart [T, r] (fp32, this CTA's own: every n below T is written exactly once, provided the CTA has a row block).
template <bool L_IS_A, int NT, bool WITH_DB = false, int MAXB = LDS_MAXB>   // MAXB: row blocks this instantiation keeps accumulators for
__device__ __forceinline__ void lora_down_stream(int M, int T, int r, const __nv_bfloat16* __restrict__ In,
                                                 const __nv_bfloat16* __restrict__ L, float* __restrict__ P, int first_block,
                                                 int block_stride, uint8_t* smem, int stages, volatile int* abort_flag,
                                                 const float* __restrict__ Hm = nullptr, float* __restrict__ dBpart = nullptr) {
    static_assert(!(WITH_DB && L_IS_A), "dB rides on the backward's pass over dY");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const uint32_t ring = smem_u32(smem);
    const uint32_t bar_full = ring + (uint32_t)stages * LDS_STAGE_BYTES;
    const uint32_t bar_empty = bar_full + 8u * (uint32_t)stages;
    const int n_blocks = (M + 15) / 16;
    int nb = first_block < n_blocks ? (n_blocks - first_block + block_stride - 1) / block_stride : 0;
    if (nb > MAXB) nb = MAXB;
    const int n_chunks = (T + LDS_TC - 1) / LDS_TC;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, LDS_CWARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    float acc[MAXB][NT][4];
#pragma unroll
    for (int b = 0; b < MAXB; ++b)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[b][nt][0] = acc[b][nt][1] = acc[b][nt][2] = acc[b][nt][3] = 0.f;

    if (warp == LDS_CWARPS) {
        // ---------------------------------------------------------------- copy issuer: lane 0 waits for the slot and posts
        // the byte count, then lane `row` issues the copy of that row (one thread issuing all 16 was the bottleneck)
        uint32_t slot = 0, phase = 0;
        bool live = true;
        for (int c = 0; c < n_chunks && live; ++c) {
            const int t0 = c * LDS_TC;
            const uint32_t row_bytes = (uint32_t)((T - t0 < LDS_TC ? T - t0 : LDS_TC) * 2);   // T % 8 == 0: a multiple of 16
            for (int b = 0; b < nb; ++b) {
                const int m0 = (first_block + b * block_stride) * 16;
                const int rows = M - m0 < 16 ? M - m0 : 16;
                uint32_t ok = 1;
                if (lane == 0) {
                    ok = mbar_wait(bar_empty + 8 * slot, phase ^ 1u, abort_flag) ? 1u : 0u;
                    if (ok) mbar_expect_tx(bar_full + 8 * slot, row_bytes * (uint32_t)rows);
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                if (!ok) { live = false; break; }
                if (lane < rows)
                    bulk_copy_g2s(ring + slot * LDS_STAGE_BYTES + lane * LDS_ROW_BYTES, In + (size_t)(m0 + lane) * T + t0, row_bytes,
                                  bar_full + 8 * slot);
                if (++slot == (uint32_t)stages) { slot = 0; phase ^= 1u; }
            }
        }
    } else if (warp < LDS_CWARPS) {
        // ---------------------------------------------------------------- consumers (warps beyond the issuer's have no part)
        uint32_t slot = 0, phase = 0;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        bool live = true;
        for (int c = 0; c < n_chunks && live; ++c) {
            const int t0 = c * LDS_TC;
            const int chunk_len = T - t0 < LDS_TC ? T - t0 : LDS_TC;
            // this warp's adapter fragments of the chunk (steps warp, warp + 14, ...), reused for every row block
            uint4 lf[LDS_STEPS][NT];
#pragma unroll
            for (int i = 0; i < LDS_STEPS; ++i) {
                const int k0 = t0 + (warp + i * LDS_CWARPS) * 32;          // warp-uniform
                const int k = k0 + q * 8;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    uint4 lv = zero4;
                    if ((warp + i * LDS_CWARPS) * 32 < chunk_len) {
                        if (L_IS_A) {
                            const int j = nt * 8 + g;
                            if (k < T && j < r) lv = __ldg(reinterpret_cast<const uint4*>(L + (size_t)j * T + k));
                        } else {
                            // 8 x 8 tiles of B loaded row-wise and transposed across the warp (see lora_down.cuh)
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
                    }
                    lf[i][nt] = lv;
                }
            }
            float dbacc[WITH_DB ? LDS_STEPS : 1][2][NT][4];
            if constexpr (WITH_DB) {
#pragma unroll
                for (int i = 0; i < LDS_STEPS; ++i)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) dbacc[i][h][nt][0] = dbacc[i][h][nt][1] = dbacc[i][h][nt][2] = dbacc[i][h][nt][3] = 0.f;
            }
#pragma unroll
            for (int b = 0; b < MAXB; ++b) {
                if (b < nb && live) {
                    uint32_t hb[NT][2];                                    // H rows of the block as the 8-column operand (tokens = contraction)
                    if constexpr (WITH_DB) {
                        const int mh = (first_block + b * block_stride) * 16 + 2 * q;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const int j = nt * 8 + g;
                            float h0 = 0.f, h1 = 0.f, h2 = 0.f, h3 = 0.f;
                            if (j < r) {
                                if (mh < M) h0 = Hm[(size_t)mh * r + j];
                                if (mh + 1 < M) h1 = Hm[(size_t)(mh + 1) * r + j];
                                if (mh + 8 < M) h2 = Hm[(size_t)(mh + 8) * r + j];
                                if (mh + 9 < M) h3 = Hm[(size_t)(mh + 9) * r + j];
                            }
                            const __nv_bfloat162 p0 = __floats2bfloat162_rn(h0, h1), p1 = __floats2bfloat162_rn(h2, h3);
                            hb[nt][0] = *reinterpret_cast<const uint32_t*>(&p0);
                            hb[nt][1] = *reinterpret_cast<const uint32_t*>(&p1);
                        }
                    }
                    if (!warp_wait(bar_full + 8 * slot, phase, abort_flag, lane)) { live = false; break; }
                    const int m0 = (first_block + b * block_stride) * 16;
                    const bool v0 = m0 + g < M, v1 = m0 + g + 8 < M;       // rows beyond M were not copied
                    const uint8_t* st = smem + slot * LDS_STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < LDS_STEPS; ++i) {
                        const int kl = (warp + i * LDS_CWARPS) * 32;       // warp-uniform
                        if (kl < chunk_len) {
                            const int k = kl + q * 8;                      // chunk_len % 8 == 0: 8 elements are all-in or all-out
                            const uint4 xlo = (v0 && k < chunk_len) ? *reinterpret_cast<const uint4*>(st + g * LDS_ROW_BYTES + k * 2) : zero4;
                            const uint4 xhi = (v1 && k < chunk_len) ? *reinterpret_cast<const uint4*>(st + (g + 8) * LDS_ROW_BYTES + k * 2) : zero4;
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                mma_bf16_16816(acc[b][nt], xlo.x, xhi.x, xlo.y, xhi.y, lf[i][nt].x, lf[i][nt].y);
                                mma_bf16_16816(acc[b][nt], xlo.z, xhi.z, xlo.w, xhi.w, lf[i][nt].z, lf[i][nt].w);
                            }
                            if constexpr (WITH_DB) {
                                // transposed 8 x 8 blocks: lane (g, q) then holds tokens 2q, 2q + 1 (+ 8) of column
                                // kl + 8 (g >> 1) + (g & 1) + {0, 2, 4, 6} -- the rows of the two products below
                                const uint32_t t0x = movmatrix_trans(xlo.x), t0y = movmatrix_trans(xlo.y), t1x = movmatrix_trans(xhi.x), t1y = movmatrix_trans(xhi.y);
                                const uint32_t t0z = movmatrix_trans(xlo.z), t0w = movmatrix_trans(xlo.w), t1z = movmatrix_trans(xhi.z), t1w = movmatrix_trans(xhi.w);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    mma_bf16_16816(dbacc[i][0][nt], t0x, t0y, t1x, t1y, hb[nt][0], hb[nt][1]);
                                    mma_bf16_16816(dbacc[i][1][nt], t0z, t0w, t1z, t1w, hb[nt][0], hb[nt][1]);
                                }
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
                    if (++slot == (uint32_t)stages) { slot = 0; phase ^= 1u; }
                }
            }
            if constexpr (WITH_DB) {
                // accumulator (i, h, nt): rows g / g + 8 = columns n and n + 2, n = step base + 4 h + 8 (g >> 1) + (g & 1); ranks 2q, 2q + 1
                if (live && nb > 0) {
#pragma unroll
                    for (int i = 0; i < LDS_STEPS; ++i) {
                        const int kl = (warp + i * LDS_CWARPS) * 32;
                        if (kl < chunk_len) {
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    const int n = t0 + kl + 4 * h + 8 * (g >> 1) + (g & 1), j = nt * 8 + 2 * q;
                                    if (j < r) {
                                        if (n < T) *reinterpret_cast<float2*>(dBpart + (size_t)n * r + j) = make_float2(dbacc[i][h][nt][0], dbacc[i][h][nt][1]);
                                        if (n + 2 < T) *reinterpret_cast<float2*>(dBpart + (size_t)(n + 2) * r + j) = make_float2(dbacc[i][h][nt][2], dbacc[i][h][nt][3]);
                                    }
                                }
                        }
                    }
                }
            }
        }
    }
    __syncthreads();   // every stage has landed and been read: the ring is free for the reduction
    if (*abort_flag) return;
    float* red = reinterpret_cast<float*>(smem);   // [warp][b][nt][c][lane]
    if (warp < LDS_CWARPS) {
#pragma unroll
        for (int b = 0; b < MAXB; ++b)
            if (b < nb)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) red[(((warp * LDS_MAXB + b) * NT + nt) * 4 + c) * 32 + lane] = acc[b][nt][c];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < nb * NT * 128; idx += blockDim.x) {
        const int b = idx / (NT * 128), nt = (idx >> 7) % NT, c = (idx >> 5) & 3, ln = idx & 31;
        float v = 0.f;
        for (int w = 0; w < LDS_CWARPS; ++w) v += red[(((w * LDS_MAXB + b) * NT + nt) * 4 + c) * 32 + ln];
        const int row = (first_block + b * block_stride) * 16 + (ln >> 2) + ((c & 2) ? 8 : 0);
        const int col = nt * 8 + (ln & 3) * 2 + (c & 1);
        if (row < M && col < r) P[(size_t)row * r + col] = v;
    }
    __syncthreads();
}

struct LdsParams {
    int M, T, r, stages, wait_limit_us;
    const __nv_bfloat16* In;
    const __nv_bfloat16* L;
    float* P;
};

template <bool L_IS_A>
__global__ void __launch_bounds__(kThreads, 1) lora_down_stream_kernel(const LdsParams p) {
    extern __shared__ uint8_t lds_raw[];
    __shared__ int abort_flag_s[2];   // [0] set when a wait gave up, [1] the wait limit in microseconds
    pdl_launch_dependents();
    uint8_t* smem = lds_raw + ((128u - (smem_u32(lds_raw) & 127u)) & 127u);
    if (threadIdx.x == 0) { abort_flag_s[0] = 0; abort_flag_s[1] = p.wait_limit_us; }
    __syncthreads();
    pdl_wait();
    if (p.r <= 8) lora_down_stream<L_IS_A, 1>(p.M, p.T, p.r, p.In, p.L, p.P, (int)blockIdx.x, (int)gridDim.x, smem, p.stages, abort_flag_s);
    else          lora_down_stream<L_IS_A, 2>(p.M, p.T, p.r, p.In, p.L, p.P, (int)blockIdx.x, (int)gridDim.x, smem, p.stages, abort_flag_s);
    if (abort_flag_s[0]) {   // give copies that may still be in flight time to land before the CTA's memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
}

// Stand-alone launch (r <= 16): one CTA per SM at most, each with up to LDS_MAXB row blocks.
int launch_lora_down_stream_impl(int M, int T, int r, bool l_is_A, const void* In, const void* L, float* P, cudaStream_t st) {
    if (M == 0 || r == 0) return QLORA_OK;
    const int n_blocks = (M + 15) / 16;
    int grid = n_blocks < sm_count() ? n_blocks : sm_count();
    if ((n_blocks + grid - 1) / grid > LDS_MAXB) grid = (n_blocks + LDS_MAXB - 1) / LDS_MAXB;   // several waves of CTAs
    LdsParams p{};
    p.M = M; p.T = T; p.r = r; p.stages = 6; p.wait_limit_us = kWaitLimitUs;
    p.In = (const __nv_bfloat16*)In; p.L = (const __nv_bfloat16*)L; p.P = P;
    const size_t smem_bytes = lds_smem_bytes(p.stages) + 128;
    static SmemLimit limit_a, limit_b;
    if (!limit_a.raise(lora_down_stream_kernel<true>, smem_bytes) || !limit_b.raise(lora_down_stream_kernel<false>, smem_bytes)) return QLORA_ERR_CUDA;
    const cudaError_t err = l_is_A ? launch_pdl(lora_down_stream_kernel<true>, dim3((unsigned)grid), dim3(kThreads), smem_bytes, st, 1, p)
                                   : launch_pdl(lora_down_stream_kernel<false>, dim3((unsigned)grid), dim3(kThreads), smem_bytes, st, 1, p);
    return err == cudaSuccess ? QLORA_OK : QLORA_ERR_CUDA;
}
