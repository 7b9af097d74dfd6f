/*
 * qlora.h -- C ABI of the B200 (sm_100a) library for the frozen-quantized linear layer with a trainable
 * LoRA branch, forward and backward: the per-projection hot path of EMEF / LREC fine-tuning
 * (INT2.1 paper, Section 3.1 and Figure 1).
 *
 * Notation.  M tokens, K input features, N output features, LoRA rank r, s = alpha / r.
 *   X  bf16 [M, K]      activations               dY bf16 [M, N]   upstream gradient
 *   Q  int32 [K*bits/32, N]  packed codes (frozen) scales, zeros fp16 [K/g, N]  per-group parameters
 *   W  = dequant(Q) [N, K],  W[n,k] = scales[k/g, n] * (q[k,n] - zeros[k/g, n])
 *   A  bf16 [r, K]  LoRA down-projection           B  bf16 [N, r]   LoRA up-projection
 *   H  = X A^T  fp32 [M, r]                        G  = dY B  fp32 [M, r]
 * (Appendix B of the paper names the pair the other way round; this header follows
 *  Y = X W^T + s (X A^T) B^T, i.e. A is the matrix applied to the input first.)
 *
 * Packed format (Section 3.1, "Implementation Details": the frozen weights are a bit-packed INT32 matrix;
 * the bit layout is this library's definition).  For each output column n the K codes form a little-endian
 * bit stream: code k occupies stream bits [k*bits, k*bits+bits), LSB first, and word i of the column
 * (element Q[i*N + n]) holds stream bits [32i, 32i+32).  bits = 2, 4, 8: 16, 8, 4 codes per word.  bits = 3:
 * every 32 codes fill three consecutive words of the column; codes 10 and 21 of each block straddle two words.
 * Words are to be read as unsigned.  Zero-points are fp16 values holding integers in [0, 2^bits - 1].
 * Groups are contiguous along K: group(k) = k / group_size.
 *
 * Stacked adapters (Appendix D: a frozen error-correcting pair A2 [r2, K], B2 [N, r2] with scale s2 that stays with the
 * quantized weight, plus a newly injected trainable pair): pass ONE adapter of rank r + r2 whose A is the two A stacked
 * row-wise and whose B is [B | (s2 / s) B2] column-wise, with alpha = s (r + r2).  Y and dX are then those of the stacked
 * layer, and rows 0 .. r-1 of dA / columns 0 .. r-1 of dB are the trainable pair's gradients (the rest is ignored).
 *
 * General rules for every entry point below.
 *   - All tensor pointers are DEVICE pointers owned by the caller, dense row-major, 16-byte aligned.  The
 *     descriptor is a HOST pointer.  The library allocates no device memory and never frees anything.  What it keeps
 *     between calls is host-side and per device ordinal: which of its kernels have had their shared-memory limit
 *     raised there, the SM count and cluster occupancy it queried, one sticky health word on the device
 *     (qlora_device_status) and the fixed array of qlora_bwd_lora_static.  Nothing is keyed by a caller's pointer and no
 *     result depends on the history of calls.
 *   - Q, scales, zeros, A, B are read-only for the library.  Q, scales and zeros are FROZEN (theta_q has no gradient;
 *     Section 3.1): the layer calls are launched with programmatic stream serialization and may read these three -- and
 *     only these -- while the preceding kernel in the stream is still finishing.  A and B are theta_l, which an optimizer
 *     rewrites every step (Section 3.2, Eq. 3): they, the activations, H / G, the workspace and the outputs are touched
 *     only after the preceding kernel has completed and its writes are visible (griddepcontrol.wait).  A caller that
 *     rewrites Q, scales or zeros in the same stream must synchronise that stream (or use another stream and an event)
 *     before the next layer call on them.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the legacy default stream) of
 *     the current device.  No call synchronises the device; outputs are valid in stream order.
 *   - Calls given the same workspace must be ordered one after the other (same stream, or events): they share
 *     its contents, which include a few counters through which CTAs of one launch signal each other (set to zero in
 *     stream order ahead of the launch, so the workspace needs no initialisation).  Calls with different workspaces may
 *     overlap freely.
 *     (With many tokens a launch coordinates its CTAs through those counters: tiles wait for the CTAs that form H / G,
 *     the finishing half of a split tile for the giving half.  These waits point to CTAs dispatched earlier, so a launch
 *     never waits for itself; where the forming CTAs also own tiles -- more tiles than SM pairs -- two such launches
 *     running at the same time on different streams can still hold each other's SMs.  Every wait is bounded: after
 *     250 ms the call gives up and qlora_device_status reports QLORA_ERR_TIMEOUT.)
 *   - Return value: QLORA_OK or a negative QLORA_ERR_* code.  Arguments are validated before anything is
 *     launched; on error nothing has been enqueued.  Nothing is printed, nothing throws.
 *   - Same inputs give bitwise the same outputs on every run (fixed-order reductions, no floating-point atomics).
 *   - Supported shapes: M >= 1 (M = 0 is accepted and does nothing); K % 32 == 0; group_size % 32 == 0 and
 *     K % group_size == 0; N % 8 == 0; r in {0, 8, 16, 24, ..., 64}.  Anything else: QLORA_ERR_UNSUPPORTED.
 *     r = 0 means "no LoRA branch" (A, B may be NULL).
 */
#ifndef QLORA_H_
#define QLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    QLORA_OK = 0,
    QLORA_ERR_INVALID_ARG = -1, /* NULL where a pointer is required, negative size, bad flag */
    QLORA_ERR_UNSUPPORTED = -2, /* shape / bits / group size / rank outside the supported set */
    QLORA_ERR_ALIGNMENT = -3,   /* a tensor pointer is not 16-byte aligned */
    QLORA_ERR_WORKSPACE = -4,   /* workspace missing or smaller than qlora_workspace_bytes() */
    QLORA_ERR_CUDA = -5,        /* a CUDA runtime / driver call failed (launch, tensor-map encoding, ...) */
    QLORA_ERR_TIMEOUT = -6,     /* a bounded device-side wait gave up (reported by qlora_device_status) */
    QLORA_ERR_STATIC_LIMIT = -7 /* qlora_bwd_lora_static: the call needs more scratch than the built-in array holds */
};

/* Layer descriptor (host memory). */
typedef struct {
    int bits;       /* 2, 3, 4 or 8 */
    int group_size; /* g: codes per (scale, zero) pair along K */
    int K;          /* input features */
    int N;          /* output features */
    int r;          /* LoRA rank (0 = no branch) */
    float alpha;    /* LoRA "linear stretch"; the branch is scaled by alpha / r (Appendix B: 16 with r = 8) */
} qlora_desc;

/* Bytes of scratch the three layer calls may need for M tokens (the maximum over the calls, so one buffer
 * serves all).  The paper has no counterpart: it is how a library that allocates nothing gets its scratch.  `out` is a
 * host pointer.  The scratch holds H / G when the caller does not keep them, the partial sums of the LoRA gradients, a
 * few counters, and -- last, and optional -- two areas the tensor-core kernels use when the workspace reaches that far:
 * the one through which two SM pairs exchange the halves of an output tile whose contraction they share (many tokens,
 * last wave partly filled: up to 12 MiB on LLaMA-7B MLP shapes), and the parts of dB of qlora_bwd_input_db (8 MiB at
 * N = 4096, r = 8, 2048 tokens).  A call given less still works, without the split and with dB from the gradient
 * kernels.  Contents are undefined between calls.  The figure is computed for the current device (its SM count decides
 * what is split and how many SMs can take dB on). */
int qlora_workspace_bytes(const qlora_desc* desc, int M, size_t* out);

/* Forward (Figure 1, forward path):  Y = X W^T + s (X A^T) B^T,  bf16 output, fp32 accumulation.
 * H_out: optional fp32 [M, r]; when non-NULL receives H = X A^T for reuse by qlora_bwd_lora. */
int qlora_fwd(const qlora_desc* desc, int M, const void* X, const int32_t* Q, const void* scales,
              const void* zeros, const void* A, const void* B, void* Y, float* H_out, void* workspace,
              size_t workspace_bytes, void* cuda_stream);

/* Backward through the frozen weight (Section 3.1: transposition of the packed matrix, unpacking and the matrix
 * product fused in one kernel; Figure 1, backward path):  dX = dY W + s (dY B) A,  bf16 output.
 * G_out: optional fp32 [M, r]; when non-NULL receives G = dY B for reuse by qlora_bwd_lora. */
int qlora_bwd_input(const qlora_desc* desc, int M, const void* dY, const int32_t* Q, const void* scales,
                    const void* zeros, const void* A, const void* B, void* dX, float* G_out, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);

/* qlora_bwd_input that also produces dB = s dY^T H (Figure 1: the backward arrow into the second LoRA block leaves the
 * same dY that flows back through the frozen weight), so that dY is read once for both.  H: fp32 [M, r], the forward's
 * H_out (required when r > 0); dB: fp32 [N, r]; accumulate as in qlora_bwd_lora.  With many tokens and r <= 16 the SMs
 * that stream dY to form G inside the backward kernel form dB on the same pass (each leaves a part in the workspace,
 * the CTAs that own tiles add the parts in a fixed order while their main loops run); for other shapes dB comes from the gradient kernels after
 * the backward kernel.  Either way dB is complete when the call's work is, and the same inputs give the same bits on a
 * given device; the two routes group the sum over tokens differently, so their bits differ from each other (and from
 * qlora_bwd_lora's) in the last places.  Follow it with qlora_bwd_lora(..., dB = NULL) for dA. */
int qlora_bwd_input_db(const qlora_desc* desc, int M, const void* dY, const int32_t* Q, const void* scales,
                       const void* zeros, const void* A, const void* B, const float* H, void* dX, float* G_out, float* dB,
                       int accumulate, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Which way qlora_bwd_input_db goes for this shape on the current device, given the whole workspace: 1 = dB is formed
 * on the backward kernel's pass over dY (then qlora_bwd_input_db + qlora_bwd_lora(dB = NULL) is the cheaper pair of
 * calls), 0 = dB is handed to the gradient kernels (then qlora_bwd_input + qlora_bwd_lora is: one gradient launch
 * instead of two); negative: a QLORA_ERR_* code.  Launches nothing.  The paper has no counterpart. */
int qlora_bwd_input_db_on_producers(const qlora_desc* desc, int M);

/* Gradients of the trainable pair (Section 3.1: only theta_l is updated; Figure 1, arrows into the LoRA blocks):
 *   dA = s (dY B)^T X  fp32 [r, K],     dB = s dY^T (X A^T)  fp32 [N, r].
 * H, G: fp32 [M, r] saved by the calls above, or NULL to recompute them here (the case under gradient
 * checkpointing, Section 4.1).  accumulate = 0 overwrites dA / dB, 1 adds to their current contents
 * (micro-batch accumulation, Appendix B).  dB may be NULL (it came from qlora_bwd_input_db): only dA is computed, and
 * dY may then be NULL too when G is given. */
int qlora_bwd_lora(const qlora_desc* desc, int M, const void* X, const void* dY, const void* A, const void* B,
                   const float* H, const float* G, float* dA, float* dB, int accumulate, void* workspace,
                   size_t workspace_bytes, void* cuda_stream);

/* LoRA dropout (Appendix B: dropout 0.05 on the LoRA branch).  The branch sees D(X) = keep_scale * mask (.) X instead of X,
 * the frozen weight still sees X:
 *   Y  = X W^T + s (D(X) A^T) B^T                     H_out = D(X) A^T
 *   dX = dY W + keep_scale * mask (.) (s (dY B) A)    G_out = dY B
 *   dA = s (dY B)^T D(X)                              dB = s dY^T (D(X) A^T)
 * mask: uint8 [M, K] device pointer, non-zero = keep (the random draw is the caller's: it is an input, so that a test can
 * hand the same mask to an independent implementation); keep_scale = 1 / (1 - p) >= 1.  Pass the same mask to all three
 * calls of a step.  H passed to qlora_bwd_lora_dropout must come from qlora_fwd_dropout with that mask (or be NULL: it
 * is then recomputed with the mask).  The backward-input call runs the dense kernel without the branch and adds the masked
 * LoRA term in a second, elementwise pass over dX.  Everything else is as for the calls without dropout. */
int qlora_fwd_dropout(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const int32_t* Q,
                      const void* scales, const void* zeros, const void* A, const void* B, void* Y, float* H_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);
int qlora_bwd_input_dropout(const qlora_desc* desc, int M, const void* dY, const uint8_t* mask, float keep_scale,
                            const int32_t* Q, const void* scales, const void* zeros, const void* A, const void* B, void* dX,
                            float* G_out, void* workspace, size_t workspace_bytes, void* cuda_stream);
int qlora_bwd_lora_dropout(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const void* dY,
                           const void* A, const void* B, const float* H, const float* G, float* dA, float* dB, int accumulate,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Size of the scratch array built into the library for qlora_bwd_lora_static (16 MiB, held by every GPU that loads
 * the library until the process exits). */
#define QLORA_STATIC_SCRATCH_BYTES (16u << 20)

/* qlora_bwd_lora without a workspace argument, for callers that cannot allocate device memory when they call the
 * library: a host that has handed the whole device to its own memory pool, or a step loop that forbids allocation calls
 * because cudaMalloc / cudaFree synchronise the device.  The paper has no counterpart; this is a packaging variant of
 * qlora_bwd_lora: same arguments otherwise, same kernels, same results bit for bit.  Its scratch is a fixed array of
 * QLORA_STATIC_SCRATCH_BYTES inside the library; the call itself allocates and frees nothing.
 *   - Limit: returns QLORA_ERR_STATIC_LIMIT, with nothing enqueued, when the scratch qlora_bwd_lora needs (the part of
 *     qlora_workspace_bytes(desc, M) that is not optional) exceeds QLORA_STATIC_SCRATCH_BYTES (LLaMA-7B projections at
 *     M = 2048 with r <= 16 need 5 - 11 MiB).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *     current) and remembers it; make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which still holds what the previous call left there.  A call
 *     overwrites every element it later reads, so nothing has to be cleared; but two calls whose kernels overlap on
 *     the GPU (different streams, no ordering between them) race on it.  Keep the calls of one device in stream order. */
int qlora_bwd_lora_static(const qlora_desc* desc, int M, const void* X, const void* dY, const void* A, const void* B,
                          const float* H, const float* G, float* dA, float* dB, int accumulate, void* cuda_stream);

/* Format utilities (Section 3.1: bit-packed INT32 storage).  codes: uint8 [K, N], one code per byte.
 * qlora_pack rejects nothing about code values: only the low `bits` bits of each byte are used. */
int qlora_pack(int bits, int K, int N, const uint8_t* codes, int32_t* Q, void* cuda_stream);
int qlora_unpack(int bits, int K, int N, const int32_t* Q, uint8_t* codes, void* cuda_stream);

/* Fused LREC training loss and its gradient (Section 3.2, Eq. 1-2): per token, with p = softmax(student logits) and
 * q = softmax(teacher logits) over the V vocabulary entries,
 *     loss_tokens[t] = lambda_kl * sum_i p_i log(p_i / q_i)  +  lambda_ce * ( -log p[labels[t]] )
 *     dlogits[t, j]  = grad_scale * ( lambda_kl * p_j ((log p_j - log q_j) - KL_t) + lambda_ce * (p_j - [j == labels[t]]) )
 * (the paper prints the cross-entropy with its arguments exchanged; this is the usual next-token cross-entropy).
 * student_logits, teacher_logits: bf16 [T, V] (the teacher's are the cached targets of the full-precision model,
 * Appendix C); labels: int32 [T] or NULL, entries outside [0, V) drop the cross-entropy term of that token;
 * loss_tokens: fp32 [T] (the mean over the batch is left to the caller: pass grad_scale = 1 / n for the gradient of the
 * mean); dlogits: bf16 [T, V] or NULL (loss only).  V % 8 == 0 and V <= 32768, else QLORA_ERR_UNSUPPORTED.
 * fp32 arithmetic, fixed-order reductions (bitwise reproducible).  Each logit matrix is read once. */
int qlora_lrec_loss(int T, int V, const void* student_logits, const void* teacher_logits, const int32_t* labels, float lambda_kl,
                    float lambda_ce, float grad_scale, float* loss_tokens, void* dlogits, void* cuda_stream);

/* Column gather  out[m, j] = in[m, perm[j]]  for 2-byte (bf16) or 4-byte (fp32) elements; perm: int32 [cols] device
 * pointer holding a permutation of 0 .. cols-1 (not checked); in and out must not overlap.
 * This is the per-call step of the activation-order format (Appendix A, "activation order": the group of input feature k
 * is g_idx[k], not k / group_size).  With perm = a stable sort of the features by g_idx, the packed matrix whose code
 * rows are permuted once (codes[perm, :] re-packed) has contiguous groups, and
 *     Y = gather(X, perm) W'^T + s (gather(X, perm) gather(A, perm)^T) B^T
 * is the activation-order layer's Y; dX and dA come back in the permuted order and are un-permuted with the inverse
 * permutation (the same call). */
int qlora_gather_columns(int elem_bytes, int rows, int cols, const void* in, const int32_t* perm, void* out, void* cuda_stream);

/* Full dequantisation (Section 3.1: the weights are unpacked to floating point before every matrix product; here as a
 * stand-alone utility, for checks and for callers that want the dense weight) to the bf16 weight the tensor-core kernels stage:  W[n,k] = bf16_rne(fp32(scale) * (q - zero)),
 * bf16 [N, K].  The fp32 product is exact (an 11-bit significand times an integer of at most 9 bits), so the result
 * is a single rounding of the closed form.  desc->r and desc->alpha are ignored. */
int qlora_dequant(const qlora_desc* desc, const int32_t* Q, const void* scales, const void* zeros, void* W,
                  void* cuda_stream);

/* Asymmetric min-max round-to-nearest quantizer: the "RTN" baseline of the paper's tables (Section 4.2) and the way the
 * benchmark layers are produced.  W: fp32 [N, K] device pointer (the weight as the paper writes it, one row per output
 * feature).  For every output feature n and every group of group_size consecutive k:
 *     lo = min(0, min w), hi = max(0, max w), qmax = 2^bits - 1,
 *     scale = fp16((hi - lo) / qmax), 1 when that is 0;  zero = clamp(rint(-lo / scale), 0, qmax);
 *     q[k] = clamp(rint(w[k] / scale) + zero, 0, qmax)
 * in float32 with the fp16-rounded scale, halves to even.  Outputs: Q int32 [K*bits/32, N] (packed as above), scales and
 * zeros fp16 [K/g, N].  Integer results: the same bits as a plain CPU evaluation of these formulas.  Weights must be
 * finite.  desc->r and desc->alpha are ignored. */
int qlora_quantize_rtn(const qlora_desc* desc, const float* W, int32_t* Q, void* scales, void* zeros, void* cuda_stream);

/* Health check of the kernels enqueued so far on the current device.  Every wait inside the tensor-core kernels (on a
 * TMA transfer, on another warp, on the tensor cores) is bounded; if one ever runs out, the kernel stops early, leaves
 * its outputs incomplete and sets a sticky per-device status word instead of hanging the GPU.  This call SYNCHRONISES
 * the device, copies the word to *status_out (host pointer; 0 = healthy), clears it when `clear` is non-zero, and
 * returns QLORA_OK or QLORA_ERR_TIMEOUT.  The paper has no counterpart; it exists so that a synchronisation fault cannot hang a device. */
int qlora_device_status(unsigned int* status_out, int clear);

/* Self-test of the give-up path behind qlora_device_status (the paper has no counterpart).  Enqueues a one-CTA kernel in
 * which one thread waits, with the same bounded wait the tensor-core kernels use, on a shared-memory barrier that nobody
 * arrives at.  After limit_us microseconds (1 .. 1000000) the wait gives up, the sticky status word is set and the kernel
 * ends normally; the next qlora_device_status call reports QLORA_ERR_TIMEOUT (and clears the word if asked to).  No real
 * kernel is stalled and nothing else on the device is touched. */
int qlora_selftest_bounded_wait(int limit_us, void* cuda_stream);

/* Human-readable name of a status code (static storage; never NULL).  The paper has no counterpart. */
const char* qlora_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* QLORA_H_ */
