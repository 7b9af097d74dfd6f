// The C ABI declared in qlora.h: argument validation, workspace carving and kernel dispatch.  No kernel lives here.
#include <cuda_runtime.h>

#include "launch.h"
#include "qlora.h"

namespace {

using namespace qlora;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_bits(int bits) { return (bits == 2 || bits == 3 || bits == 4 || bits == 8) ? QLORA_OK : QLORA_ERR_UNSUPPORTED; }

int check_format(int bits, int K, int N) {
    if (K < 0 || N < 0) return QLORA_ERR_INVALID_ARG;
    if (check_bits(bits) != QLORA_OK) return QLORA_ERR_UNSUPPORTED;
    if (K % 32 != 0 || N % 8 != 0) return QLORA_ERR_UNSUPPORTED;
    return QLORA_OK;
}

int check_desc(const qlora_desc* d, bool need_lora) {
    if (d == nullptr) return QLORA_ERR_INVALID_ARG;
    const int rc = check_format(d->bits, d->K, d->N);
    if (rc != QLORA_OK) return rc;
    if (d->group_size <= 0) return QLORA_ERR_INVALID_ARG;
    if (d->group_size % 32 != 0 || d->K % d->group_size != 0) return QLORA_ERR_UNSUPPORTED;
    if (need_lora) {
        if (d->r < 0) return QLORA_ERR_INVALID_ARG;
        if (d->r % 8 != 0 || d->r > 64) return QLORA_ERR_UNSUPPORTED;
        if (!(d->alpha == d->alpha)) return QLORA_ERR_INVALID_ARG;   // NaN
    }
    return QLORA_OK;
}

struct Workspace {
    size_t p0_off, p1_off, grad_off, sync_off, split_off, db_off;
    size_t required;   // what a call cannot do without
    size_t total;      // ... plus the optional areas, each used when the workspace reaches that far: the exchange area
                       // of split tiles, then the producers' parts of dB (qlora_bwd_input_db)
};

Workspace carve(const qlora_desc& d, int M) {
    Workspace w{};
    const size_t p = align_up((size_t)M * (size_t)d.r * sizeof(float), 256);
    w.p0_off = 0;
    w.p1_off = p;
    w.grad_off = 2 * p;
    w.sync_off = w.grad_off + align_up(lora_grad_scratch_bytes(M, d.K, d.N, d.r), 256);
    w.split_off = w.sync_off + 256;      // the counters of the tensor-core kernels: producer clusters, split tiles
    w.required = w.split_off;
    w.db_off = w.split_off + align_up(umma_split_scratch_bytes(d, M), 256);
    w.total = w.db_off + umma_db_part_bytes(d, M);
    return w;
}

}  // namespace

// What the layer calls cannot do without: qlora_workspace_bytes minus the exchange area of split tiles, which
// qlora_fwd / qlora_bwd_input use only when it is there (and qlora_bwd_lora never).
size_t qlora::required_workspace_bytes(const qlora_desc& d, int M) { return carve(d, M).required; }

extern "C" {

const char* qlora_status_string(int status) {
    switch (status) {
        case QLORA_OK: return "ok";
        case QLORA_ERR_INVALID_ARG: return "invalid argument";
        case QLORA_ERR_UNSUPPORTED: return "unsupported shape, bit width, group size or rank";
        case QLORA_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case QLORA_ERR_WORKSPACE: return "workspace missing or too small";
        case QLORA_ERR_CUDA: return "CUDA call failed";
        case QLORA_ERR_TIMEOUT: return "bounded device-side wait gave up";
        case QLORA_ERR_STATIC_LIMIT: return "scratch need exceeds the library's built-in array";
        default: return "unknown status";
    }
}

int qlora_device_status(unsigned int* status_out, int clear) {
    if (status_out == nullptr) return QLORA_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return QLORA_ERR_CUDA;
    const int rc = read_device_status(status_out, clear);
    if (rc != QLORA_OK) return rc;
    return *status_out == 0 ? QLORA_OK : QLORA_ERR_TIMEOUT;
}

int qlora_selftest_bounded_wait(int limit_us, void* cuda_stream) {
    if (limit_us < 1 || limit_us > 1000000) return QLORA_ERR_INVALID_ARG;
    return launch_wait_probe(limit_us, (cudaStream_t)cuda_stream);
}

int qlora_workspace_bytes(const qlora_desc* desc, int M, size_t* out) {
    if (out == nullptr || M < 0) return QLORA_ERR_INVALID_ARG;
    const int rc = check_desc(desc, true);
    if (rc != QLORA_OK) return rc;
    *out = carve(*desc, M).total;
    return QLORA_OK;
}

int qlora_pack(int bits, int K, int N, const uint8_t* codes, int32_t* Q, void* cuda_stream) {
    const int rc = check_format(bits, K, N);
    if (rc != QLORA_OK) return rc;
    if (K == 0 || N == 0) return QLORA_OK;
    if (codes == nullptr || Q == nullptr) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(Q)) return QLORA_ERR_ALIGNMENT;
    return launch_pack(bits, K, N, codes, Q, (cudaStream_t)cuda_stream);
}

int qlora_unpack(int bits, int K, int N, const int32_t* Q, uint8_t* codes, void* cuda_stream) {
    const int rc = check_format(bits, K, N);
    if (rc != QLORA_OK) return rc;
    if (K == 0 || N == 0) return QLORA_OK;
    if (codes == nullptr || Q == nullptr) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(Q)) return QLORA_ERR_ALIGNMENT;
    return launch_unpack(bits, K, N, Q, codes, (cudaStream_t)cuda_stream);
}

int qlora_lrec_loss(int T, int V, const void* student_logits, const void* teacher_logits, const int32_t* labels, float lambda_kl,
                    float lambda_ce, float grad_scale, float* loss_tokens, void* dlogits, void* cuda_stream) {
    if (T < 0 || V < 0) return QLORA_ERR_INVALID_ARG;
    if (V == 0 || V % 8 != 0 || V > 32768) return QLORA_ERR_UNSUPPORTED;
    if (T == 0) return QLORA_OK;
    if (!student_logits || !teacher_logits || !loss_tokens) return QLORA_ERR_INVALID_ARG;
    if (!(lambda_kl == lambda_kl) || !(lambda_ce == lambda_ce) || !(grad_scale == grad_scale)) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(student_logits) || !aligned16(teacher_logits) || !aligned16(labels) || !aligned16(loss_tokens) ||
        !aligned16(dlogits))
        return QLORA_ERR_ALIGNMENT;
    return launch_lrec_loss(T, V, student_logits, teacher_logits, labels, lambda_kl, lambda_ce, grad_scale, loss_tokens, dlogits,
                            (cudaStream_t)cuda_stream);
}

int qlora_gather_columns(int elem_bytes, int rows, int cols, const void* in, const int32_t* perm, void* out, void* cuda_stream) {
    if (rows < 0 || cols < 0) return QLORA_ERR_INVALID_ARG;
    if (elem_bytes != 2 && elem_bytes != 4) return QLORA_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return QLORA_OK;
    if (!in || !perm || !out || in == out) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(perm) || !aligned16(out)) return QLORA_ERR_ALIGNMENT;
    return launch_gather_columns(elem_bytes, rows, cols, in, perm, out, (cudaStream_t)cuda_stream);
}

int qlora_dequant(const qlora_desc* desc, const int32_t* Q, const void* scales, const void* zeros, void* W,
                  void* cuda_stream) {
    const int rc = check_desc(desc, false);
    if (rc != QLORA_OK) return rc;
    if (desc->K == 0 || desc->N == 0) return QLORA_OK;
    if (!Q || !scales || !zeros || !W) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(zeros) || !aligned16(W)) return QLORA_ERR_ALIGNMENT;
    return launch_dequant(*desc, Q, scales, zeros, W, (cudaStream_t)cuda_stream);
}

int qlora_quantize_rtn(const qlora_desc* desc, const float* W, int32_t* Q, void* scales, void* zeros, void* cuda_stream) {
    const int rc = check_desc(desc, false);
    if (rc != QLORA_OK) return rc;
    if (desc->K == 0 || desc->N == 0) return QLORA_OK;
    if (!W || !Q || !scales || !zeros) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(Q) || !aligned16(scales) || !aligned16(zeros)) return QLORA_ERR_ALIGNMENT;
    if ((long long)desc->K / desc->group_size > 65535) return QLORA_ERR_UNSUPPORTED;
    return launch_quantize_rtn(*desc, W, Q, scales, zeros, (cudaStream_t)cuda_stream);
}

// mask == NULL: the plain layer.  Otherwise LoRA dropout: the branch sees keep_scale * mask (.) X.
static int fwd_common(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const int32_t* Q,
                      const void* scales, const void* zeros, const void* A, const void* B, void* Y, float* H_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = check_desc(desc, true);
    if (rc != QLORA_OK) return rc;
    if (M < 0) return QLORA_ERR_INVALID_ARG;
    const qlora_desc& d = *desc;
    if (M == 0 || d.N == 0) return QLORA_OK;
    if (!X || !Q || !scales || !zeros || !Y) return QLORA_ERR_INVALID_ARG;
    if (d.r > 0 && (!A || !B)) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Q) || !aligned16(scales) || !aligned16(zeros) || !aligned16(Y) ||
        !aligned16(A) || !aligned16(B) || !aligned16(H_out) || !aligned16(workspace))
        return QLORA_ERR_ALIGNMENT;
    const Workspace w = carve(d, M);
    if (workspace == nullptr || workspace_bytes < w.required) return QLORA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* H = H_out ? H_out : reinterpret_cast<float*>(static_cast<char*>(workspace) + w.p0_off);
    unsigned int* sync = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + w.sync_off);
    if (stream_supported(d, M, false)) {                              // up to 16 tokens: the weight-streaming kernels
        const bool fused = d.r > 0 && d.r <= 16 && mask == nullptr;   // the down-projection rides along inside the kernel
        if (d.r > 0 && !fused) {
            rc = launch_lora_down(M, d.K, d.r, true, X, A, H, st, mask, keep_scale);
            if (rc != QLORA_OK) return rc;
        }
        return launch_stream_gemm(d, M, false, X, Q, scales, zeros, A, B, H, !fused, Y, st);
    }
    // the tensor-core path computes H itself when given A (beside its tiles where SM pairs are idle, else ahead of them)
    if (umma_supported(d, M) && mask == nullptr) return launch_umma_gemm(d, M, false, X, Q, scales, zeros, B, H, Y, st, A, sync, static_cast<char*>(workspace) + w.split_off,
                                workspace_bytes - w.split_off);
    if (d.r > 0) {
        rc = launch_lora_down(M, d.K, d.r, true, X, A, H, st, mask, keep_scale);
        if (rc != QLORA_OK) return rc;
    }
    if (umma_supported(d, M)) return launch_umma_gemm(d, M, false, X, Q, scales, zeros, B, H, Y, st);
    return launch_simt_gemm(d, M, false, X, Q, scales, zeros, B, H, Y, st);
}

// mask == NULL: the plain layer.  Otherwise LoRA dropout: the LoRA term of dX is keep_scale * mask (.) (s G A); the dense
// kernels then run without the branch (rank 0) and an elementwise pass adds the masked term.
static int bwd_input_common(const qlora_desc* desc, int M, const void* dY, const uint8_t* mask, float keep_scale,
                            const int32_t* Q, const void* scales, const void* zeros, const void* A, const void* B, void* dX,
                            float* G_out, void* workspace, size_t workspace_bytes, void* cuda_stream, DbFuse* db = nullptr) {
    int rc = check_desc(desc, true);
    if (rc != QLORA_OK) return rc;
    if (M < 0) return QLORA_ERR_INVALID_ARG;
    const qlora_desc& d = *desc;
    if (M == 0 || d.K == 0) return QLORA_OK;
    if (!dY || !Q || !scales || !zeros || !dX) return QLORA_ERR_INVALID_ARG;
    if (d.r > 0 && (!A || !B)) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(dY) || !aligned16(Q) || !aligned16(scales) || !aligned16(zeros) || !aligned16(dX) ||
        !aligned16(A) || !aligned16(B) || !aligned16(G_out) || !aligned16(workspace))
        return QLORA_ERR_ALIGNMENT;
    const Workspace w = carve(d, M);
    if (workspace == nullptr || workspace_bytes < w.required) return QLORA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* G = G_out ? G_out : reinterpret_cast<float*>(static_cast<char*>(workspace) + w.p0_off);
    if (mask != nullptr && d.r > 0) {
        rc = launch_lora_down(M, d.N, d.r, false, dY, B, G, st);
        if (rc != QLORA_OK) return rc;
        qlora_desc d0 = d;
        d0.r = 0;
        if (stream_supported(d0, M, true)) rc = launch_stream_gemm(d0, M, true, dY, Q, scales, zeros, B, A, G, true, dX, st);
        else if (umma_supported(d0, M)) rc = launch_umma_gemm(d0, M, true, dY, Q, scales, zeros, A, G, dX, st);
        else rc = launch_simt_gemm(d0, M, true, dY, Q, scales, zeros, A, G, dX, st);
        if (rc != QLORA_OK) return rc;
        return launch_lora_masked_update(M, d.K, d.r, keep_scale * d.alpha / (float)d.r, G, A, mask, dX, st);
    }
    if (stream_supported(d, M, true)) {
        const bool fused = d.r > 0 && d.r <= 16;
        if (d.r > 0 && !fused) {
            rc = launch_lora_down(M, d.N, d.r, false, dY, B, G, st);
            if (rc != QLORA_OK) return rc;
        }
        return launch_stream_gemm(d, M, true, dY, Q, scales, zeros, B, A, G, !fused, dX, st);
    }
    unsigned int* sync = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + w.sync_off);
    if (umma_supported(d, M)) {                                        // computes G (and takes dB on where it can)
        const size_t split_bytes = workspace_bytes < w.db_off ? workspace_bytes - w.split_off : w.db_off - w.split_off;
        if (db != nullptr) {
            db->part = reinterpret_cast<float*>(static_cast<char*>(workspace) + w.db_off);
            db->part_bytes = workspace_bytes > w.db_off ? workspace_bytes - w.db_off : 0;
        }
        return launch_umma_gemm(d, M, true, dY, Q, scales, zeros, A, G, dX, st, B, sync, static_cast<char*>(workspace) + w.split_off,
                                split_bytes, db);
    }
    if (d.r > 0) {
        rc = launch_lora_down(M, d.N, d.r, false, dY, B, G, st);
        if (rc != QLORA_OK) return rc;
    }
    return launch_simt_gemm(d, M, true, dY, Q, scales, zeros, A, G, dX, st);
}

// mask == NULL: the plain layer.  Otherwise LoRA dropout: H (if recomputed) and dA use keep_scale * mask (.) X.
static int bwd_lora_common(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const void* dY,
                           const void* A, const void* B, const float* H, const float* G, float* dA, float* dB, int accumulate,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = check_desc(desc, true);
    if (rc != QLORA_OK) return rc;
    if (M < 0 || (accumulate != 0 && accumulate != 1)) return QLORA_ERR_INVALID_ARG;
    const qlora_desc& d = *desc;
    if (d.r == 0) return QLORA_OK;
    if (!dA) return QLORA_ERR_INVALID_ARG;
    const bool want_dB = dB != nullptr;                     // NULL: dB was computed by qlora_bwd_input_db; only dA is wanted
    if (M > 0 && (!X || (!dY && (want_dB || !G)))) return QLORA_ERR_INVALID_ARG;
    if (M > 0 && ((want_dB && !H && !A) || (!G && !B))) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(dY) || !aligned16(A) || !aligned16(B) || !aligned16(H) || !aligned16(G) ||
        !aligned16(dA) || !aligned16(dB) || !aligned16(workspace))
        return QLORA_ERR_ALIGNMENT;
    const Workspace w = carve(d, M);
    if (workspace == nullptr || workspace_bytes < w.required) return QLORA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char* ws = static_cast<char*>(workspace);
    const float s = d.alpha / (float)d.r;
    if (M > 0 && !H && want_dB) {
        float* Hs = reinterpret_cast<float*>(ws + w.p0_off);
        rc = launch_lora_down(M, d.K, d.r, true, X, A, Hs, st, mask, keep_scale);
        if (rc != QLORA_OK) return rc;
        H = Hs;
    }
    if (M > 0 && !G) {
        float* Gs = reinterpret_cast<float*>(ws + w.p1_off);
        rc = launch_lora_down(M, d.N, d.r, false, dY, B, Gs, st);
        if (rc != QLORA_OK) return rc;
        G = Gs;
    }
    return launch_lora_grads(M, d.K, d.N, d.r, s, X, dY, H, G, dA, dB, accumulate, ws + w.grad_off, st, mask, keep_scale, want_dB ? 3 : 2);
}

static int check_dropout(const void* mask, float keep_scale, int M) {
    if (M > 0 && mask == nullptr) return QLORA_ERR_INVALID_ARG;
    if (!(keep_scale >= 1.0f) || !(keep_scale < 1e6f)) return QLORA_ERR_INVALID_ARG;   // 1 / (1 - p), p in [0, 1)
    if (!aligned16(mask)) return QLORA_ERR_ALIGNMENT;
    return QLORA_OK;
}

int qlora_fwd(const qlora_desc* desc, int M, const void* X, const int32_t* Q, const void* scales, const void* zeros,
              const void* A, const void* B, void* Y, float* H_out, void* workspace, size_t workspace_bytes,
              void* cuda_stream) {
    return fwd_common(desc, M, X, nullptr, 1.0f, Q, scales, zeros, A, B, Y, H_out, workspace, workspace_bytes, cuda_stream);
}

int qlora_bwd_input(const qlora_desc* desc, int M, const void* dY, const int32_t* Q, const void* scales,
                    const void* zeros, const void* A, const void* B, void* dX, float* G_out, void* workspace,
                    size_t workspace_bytes, void* cuda_stream) {
    return bwd_input_common(desc, M, dY, nullptr, 1.0f, Q, scales, zeros, A, B, dX, G_out, workspace, workspace_bytes, cuda_stream);
}

int qlora_bwd_input_db(const qlora_desc* desc, int M, const void* dY, const int32_t* Q, const void* scales,
                       const void* zeros, const void* A, const void* B, const float* H, void* dX, float* G_out, float* dB,
                       int accumulate, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (desc == nullptr) return QLORA_ERR_INVALID_ARG;
    if (accumulate != 0 && accumulate != 1) return QLORA_ERR_INVALID_ARG;
    if (desc->r > 0 && M > 0 && (!H || !dB)) return QLORA_ERR_INVALID_ARG;
    if (!aligned16(H) || !aligned16(dB)) return QLORA_ERR_ALIGNMENT;
    DbFuse db{H, dB, accumulate, nullptr, 0, false};
    int rc = bwd_input_common(desc, M, dY, nullptr, 1.0f, Q, scales, zeros, A, B, dX, G_out, workspace, workspace_bytes, cuda_stream,
                              desc->r > 0 ? &db : nullptr);
    if (rc != QLORA_OK || desc->r == 0 || db.done || M < 0) return rc;
    // the backward kernel of this shape has no producer clusters to do it: dB by the LoRA-gradient kernels (dY is read again)
    const qlora_desc& d = *desc;
    if (d.N == 0) return QLORA_OK;
    const Workspace w = carve(d, M);
    return launch_lora_grads(M, d.K, d.N, d.r, d.alpha / (float)d.r, nullptr, dY, H, nullptr, nullptr, dB, accumulate,
                             static_cast<char*>(workspace) + w.grad_off, (cudaStream_t)cuda_stream, nullptr, 1.0f, 1);
}

int qlora_bwd_input_db_on_producers(const qlora_desc* desc, int M) {
    const int rc = check_desc(desc, true);
    if (rc != QLORA_OK) return rc;
    if (M < 0) return QLORA_ERR_INVALID_ARG;
    return umma_db_on_producers(*desc, M) > 0 ? 1 : 0;
}

int qlora_bwd_lora(const qlora_desc* desc, int M, const void* X, const void* dY, const void* A, const void* B,
                   const float* H, const float* G, float* dA, float* dB, int accumulate, void* workspace,
                   size_t workspace_bytes, void* cuda_stream) {
    return bwd_lora_common(desc, M, X, nullptr, 1.0f, dY, A, B, H, G, dA, dB, accumulate, workspace, workspace_bytes, cuda_stream);
}

int qlora_fwd_dropout(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const int32_t* Q,
                      const void* scales, const void* zeros, const void* A, const void* B, void* Y, float* H_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    const int rc = check_dropout(mask, keep_scale, M);
    if (rc != QLORA_OK) return rc;
    return fwd_common(desc, M, X, mask, keep_scale, Q, scales, zeros, A, B, Y, H_out, workspace, workspace_bytes, cuda_stream);
}

int qlora_bwd_input_dropout(const qlora_desc* desc, int M, const void* dY, const uint8_t* mask, float keep_scale,
                            const int32_t* Q, const void* scales, const void* zeros, const void* A, const void* B, void* dX,
                            float* G_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    const int rc = check_dropout(mask, keep_scale, M);
    if (rc != QLORA_OK) return rc;
    return bwd_input_common(desc, M, dY, mask, keep_scale, Q, scales, zeros, A, B, dX, G_out, workspace, workspace_bytes, cuda_stream);
}

int qlora_bwd_lora_dropout(const qlora_desc* desc, int M, const void* X, const uint8_t* mask, float keep_scale, const void* dY,
                           const void* A, const void* B, const float* H, const float* G, float* dA, float* dB, int accumulate,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    const int rc = check_dropout(mask, keep_scale, M);
    if (rc != QLORA_OK) return rc;
    return bwd_lora_common(desc, M, X, mask, keep_scale, dY, A, B, H, G, dA, dB, accumulate, workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"
