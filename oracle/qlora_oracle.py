"""CPU oracle for the frozen-quantized linear layer with a LoRA branch (EMEF / LREC hot path).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA library is
checked against.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it; the product path never does, and this module imports nothing from the CUDA package.

Everything is numpy in float64 (the inputs are bf16 / fp16 valued, so every product below is exact
in float64 and only the summation order rounds).  Matrix products use numpy's matmul as a library
step; there is no blocking, fusion or re-association beyond what the formulas state.

Notation (Section 3.1, Figure 1, Appendix B of the paper; the packed format itself is only
described there as "a bit-packed, compact INT32 datatype matrix", so the bit layout below is this
library's definition):

    X  [M, K]  activations            W = dequant(Q)  [N, K]  frozen weight
    A  [r, K]  LoRA down-projection   B  [N, r]  LoRA up-projection      s = alpha / r
    Y  = X W^T + s (X A^T) B^T                                   (forward, Figure 1)
    dX = dY W + s (dY B) A                                       (backward through the frozen weight)
    dA = s (dY B)^T X          dB = s dY^T (X A^T)               (only the LoRA pair is trained)

Pins (tests/test_oracle_*.py): pack/unpack against a big-integer bit-stream and hand-computed words;
dequant against the closed form on every code value; forward/backward against brute-force loops,
central finite differences, the adjoint identity and the B=0 / A=0 / q=zero special cases.
quantize_rtn against hand-worked groups (incl. ties), the half-step error bound and its invariants.
The choice of bit layout is "format unpinned by the paper" (no example is printed there).
"""
from __future__ import annotations

import numpy as np

SUPPORTED_BITS = (2, 3, 4, 8)


# ----------------------------------------------------------------------------------------------
# Packed storage format (Section 3.1, "Implementation Details": bit-packed INT32 matrix)
# ----------------------------------------------------------------------------------------------
def packed_rows(K: int, bits: int) -> int:
    """Number of int32 rows that hold K codes of `bits` bits for one output column."""
    if bits not in SUPPORTED_BITS:
        raise ValueError(f"bits must be one of {SUPPORTED_BITS}")
    if K % 32 != 0:
        raise ValueError("K must be a multiple of 32")
    return K * bits // 32


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    """codes uint8 [K, N] (values < 2**bits)  ->  Q int32 [K*bits/32, N].

    Definition: for every output column n, the K codes form a little-endian bit stream in which
    code k occupies stream bits [k*bits, (k+1)*bits), least significant bit first.  Word i of the
    column holds stream bits [32 i, 32 i + 32), stream bit 32 i being the word's bit 0.
    For bits in {2, 4, 8} no code crosses a word; for bits = 3 every 32 codes fill exactly three
    words and codes 10 and 21 of each block straddle two of them.
    """
    codes = np.asarray(codes)
    K, N = codes.shape
    rows = packed_rows(K, bits)
    if codes.size and int(codes.max()) >= (1 << bits):
        raise ValueError("code out of range")
    # stream[k*bits + t, n] = bit t of codes[k, n]
    stream = np.empty((K, bits, N), dtype=np.uint8)
    for t in range(bits):
        stream[:, t, :] = (codes >> t) & 1
    stream = stream.reshape(K * bits, N)
    words = np.zeros((rows, N), dtype=np.uint64)
    grouped = stream.reshape(rows, 32, N)
    for u in range(32):
        words |= grouped[:, u, :].astype(np.uint64) << np.uint64(u)
    return words.astype(np.uint32).view(np.int32)


def unpack(Q: np.ndarray, bits: int) -> np.ndarray:
    """Inverse of `pack`: Q int32 [K*bits/32, N] -> codes uint8 [K, N]."""
    if bits not in SUPPORTED_BITS:
        raise ValueError(f"bits must be one of {SUPPORTED_BITS}")
    words = np.ascontiguousarray(Q).view(np.uint32)
    rows, N = words.shape
    if (rows * 32) % bits != 0:
        raise ValueError("row count does not hold a whole number of codes")
    K = rows * 32 // bits
    stream = np.empty((rows, 32, N), dtype=np.uint8)
    for u in range(32):
        stream[:, u, :] = (words >> np.uint32(u)) & np.uint32(1)
    per_code = stream.reshape(K, bits, N)
    codes = np.zeros((K, N), dtype=np.uint8)
    for t in range(bits):
        codes |= per_code[:, t, :] << t
    return codes


# ----------------------------------------------------------------------------------------------
# Dequantisation: w = scale * (q - zero), per group of g consecutive k (group(k) = k // g)
# ----------------------------------------------------------------------------------------------
def dequant(Q: np.ndarray, scales: np.ndarray, zeros: np.ndarray, bits: int, group_size: int) -> np.ndarray:
    """Exact float64 weight W [N, K]: W[n, k] = scales[k//g, n] * (q[k, n] - zeros[k//g, n]).

    scales, zeros: float16 [K/g, N].  The product of an fp16 value and an integer of at most nine
    bits is exact in float64 (and in float32), so this is the mathematical value, unrounded.
    """
    q = unpack(Q, bits).astype(np.float64)                      # [K, N]
    K, N = q.shape
    if K % group_size != 0:
        raise ValueError("group_size must divide K")
    s = np.asarray(scales, dtype=np.float16).astype(np.float64)  # [K/g, N]
    z = np.asarray(zeros, dtype=np.float16).astype(np.float64)
    if s.shape != (K // group_size, N) or z.shape != s.shape:
        raise ValueError("scales / zeros must be [K/g, N]")
    s_full = np.repeat(s, group_size, axis=0)                    # [K, N]
    z_full = np.repeat(z, group_size, axis=0)
    return np.ascontiguousarray((s_full * (q - z_full)).T)      # [N, K]


def dequant_gidx(Q: np.ndarray, scales: np.ndarray, zeros: np.ndarray, bits: int, g_idx: np.ndarray) -> np.ndarray:
    """Activation-order format (Appendix A): the group of input feature k is g_idx[k] instead of k // g.
    W[n, k] = scales[g_idx[k], n] * (q[k, n] - zeros[g_idx[k], n]).  float64 [N, K]."""
    q = unpack(Q, bits).astype(np.float64)                      # [K, N]
    g_idx = np.asarray(g_idx)
    if g_idx.shape != (q.shape[0],):
        raise ValueError("g_idx must have one entry per input feature")
    s = np.asarray(scales, dtype=np.float16).astype(np.float64)[g_idx]   # [K, N]
    z = np.asarray(zeros, dtype=np.float16).astype(np.float64)[g_idx]
    return np.ascontiguousarray((s * (q - z)).T)


def quantize_rtn(W: np.ndarray, bits: int, group_size: int):
    """Asymmetric min-max round-to-nearest quantizer, the "RTN" baseline the paper's quantized models are
    compared with and the way the benchmark configurations produce their codes ("asymmetric round-to-nearest
    min-max", group size g along K).  W float32 [N, K]  ->  codes uint8 [K, N], scales fp16 [K/g, N],
    zeros fp16 [K/g, N] (integer valued).

    For every output row n and every group of g consecutive k (written out one group at a time):
        lo = min(0, min w)          hi = max(0, max w)           qmax = 2^bits - 1
        scale = fp16_rne((hi - lo) / qmax);  scale = 1 when that is 0
        zero  = clamp(rint(-lo / scale), 0, qmax)
        q[k]  = clamp(rint(w[k] / scale) + zero, 0, qmax)
    rint rounds halves to even.  The codes are integers decided by floating-point arithmetic, so the
    precision is part of the definition: float32 throughout, with the fp16-rounded scale, which is what
    a GPU kernel computes in too (IEEE division and rint give the same bits on both sides).
    """
    W = np.asarray(W, dtype=np.float32)
    N, K = W.shape
    if K % group_size != 0:
        raise ValueError("group_size must divide K")
    qmax = np.float32((1 << bits) - 1)
    zero32 = np.float32(0.0)
    G = K // group_size
    codes = np.empty((K, N), dtype=np.uint8)
    scales = np.empty((G, N), dtype=np.float16)
    zeros = np.empty((G, N), dtype=np.float16)
    for gi in range(G):
        w = W[:, gi * group_size:(gi + 1) * group_size]                # [N, g]
        lo = np.minimum(w.min(axis=1), zero32)
        hi = np.maximum(w.max(axis=1), zero32)
        sc16 = ((hi - lo) / qmax).astype(np.float16)                   # one rounding, nearest even
        sc16 = np.where(sc16 == np.float16(0.0), np.float16(1.0), sc16)
        sc = sc16.astype(np.float32)
        z = np.clip(np.rint((-lo) / sc), zero32, qmax)
        q = np.clip(np.rint(w / sc[:, None]) + z[:, None], zero32, qmax)
        codes[gi * group_size:(gi + 1) * group_size, :] = q.T.astype(np.uint8)
        scales[gi, :] = sc16
        zeros[gi, :] = z.astype(np.float16)
    return codes, scales, zeros


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values (exactly representable in float32) to bf16, nearest-even; returns uint16 bit patterns."""
    f32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    if not np.array_equal(f32.astype(np.float64), np.asarray(x, dtype=np.float64)):
        raise ValueError("value is not exactly representable in float32")
    u = f32.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    rounded = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(bits16: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 values."""
    u = np.asarray(bits16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def dequant_bf16_bits(Q, scales, zeros, bits: int, group_size: int) -> np.ndarray:
    """The canonical bf16 weight the GPU stages for its tensor cores: one nearest-even rounding of the
    exact value scale*(q-zero).  uint16 [N, K].  (The fp32 product is exact, so there is a single rounding.)"""
    return round_to_bf16_bits(dequant(Q, scales, zeros, bits, group_size))


# ----------------------------------------------------------------------------------------------
# Forward / backward of the layer (Figure 1; Section 3.1: theta_q frozen, only theta_l trained)
# ----------------------------------------------------------------------------------------------
def lora_scale(alpha: float, r: int) -> float:
    """s = alpha / r, the "linear stretch" of Appendix B (16 with r = 8 gives 2)."""
    return float(alpha) / float(r)


def forward(X, W, A, B, alpha: float):
    """Y = X W^T + s (X A^T) B^T.  Returns (Y [M,N], H [M,r]) with H = X A^T, all float64."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    r = A.shape[0]
    H = X @ A.T
    if r == 0:
        return X @ W.T, H
    s = lora_scale(alpha, r)
    Y = X @ W.T + s * (H @ B.T)
    return Y, H


def backward(X, dY, W, A, B, alpha: float):
    """Gradients of L = <dY, Y> with respect to X, A, B (the frozen weight gets none).

    dX = dY W + s (dY B) A,   dA = s (dY B)^T X,   dB = s dY^T (X A^T).
    Returns (dX [M,K], dA [r,K], dB [N,r], G [M,r]) with G = dY B, all float64.
    """
    X = np.asarray(X, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    r = A.shape[0]
    G = dY @ B
    if r == 0:
        return dY @ W, np.zeros_like(A), np.zeros_like(B), G
    s = lora_scale(alpha, r)
    H = X @ A.T
    dX = dY @ W + s * (G @ A)
    dA = s * (G.T @ X)
    dB = s * (dY.T @ H)
    return dX, dA, dB, G


# ----------------------------------------------------------------------------------------------
# Stacked adapters (Appendix D, "LREC Augmented EMEF"): a frozen error-correcting pair (A2, B2) that
# stays with the quantized weight, plus a newly injected trainable pair (A, B).  Only the new pair
# receives gradients.
# ----------------------------------------------------------------------------------------------
def forward_stacked(X, W, A, B, alpha, A2, B2, alpha2):
    """Y = X W^T + s (X A^T) B^T + s2 (X A2^T) B2^T,  s = alpha / r,  s2 = alpha2 / r2.  float64."""
    X = np.asarray(X, dtype=np.float64)
    A2 = np.asarray(A2, dtype=np.float64)
    B2 = np.asarray(B2, dtype=np.float64)
    Y, H = forward(X, W, A, B, alpha)
    s2 = lora_scale(alpha2, A2.shape[0])
    return Y + s2 * ((X @ A2.T) @ B2.T), H


def backward_stacked(X, dY, W, A, B, alpha, A2, B2, alpha2):
    """dX = dY W + s (dY B) A + s2 (dY B2) A2;  dA, dB of the trainable pair as in `backward`
    (the frozen pair appears in neither of them: Y is linear in each pair separately)."""
    dY = np.asarray(dY, dtype=np.float64)
    A2 = np.asarray(A2, dtype=np.float64)
    B2 = np.asarray(B2, dtype=np.float64)
    dX, dA, dB, G = backward(X, dY, W, A, B, alpha)
    s2 = lora_scale(alpha2, A2.shape[0])
    return dX + s2 * ((dY @ B2) @ A2), dA, dB, G


# ----------------------------------------------------------------------------------------------
# LoRA dropout (Appendix B: dropout 0.05 on the LoRA branch).  The mask is an input (the draw is
# not part of the layer's arithmetic): D(X) = mask * X / (1 - p).
# ----------------------------------------------------------------------------------------------
def forward_dropout(X, W, A, B, alpha, mask, p):
    """Y = X W^T + s (D(X) A^T) B^T.  Returns (Y, H) with H = D(X) A^T.  float64."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    Xd = X * (np.asarray(mask) != 0) / (1.0 - p)
    H = Xd @ A.T
    s = lora_scale(alpha, A.shape[0])
    return X @ W.T + s * (H @ B.T), H


def backward_dropout(X, dY, W, A, B, alpha, mask, p):
    """dX = dY W + D'(s (dY B) A) with D'(Z) = mask * Z / (1 - p);  dA = s (dY B)^T D(X);  dB = s dY^T (D(X) A^T)."""
    X = np.asarray(X, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    keep = (np.asarray(mask) != 0) / (1.0 - p)
    Xd = X * keep
    s = lora_scale(alpha, A.shape[0])
    G = dY @ B
    dX = dY @ W + keep * (s * (G @ A))
    dA = s * (G.T @ Xd)
    dB = s * (dY.T @ (Xd @ A.T))
    return dX, dA, dB, G


# ----------------------------------------------------------------------------------------------
# LREC objective (Section 3.2, Eq. 1-2): lambda_KL * KL(student || teacher) + lambda_CE * CE(student, label).
# The paper prints the cross-entropy with its two arguments exchanged (log of a one-hot target);
# the reading taken is the usual next-token cross-entropy, -log p[label].
# ----------------------------------------------------------------------------------------------
def lrec_loss(student_logits, teacher_logits, labels, lambda_kl: float, lambda_ce: float):
    """Per-token loss [T] and its gradient with respect to the student logits [T, V], float64.

    p = softmax(z), q = softmax(t);  loss_t = lambda_kl * sum_i p_i (log p_i - log q_i) + lambda_ce * (-log p[label_t]).
    Labels outside [0, V) drop the cross-entropy term of that token."""
    z = np.asarray(student_logits, dtype=np.float64)
    t = np.asarray(teacher_logits, dtype=np.float64)
    T, V = z.shape
    logp = z - z.max(axis=1, keepdims=True)
    logp = logp - np.log(np.exp(logp).sum(axis=1, keepdims=True))
    logq = t - t.max(axis=1, keepdims=True)
    logq = logq - np.log(np.exp(logq).sum(axis=1, keepdims=True))
    p = np.exp(logp)
    kl = (p * (logp - logq)).sum(axis=1)
    loss = lambda_kl * kl
    grad = lambda_kl * p * ((logp - logq) - kl[:, None])
    if labels is not None:
        labels = np.asarray(labels)
        for tok in range(T):
            lab = int(labels[tok])
            if 0 <= lab < V:
                loss[tok] += lambda_ce * (-logp[tok, lab])
                grad[tok] += lambda_ce * p[tok]
                grad[tok, lab] -= lambda_ce
    return loss, grad


def layer_reference(inputs: dict, rows=None) -> dict:
    """Convenience wrapper for the tests: takes the dict produced by the synthetic-input module
    (bf16 bit patterns for X, dY, A, B; uint8 codes; fp16 scales / zeros) and returns the oracle's
    Y, dX (optionally only for the token rows `rows`), dA, dB, H, G and the packed matrix.

    When `rows` is given, Y / dX / H / G cover just those rows; dA and dB always use every row.
    """
    bits, g, alpha = inputs["bits"], inputs["group_size"], inputs["alpha"]
    Q = pack(inputs["codes"], bits)
    W = dequant(Q, inputs["scales"], inputs["zeros"], bits, g)
    X = bf16_bits_to_f64(inputs["X"])
    dY = bf16_bits_to_f64(inputs["dY"])
    A = bf16_bits_to_f64(inputs["A"])
    B = bf16_bits_to_f64(inputs["B"])
    out = {"Q": Q}
    if rows is None:
        Y, H = forward(X, W, A, B, alpha)
        dX, dA, dB, G = backward(X, dY, W, A, B, alpha)
    else:
        rows = np.asarray(rows)
        Y, H = forward(X[rows], W, A, B, alpha)
        dX, _, _, G = backward(X[rows], dY[rows], W, A, B, alpha)
        r = A.shape[0]
        s = lora_scale(alpha, r) if r else 0.0
        dA = s * ((dY @ B).T @ X)
        dB = s * (dY.T @ (X @ A.T))
    out.update(Y=Y, H=H, dX=dX, dA=dA, dB=dB, G=G)
    return out
