"""Pins for the oracle's forward / backward and for the harness quantizer (CPU only)."""
import numpy as np
import pytest

import qlora_inputs as qi
from oracle import qlora_oracle as orc
from helpers import golden_lines, rel_err


def tiny(seed, M=5, K=32, N=8, r=4, bits=4, g=32):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    scales = rng.uniform(0.01, 0.1, size=(K // g, N)).astype(np.float16)
    zeros = rng.integers(0, 1 << bits, size=(K // g, N)).astype(np.float16)
    X = rng.standard_normal((M, K))
    dY = rng.standard_normal((M, N))
    A = rng.standard_normal((r, K)) * 0.3
    B = rng.standard_normal((N, r)) * 0.3
    return codes, scales, zeros, X, dY, A, B


def brute_weight(codes, scales, zeros, g):
    K, N = codes.shape
    W = [[0.0] * K for _ in range(N)]
    for n in range(N):
        for k in range(K):
            W[n][k] = float(scales[k // g, n]) * (int(codes[k, n]) - float(zeros[k // g, n]))
    return W


@pytest.mark.parametrize("bits,g", [(2, 32), (3, 32), (4, 32), (8, 32), (4, 64)])
def test_forward_backward_brute_force(bits, g):
    """Triple loops written straight from the index form of the definitions."""
    M, K, N, r, alpha = 3, 64, 8, 4, 6.0
    codes, scales, zeros, X, dY, A, B = tiny(bits, M, K, N, r, bits, g)
    Wl = brute_weight(codes, scales, zeros, g)
    s = alpha / r
    W = orc.dequant(orc.pack(codes, bits), scales, zeros, bits, g)
    Y, H = orc.forward(X, W, A, B, alpha)
    dX, dA, dB, G = orc.backward(X, dY, W, A, B, alpha)
    for m in range(M):
        h = [sum(X[m, k] * A[j, k] for k in range(K)) for j in range(r)]
        gg = [sum(dY[m, n] * B[n, j] for n in range(N)) for j in range(r)]
        for j in range(r):
            assert H[m, j] == pytest.approx(h[j], rel=1e-12, abs=1e-12)
            assert G[m, j] == pytest.approx(gg[j], rel=1e-12, abs=1e-12)
        for n in range(N):
            y = sum(X[m, k] * Wl[n][k] for k in range(K)) + s * sum(h[j] * B[n, j] for j in range(r))
            assert Y[m, n] == pytest.approx(y, rel=1e-11, abs=1e-11)
        for k in range(K):
            dx = sum(dY[m, n] * Wl[n][k] for n in range(N)) + s * sum(gg[j] * A[j, k] for j in range(r))
            assert dX[m, k] == pytest.approx(dx, rel=1e-11, abs=1e-11)
    for j in range(r):
        for k in range(K):
            da = s * sum(sum(dY[m, n] * B[n, j] for n in range(N)) * X[m, k] for m in range(M))
            assert dA[j, k] == pytest.approx(da, rel=1e-11, abs=1e-11)
        for n in range(N):
            db = s * sum(dY[m, n] * sum(X[m, k] * A[j, k] for k in range(K)) for m in range(M))
            assert dB[n, j] == pytest.approx(db, rel=1e-11, abs=1e-11)


def test_gradients_by_central_differences():
    """L = <dY, Y(X, A, B)> is bilinear in (X; A; B) separately, so central differences are exact up to round-off."""
    codes, scales, zeros, X, dY, A, B = tiny(1, M=4, K=32, N=8, r=4)
    alpha = 8.0
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    dX, dA, dB, _ = orc.backward(X, dY, W, A, B, alpha)

    def loss(X_, A_, B_):
        return float(np.sum(dY * orc.forward(X_, W, A_, B_, alpha)[0]))

    eps = 1e-3
    for arr, grad, which in ((X, dX, 0), (A, dA, 1), (B, dB, 2)):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            p, m = arr.copy(), arr.copy()
            p[idx] += eps
            m[idx] -= eps
            args_p = [X, A, B]
            args_m = [X, A, B]
            args_p[which], args_m[which] = p, m
            fd[idx] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        assert np.allclose(fd, grad, rtol=1e-7, atol=1e-8), which


def test_adjoint_identity():
    """<dY, X W^T> = <dY W, X> for the frozen-weight part (B = 0)."""
    codes, scales, zeros, X, dY, A, B = tiny(2, M=6, K=64, N=16, r=4)
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    Y, _ = orc.forward(X, W, A, np.zeros_like(B), 8.0)
    dX, _, _, _ = orc.backward(X, dY, W, A, np.zeros_like(B), 8.0)
    assert np.sum(dY * Y) == pytest.approx(np.sum(dX * X), rel=1e-12)


def test_special_cases():
    codes, scales, zeros, X, dY, A, B = tiny(3, M=6, K=64, N=16, r=4)
    alpha = 8.0
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    # B = 0: pure quantized layer, dA = 0
    Y0, _ = orc.forward(X, W, A, 0 * B, alpha)
    assert np.allclose(Y0, X @ W.T, rtol=0, atol=1e-12)
    dX0, dA0, dB0, _ = orc.backward(X, dY, W, A, 0 * B, alpha)
    assert np.all(dA0 == 0) and np.allclose(dX0, dY @ W, atol=1e-12)
    assert np.any(dB0 != 0)
    # A = 0: Y is the pure quantized layer again, dB = 0
    Y1, _ = orc.forward(X, W, 0 * A, B, alpha)
    assert np.allclose(Y1, X @ W.T, atol=1e-12)
    assert np.all(orc.backward(X, dY, W, 0 * A, B, alpha)[2] == 0)
    # every code equal to its zero-point: W = 0, Y is the pure LoRA branch
    K, N, g = codes.shape[0], codes.shape[1], 32
    zcodes = np.repeat(zeros.astype(np.uint8), g, axis=0)
    Wz = orc.dequant(orc.pack(zcodes, 4), scales, zeros, 4, g)
    assert np.all(Wz == 0)
    Yz, _ = orc.forward(X, Wz, A, B, alpha)
    assert np.allclose(Yz, (alpha / 4) * (X @ A.T) @ B.T, atol=1e-12)
    # identity rows: Y rows are the columns of W^T + s (B A)^T
    I = np.eye(K)
    Yi, _ = orc.forward(I, W, A, B, alpha)
    assert np.allclose(Yi, (W + (alpha / 4) * B @ A).T, atol=1e-12)
    # linearity in X
    X2 = np.random.default_rng(9).standard_normal(X.shape)
    Ya, _ = orc.forward(X + X2, W, A, B, alpha)
    Yb = orc.forward(X, W, A, B, alpha)[0] + orc.forward(X2, W, A, B, alpha)[0]
    assert np.allclose(Ya, Yb, atol=1e-11)
    # r = 0: no branch
    Yr0, _ = orc.forward(X, W, A[:0], B[:, :0], alpha)
    assert np.allclose(Yr0, X @ W.T, atol=1e-12)


def test_integer_gemm_special_case():
    """bits = 8, one group per row (g = K), scale 1, zero 0, integer activations: the layer is an integer matrix
    product whose float64 result is exact and equals numpy's int64 matmul."""
    rng = np.random.default_rng(4)
    M, K, N = 7, 64, 16
    codes = rng.integers(0, 256, size=(K, N), dtype=np.uint8)
    W = orc.dequant(orc.pack(codes, 8), np.ones((1, N), np.float16), np.zeros((1, N), np.float16), 8, K)
    Xi = rng.integers(-8, 9, size=(M, K))
    Y, _ = orc.forward(Xi.astype(np.float64), W, np.zeros((2, K)), np.zeros((N, 2)), 4.0)
    assert np.array_equal(Y.astype(np.int64), Xi.astype(np.int64) @ codes.astype(np.int64))
    assert np.array_equal(Y, Y.astype(np.int64))


def test_transposition_mistake_would_show():
    """Asymmetric shapes with every weight distinct: dX must use W (not W^T) and Y must use W^T."""
    M, K, N = 2, 32, 8
    codes = (np.arange(K * N).reshape(K, N) % 16).astype(np.uint8)
    scales = (np.arange(1, N + 1, dtype=np.float32)[None, :] / 64).astype(np.float16)
    zeros = np.zeros((1, N), np.float16)
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    assert W.shape == (N, K)
    assert W[3, 5] == float(scales[0, 3]) * codes[5, 3]
    X = np.zeros((M, K)); X[0, 5] = 1.0
    Y, _ = orc.forward(X, W, np.zeros((1, K)), np.zeros((N, 1)), 1.0)
    assert np.array_equal(Y[0], W[:, 5]) and np.all(Y[1] == 0)
    dY = np.zeros((M, N)); dY[1, 3] = 1.0
    dX = orc.backward(X, dY, W, np.zeros((1, K)), np.zeros((N, 1)), 1.0)[0]
    assert np.array_equal(dX[1], W[3, :]) and np.all(dX[0] == 0)


def test_lora_shapes_and_stretch_from_the_paper():
    (proj, d_model, r, total), = golden_lines("lora_param_count.txt")
    proj, d_model, r, total = int(proj), int(d_model), int(r), int(total)
    layer = qi.make_layer(K=d_model, N=d_model, bits=4, group_size=128, r=r, alpha=16.0, M=1, seed=0, with_tokens=False)
    assert layer["A"].shape == (r, d_model) and layer["B"].shape == (d_model, r)
    assert proj * (layer["A"].size + layer["B"].size) == total
    (alpha, r2, scale), = golden_lines("lora_stretch.txt")
    assert orc.lora_scale(float(alpha), int(r2)) == float(scale)


@pytest.mark.parametrize("bits,g", [(2, 64), (3, 128), (4, 128), (8, 128)])
def test_quantizer_properties(bits, g):
    """Harness quantizer: codes in range, integer zero-points in range, error at most half a step for every
    weight that was not clipped."""
    N, K = 16, 256
    w = qi.gaussian_weight(7, N, K, 0.02, outlier_frac=0.01)
    codes, scales, zeros = qi.quantize_minmax_rtn(w, bits, g)
    qmax = (1 << bits) - 1
    assert codes.shape == (K, N) and codes.dtype == np.uint8 and codes.max() <= qmax
    assert scales.shape == (K // g, N) and scales.dtype == np.float16 and np.all(scales > 0)
    assert zeros.dtype == np.float16 and np.all(zeros == np.rint(zeros)) and zeros.min() >= 0 and zeros.max() <= qmax
    W = orc.dequant(orc.pack(codes, bits), scales, zeros, bits, g)
    step = np.repeat(scales.astype(np.float64), g, axis=0).T
    unclipped = (codes.T > 0) & (codes.T < qmax)
    assert np.all(np.abs(W - w)[unclipped] <= 0.5 * step[unclipped] * (1 + 1e-3))
    assert codes.min() == 0 and codes.max() == qmax


def test_inputs_are_seeded_and_bf16():
    a = qi.config1()
    b = qi.config1()
    for key in ("codes", "scales", "zeros", "A", "B", "X", "dY"):
        assert np.array_equal(a[key], b[key])
    assert a["X"].dtype == np.uint16 and a["X"].shape == (64, 512) and a["dY"].shape == (64, 512)
    x = qi.bf16_bits_to_f32(a["X"]).astype(np.float64)
    assert abs(x.mean()) < 0.05 and abs(x.std() - 1) < 0.05
    bound = 1 / np.sqrt(512)
    assert np.abs(qi.bf16_bits_to_f32(a["A"])).max() <= bound * (1 + 2 ** -8)
    c = qi.config1(seed=1)
    assert not np.array_equal(a["X"], c["X"])


def test_layer_reference_row_sampling_matches_full():
    layer = qi.make_layer(K=64, N=32, bits=3, group_size=32, r=8, alpha=16.0, M=12, seed=3)
    full = orc.layer_reference(layer)
    rows = [0, 5, 11]
    part = orc.layer_reference(layer, rows=rows)
    assert np.allclose(part["Y"], full["Y"][rows], atol=1e-12)
    assert np.allclose(part["dX"], full["dX"][rows], atol=1e-12)
    assert np.allclose(part["dA"], full["dA"], atol=1e-12) and np.allclose(part["dB"], full["dB"], atol=1e-12)
    assert rel_err(full["Y"], full["Y"]) == 0.0


def test_stacked_adapters_gradients_and_reductions():
    """Frozen pair + trainable pair (Appendix D): central differences for dX, dA, dB of the trainable pair; B2 = 0 gives
    the single-pair layer; and the identity the CUDA library relies on -- one adapter of rank r + r2 made of the
    concatenated pairs (the frozen up-projection rescaled by s2 / s) is the same function, with the trainable pair's
    gradients in its first r rows / columns."""
    codes, scales, zeros, X, dY, A, B = tiny(41, M=4, K=32, N=8, r=4)
    rng = np.random.default_rng(42)
    A2 = rng.standard_normal((8, 32)) * 0.3
    B2 = rng.standard_normal((8, 8)) * 0.3
    alpha, alpha2 = 6.0, 4.0
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    Y, _ = orc.forward_stacked(X, W, A, B, alpha, A2, B2, alpha2)
    dX, dA, dB, _ = orc.backward_stacked(X, dY, W, A, B, alpha, A2, B2, alpha2)

    def loss(X_, A_, B_):
        return float(np.sum(dY * orc.forward_stacked(X_, W, A_, B_, alpha, A2, B2, alpha2)[0]))

    eps = 1e-4
    for arr, grad in ((X, dX), (A, dA), (B, dB)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(*arr.shape):
            up, dn = arr.copy(), arr.copy()
            up[idx] += eps
            dn[idx] -= eps
            args = [X, A, B]
            pos = [i for i, a in enumerate(args) if a is arr][0]
            au, ad = list(args), list(args)
            au[pos], ad[pos] = up, dn
            num[idx] = (loss(*au) - loss(*ad)) / (2 * eps)
        assert rel_err(grad, num) < 1e-6
    # B2 = 0: the plain layer
    Y0, _ = orc.forward_stacked(X, W, A, B, alpha, A2, np.zeros_like(B2), alpha2)
    assert np.allclose(Y0, orc.forward(X, W, A, B, alpha)[0], rtol=0, atol=1e-12)
    # the frozen pair's term, written out
    s2 = alpha2 / 8
    assert np.allclose(Y - orc.forward(X, W, A, B, alpha)[0], s2 * (X @ A2.T) @ B2.T, rtol=1e-12, atol=1e-12)
    # concatenation identity
    s = alpha / 4
    A_cat, B_cat = np.vstack([A, A2]), np.hstack([B, B2 * (s2 / s)])
    alpha_cat = s * 12
    Yc, _ = orc.forward(X, W, A_cat, B_cat, alpha_cat)
    dXc, dAc, dBc, _ = orc.backward(X, dY, W, A_cat, B_cat, alpha_cat)
    assert np.allclose(Yc, Y, rtol=1e-12, atol=1e-12) and np.allclose(dXc, dX, rtol=1e-12, atol=1e-12)
    assert np.allclose(dAc[:4], dA, rtol=1e-12, atol=1e-12) and np.allclose(dBc[:, :4], dB, rtol=1e-12, atol=1e-12)


def test_dropout_gradients_and_reductions():
    """LoRA dropout with the mask as an input (Appendix B): central differences of <dY, Y> for dX, dA, dB with the mask
    held fixed; an all-ones mask with p = 0 is the plain layer; an all-zero mask removes the branch (dA = 0, dB = 0, Y and
    dX those of the pure quantized layer); dropped positions of X get no gradient through the branch."""
    codes, scales, zeros, X, dY, A, B = tiny(51, M=4, K=32, N=8, r=4)
    rng = np.random.default_rng(52)
    mask = (rng.random(X.shape) > 0.3).astype(np.uint8)
    p, alpha = 0.3, 6.0
    W = orc.dequant(orc.pack(codes, 4), scales, zeros, 4, 32)
    dX, dA, dB, _ = orc.backward_dropout(X, dY, W, A, B, alpha, mask, p)

    def loss(X_, A_, B_):
        return float(np.sum(dY * orc.forward_dropout(X_, W, A_, B_, alpha, mask, p)[0]))

    eps = 1e-4
    for pos, (arr, grad) in enumerate(((X, dX), (A, dA), (B, dB))):
        num = np.zeros_like(arr)
        for idx in np.ndindex(*arr.shape):
            up, dn = arr.copy(), arr.copy()
            up[idx] += eps
            dn[idx] -= eps
            au, ad = [X, A, B], [X, A, B]
            au[pos], ad[pos] = up, dn
            num[idx] = (loss(*au) - loss(*ad)) / (2 * eps)
        assert rel_err(grad, num) < 1e-6
    ones = np.ones_like(mask)
    assert np.allclose(orc.forward_dropout(X, W, A, B, alpha, ones, 0.0)[0], orc.forward(X, W, A, B, alpha)[0], rtol=0, atol=1e-12)
    for got, want in zip(orc.backward_dropout(X, dY, W, A, B, alpha, ones, 0.0), orc.backward(X, dY, W, A, B, alpha)):
        assert np.allclose(got, want, rtol=0, atol=1e-12)
    none = np.zeros_like(mask)
    assert np.allclose(orc.forward_dropout(X, W, A, B, alpha, none, p)[0], X @ W.T, rtol=0, atol=1e-12)
    dX0, dA0, dB0, _ = orc.backward_dropout(X, dY, W, A, B, alpha, none, p)
    assert np.allclose(dX0, dY @ W, rtol=0, atol=1e-12) and not dA0.any() and not dB0.any()
    # where the mask is zero, dX is the frozen weight's term alone
    assert np.allclose(dX[mask == 0], (dY @ W)[mask == 0], rtol=0, atol=1e-12)
    # scaling: E-preserving 1 / (1 - p) on kept elements
    Yk, Hk = orc.forward_dropout(X, W, A, B, alpha, mask, p)
    assert np.allclose(Hk, ((X * mask) / 0.7) @ A.T, rtol=1e-12, atol=1e-12)
