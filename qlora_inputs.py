"""Seeded synthetic inputs for the quantized-linear + LoRA layer.

Shared by the CPU oracle's tests and by the CUDA library's tests and benchmark; it contains none of
the layer's own arithmetic (no packing, no dequantisation, no matrix product).  What it does hold:

* a per-tensor counter-based random stream (numpy Philox keyed by seed and tensor index), so the
  same bytes reach both sides;
* float32 -> bf16 (nearest-even) rounding of the generated activations and adapters, applied
  *before* either side sees them;
* the harness quantizer: plain asymmetric min-max round-to-nearest per (output column, group).
  The paper quantizes with GPTQ on calibration data (Section 4.1, Appendix A); that needs real
  weights and a dataset, so synthetic Gaussian weights quantized by min-max RTN stand in for it.
  Any codes in range are legal inputs to the layer.

All tensors are numpy arrays: codes uint8 [K, N]; scales / zeros float16 [K/g, N]; X, dY, A, B as
uint16 bf16 bit patterns.
"""
from __future__ import annotations

import numpy as np

# tensor indices inside one layer's random stream
_T_W, _T_A, _T_B, _T_X, _T_DY, _T_OUTLIER_POS, _T_OUTLIER_SIGN = range(7)


def _rng(seed: int, tensor: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(tensor)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, tensor: int, shape, std: float = 1.0) -> np.ndarray:
    x = _rng(seed, tensor).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def uniform_bf16(seed: int, tensor: int, shape, bound: float) -> np.ndarray:
    x = _rng(seed, tensor).random(shape, dtype=np.float32)
    x = (x * np.float32(2.0) - np.float32(1.0)) * np.float32(bound)
    return f32_to_bf16_bits(x)


def gaussian_weight(seed: int, N: int, K: int, std: float = 0.02,
                    outlier_frac: float = 0.0, outlier_mag: float = 0.2) -> np.ndarray:
    """W float32 [N, K] ~ N(0, std^2); optionally a fraction of entries replaced by +-outlier_mag."""
    w = _rng(seed, _T_W).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(std)
    if outlier_frac > 0.0:
        pos = _rng(seed, _T_OUTLIER_POS).random((N, K), dtype=np.float32) < np.float32(outlier_frac)
        sign = _rng(seed, _T_OUTLIER_SIGN).random((N, K), dtype=np.float32) < np.float32(0.5)
        w[pos] = np.where(sign[pos], np.float32(outlier_mag), np.float32(-outlier_mag))
    return w


def quantize_minmax_rtn(w: np.ndarray, bits: int, group_size: int):
    """Asymmetric min-max round-to-nearest, per (output column n, group of `group_size` consecutive k).

    w float32 [N, K].  For each group: lo = min(0, min w), hi = max(0, max w), qmax = 2^bits - 1,
    scale = fp16((hi - lo) / qmax) (1 if that is 0), zero = clamp(rint(-lo / scale), 0, qmax),
    q = clamp(rint(w / scale) + zero, 0, qmax); rint is round-half-even, arithmetic in float32 with the
    fp16-rounded scale.  Returns codes uint8 [K, N], scales fp16 [K/g, N], zeros fp16 [K/g, N]
    (zeros hold integers).
    """
    N, K = w.shape
    assert K % group_size == 0
    qmax = np.float32((1 << bits) - 1)
    wg = w.reshape(N, K // group_size, group_size)
    lo = np.minimum(wg.min(axis=2), np.float32(0.0))
    hi = np.maximum(wg.max(axis=2), np.float32(0.0))
    scale16 = ((hi - lo) / qmax).astype(np.float16)
    scale16[scale16 == 0] = np.float16(1.0)
    scale = scale16.astype(np.float32)
    zero = np.clip(np.rint(-lo / scale), np.float32(0.0), qmax)
    q = np.clip(np.rint(wg / scale[:, :, None]) + zero[:, :, None], np.float32(0.0), qmax)
    codes = np.ascontiguousarray(q.reshape(N, K).T.astype(np.uint8))
    return codes, np.ascontiguousarray(scale16.T), np.ascontiguousarray(zero.astype(np.float16).T)


def make_layer(K: int, N: int, bits: int, group_size: int, r: int, alpha: float, M: int, seed: int = 0,
               w_std: float = 0.02, outlier_frac: float = 0.0, outlier_mag: float = 0.2,
               b_std: float = 0.01, with_tokens: bool = True) -> dict:
    """One projection's full input set.

    W ~ N(0, w_std^2) quantized by min-max RTN; A ~ U(-1/sqrt(K), 1/sqrt(K)); B ~ N(0, b_std^2);
    X, dY ~ N(0, 1); A, B, X, dY rounded to bf16.
    """
    w = gaussian_weight(seed, N, K, w_std, outlier_frac, outlier_mag)
    codes, scales, zeros = quantize_minmax_rtn(w, bits, group_size)
    layer = dict(K=K, N=N, bits=bits, group_size=group_size, r=r, alpha=float(alpha), M=M, seed=seed,
                 codes=codes, scales=scales, zeros=zeros,
                 A=uniform_bf16(seed, _T_A, (r, K), 1.0 / np.sqrt(K)),
                 B=normal_bf16(seed, _T_B, (N, r), b_std))
    if with_tokens:
        layer["X"] = normal_bf16(seed, _T_X, (M, K))
        layer["dY"] = normal_bf16(seed, _T_DY, (M, N))
    return layer


def random_codes_layer(K: int, N: int, bits: int, group_size: int, r: int, alpha: float, M: int, seed: int = 0) -> dict:
    """Inputs that exercise the format rather than a weight distribution: uniformly random codes, every
    integer zero-point, scales spread over several binades.  Used by the bit-exact and edge-shape tests."""
    g = _rng(seed, 100)
    qmax = (1 << bits) - 1
    codes = g.integers(0, qmax + 1, size=(K, N), dtype=np.uint8)
    zeros = g.integers(0, qmax + 1, size=(K // group_size, N)).astype(np.float16)
    mant = g.integers(1024, 2048, size=(K // group_size, N)).astype(np.float32) / np.float32(1024.0)
    expo = g.integers(-9, -4, size=(K // group_size, N)).astype(np.float32)
    scales = (mant * np.exp2(expo)).astype(np.float16)
    return dict(K=K, N=N, bits=bits, group_size=group_size, r=r, alpha=float(alpha), M=M, seed=seed,
                codes=codes, scales=scales, zeros=zeros,
                A=uniform_bf16(seed, _T_A, (r, K), 1.0 / np.sqrt(K)),
                B=normal_bf16(seed, _T_B, (N, r), 0.01),
                X=normal_bf16(seed, _T_X, (M, K)),
                dY=normal_bf16(seed, _T_DY, (M, N)))


# ----------------------------------------------------------------------------------------------
# The five benchmark configurations (shapes of LLaMA-7B projections; synthetic values)
# ----------------------------------------------------------------------------------------------
def config1(seed: int = 0) -> dict:
    return make_layer(K=512, N=512, bits=4, group_size=128, r=8, alpha=16.0, M=64, seed=seed)


def config2(seed: int = 0, M: int = 2048) -> dict:
    return make_layer(K=4096, N=4096, bits=4, group_size=128, r=8, alpha=16.0, M=M, seed=1000 + seed)


CONFIG3_SHAPES = {"gate": (4096, 11008), "up": (4096, 11008), "down": (11008, 4096)}  # name -> (K, N)


def config3(which: str, seed: int = 0, M: int = 2048) -> dict:
    K, N = CONFIG3_SHAPES[which]
    idx = list(CONFIG3_SHAPES).index(which)
    return make_layer(K=K, N=N, bits=2, group_size=64, r=16, alpha=32.0, M=M, seed=2000 + 10 * idx + seed,
                      outlier_frac=0.001, outlier_mag=0.2)


CONFIG4_M = (1, 16, 128, 2048, 8192)


def config4(bits: int, M: int, seed: int = 0) -> dict:
    assert bits in (3, 8)
    return make_layer(K=4096, N=4096, bits=bits, group_size=128, r=8, alpha=16.0, M=M, seed=3000 + bits + seed)


# config 5: name -> (K, N), in execution order inside one decoder block
CONFIG5_PROJECTIONS = (("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                       ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096))
CONFIG5_LAYERS = 32
CONFIG5_M = 4096


def config5_projection(layer: int, name: str, seed: int = 0) -> dict:
    """Weights and adapters of one projection of config 5 (INT2, group 64, r = 8, alpha = 16); no tokens."""
    names = [p[0] for p in CONFIG5_PROJECTIONS]
    _, K, N = CONFIG5_PROJECTIONS[names.index(name)]
    return make_layer(K=K, N=N, bits=2, group_size=64, r=8, alpha=16.0, M=CONFIG5_M,
                      seed=5000 + 10 * layer + names.index(name) + 1000 * seed, with_tokens=False)


def config5_tokens(seed: int = 0):
    """Layer-0 input X [M, 4096] and the seeded upstream gradients used where the chain supplies none."""
    return normal_bf16(4999 + seed, _T_X, (CONFIG5_M, 4096))


def config5_seed_grad(layer: int, name: str, N: int, seed: int = 0) -> np.ndarray:
    names = [p[0] for p in CONFIG5_PROJECTIONS]
    return normal_bf16(5000 + 10 * layer + names.index(name) + 1000 * seed, _T_DY, (CONFIG5_M, N))
