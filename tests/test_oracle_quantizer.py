"""Pins of the oracle's min-max round-to-nearest quantizer: hand-worked groups (ties included), the half-step error
bound, the invariants of the definition, and agreement with what dequant() makes of its output."""
import os

import numpy as np
import pytest

import qlora_inputs as qi
from oracle import qlora_oracle as orc
from helpers import GOLDEN


def _worked_groups():
    out = []
    with open(os.path.join(GOLDEN, "rtn_worked_groups.txt")) as f:
        for ln in f:
            if not ln.strip() or ln.startswith("#"):
                continue
            bits, ws, scale, zero, cs, rest = [t.strip() for t in ln.split("|")]
            w = np.zeros(32, dtype=np.float32)
            for item in ws.split():
                i, v = item.split(":")
                w[int(i)] = np.float32(float(v))
            codes = np.full(32, int(rest), dtype=np.uint8)
            for item in cs.split():
                i, c = item.split(":")
                codes[int(i)] = int(c)
            out.append((int(bits), w, float(scale), int(zero), codes))
    return out


@pytest.mark.parametrize("case", range(5))
def test_hand_worked_groups(case):
    bits, w, scale, zero, codes = _worked_groups()[case]
    # the group is placed second of three in row 1 of a 2-row matrix, so a wrong axis or offset shows
    W = np.zeros((2, 96), dtype=np.float32)
    W[1, 32:64] = w
    q, s, z = orc.quantize_rtn(W, bits, 32)
    assert q.shape == (96, 2) and s.shape == (3, 2) and z.shape == (3, 2) and s.dtype == np.float16 and z.dtype == np.float16
    assert float(s[1, 1]) == scale and float(z[1, 1]) == zero
    assert np.array_equal(q[32:64, 1], codes)
    # every other group is all zero: scale 1, zero 0, codes 0
    mask = np.ones((3, 2), dtype=bool); mask[1, 1] = False
    assert np.all(s[mask] == 1.0) and np.all(z[mask] == 0.0)
    assert not q[:32].any() and not q[64:].any() and not q[:, 0].any()


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("g", [32, 128])
def test_error_bound_and_invariants(bits, g):
    N, K = 24, 512
    W = qi.gaussian_weight(11 + bits, N, K, 0.02, outlier_frac=0.01)
    W[3] = np.abs(W[3]); W[4] = -np.abs(W[4]); W[5] = 0.0                      # one-sided and empty rows
    q, s, z = orc.quantize_rtn(W, bits, g)
    qmax = (1 << bits) - 1
    sf = s.astype(np.float64); zf = z.astype(np.float64)
    assert np.all(sf > 0) and np.all(zf == np.rint(zf)) and zf.min() >= 0 and zf.max() <= qmax and q.max() <= qmax
    Wd = orc.dequant(orc.pack(q, bits), s, z, bits, g)                         # [N, K]
    step = np.repeat(sf.T, g, axis=1)                                          # [N, K]
    err = np.abs(W.astype(np.float64) - Wd)
    # the grid point next to w: rint(w / scale) + zero, before clamping
    unclipped = np.rint(W.astype(np.float64) / step) + np.repeat(zf.T, g, axis=1)
    inside = (unclipped >= 0) & (unclipped <= qmax)
    assert np.all(err[inside] <= 0.5 * step[inside] * (1 + 1e-6))
    assert np.all(err[~inside] <= 1.0 * step[~inside] * (1 + 1e-6))           # the clamp costs at most half a step more
    assert inside.mean() > 0.99
    # the codes of a group whose weights have both signs reach both ends of the range (to within the rounding of zero)
    qg = q.reshape(K // g, g, N)
    both = (W.reshape(N, K // g, g).min(axis=2) < 0) & (W.reshape(N, K // g, g).max(axis=2) > 0)
    assert np.all(qg.min(axis=1).T[both] <= 1) and np.all(qg.max(axis=1).T[both] >= qmax - 1)
    # zero weights map exactly to the zero-point (0 is on the grid)
    assert np.array_equal(q[:, 5], np.repeat(z[:, 5], g).astype(np.uint8))
    assert np.all(Wd[5] == 0.0)


def test_scale_is_the_fp16_rounding_of_the_range():
    W = qi.gaussian_weight(5, 8, 256, 0.02)
    _, s, _ = orc.quantize_rtn(W, 4, 128)
    wg = W.reshape(8, 2, 128).astype(np.float64)
    rng = (np.maximum(wg.max(axis=2), 0) - np.minimum(wg.min(axis=2), 0)) / 15.0
    assert np.all(np.abs(s.T.astype(np.float64) - rng) <= np.abs(rng) * 2.0 ** -11 * 1.001 + 1e-12)


def test_quantizing_the_grid_returns_the_codes():
    """Weights that already lie on a grid spanning the full code range come back as the same codes."""
    rng = np.random.default_rng(0)
    for bits in (2, 3, 4, 8):
        qmax = (1 << bits) - 1
        codes = rng.integers(0, qmax + 1, size=(64, 6)).astype(np.uint8)
        codes[0, :] = 0; codes[1, :] = qmax; codes[32, :] = 0; codes[33, :] = qmax
        zero = rng.integers(1, qmax, size=(2, 6)).astype(np.float64) if bits > 2 else np.ones((2, 6))
        scale = 2.0 ** rng.integers(-8, -2, size=(2, 6)).astype(np.float64)      # powers of two: every product exact
        W = (np.repeat(scale, 32, axis=0) * (codes - np.repeat(zero, 32, axis=0))).T.astype(np.float32)
        q, s, z = orc.quantize_rtn(W, bits, 32)
        assert np.array_equal(q, codes) and np.array_equal(s.astype(np.float64), scale) and np.array_equal(z.astype(np.float64), zero)


def test_generator_codes_are_the_oracles():
    """The synthetic-input module produces the layers' codes; the oracle's statement of the quantizer gives the same."""
    W = qi.gaussian_weight(3, 16, 256, 0.02, outlier_frac=0.02)
    for bits, g in ((2, 64), (3, 128), (4, 32), (8, 256)):
        a = qi.quantize_minmax_rtn(W, bits, g)
        b = orc.quantize_rtn(W, bits, g)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
