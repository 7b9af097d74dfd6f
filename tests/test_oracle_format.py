"""Pins for the oracle's packed format and dequantisation (CPU only)."""
import itertools

import numpy as np
import pytest

from oracle import qlora_oracle as orc
from helpers import golden_lines

BITS = (2, 3, 4, 8)


def bigint_pack(col_codes, bits):
    """Independent statement of the format: one Python integer per column, sliced into 32-bit words."""
    stream = 0
    for k, q in enumerate(col_codes):
        stream |= int(q) << (k * bits)
    nwords = len(col_codes) * bits // 32
    return [(stream >> (32 * i)) & 0xFFFFFFFF for i in range(nwords)]


def bigint_unpack(words, bits):
    stream = 0
    for i, w in enumerate(words):
        stream |= int(w) << (32 * i)
    return [(stream >> (k * bits)) & ((1 << bits) - 1) for k in range(len(words) * 32 // bits)]


@pytest.mark.parametrize("bits", BITS)
def test_pack_matches_bigint_stream(bits):
    rng = np.random.default_rng(bits)
    K, N = 96, 5
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    Q = orc.pack(codes, bits).view(np.uint32)
    assert Q.shape == (K * bits // 32, N) and Q.dtype == np.uint32
    for n in range(N):
        assert [int(x) for x in Q[:, n]] == bigint_pack(codes[:, n], bits)
        assert bigint_unpack(Q[:, n], bits) == [int(x) for x in codes[:, n]]


@pytest.mark.parametrize("bits", BITS)
def test_unpack_pack_identity_random_and_ramp(bits):
    rng = np.random.default_rng(10 + bits)
    K, N = 256, 24
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    assert np.array_equal(orc.unpack(orc.pack(codes, bits), bits), codes)
    ramp = (np.arange(K)[:, None] + np.arange(N)[None, :]) % (1 << bits)
    ramp = ramp.astype(np.uint8)
    assert np.array_equal(orc.unpack(orc.pack(ramp, bits), bits), ramp)


@pytest.mark.parametrize("bits", BITS)
def test_pack_unpack_identity_on_random_words(bits):
    # every bit of every word carries a code bit (also for 3 bits: 96 bits = 32 codes), so pack(unpack(Q)) == Q
    rng = np.random.default_rng(20 + bits)
    rows = 3 * 8 * bits  # multiple of 3 for the 3-bit blocks
    Q = rng.integers(0, 1 << 32, size=(rows, 7), dtype=np.uint64).astype(np.uint32).view(np.int32)
    assert np.array_equal(orc.pack(orc.unpack(Q, bits), bits), Q)


def test_words_are_int32_and_high_bit_survives():
    codes = np.zeros((32, 1), dtype=np.uint8)
    codes[7, 0] = 0xF  # bits 28..31 -> negative int32
    Q = orc.pack(codes, 4)
    assert Q.dtype == np.int32 and Q[0, 0] < 0
    assert orc.unpack(Q, 4)[7, 0] == 0xF and orc.unpack(Q, 4).sum() == 0xF


def test_golden_int3_ramp():
    (bits, rule, *words), = golden_lines("int3_ramp_words.txt")
    assert bits == "3" and rule == "ramp_mod8"
    codes = (np.arange(32) % 8).astype(np.uint8)[:, None]
    got = orc.pack(codes, 3).view(np.uint32)[:, 0]
    assert [f"{int(w):08X}" for w in got] == words


def test_golden_onehot_words():
    for bits, k, val, *words in golden_lines("onehot_words.txt"):
        bits, k, val = int(bits), int(k), int(val)
        K = len(words) * 32 // bits
        codes = np.zeros((K, 1), dtype=np.uint8)
        codes[k, 0] = val
        got = orc.pack(codes, bits).view(np.uint32)[:, 0]
        assert [f"{int(w):08X}" for w in got] == words, (bits, k, val)
        expect = np.array([int(w, 16) for w in words], dtype=np.uint32).view(np.int32)[:, None]
        assert np.array_equal(orc.unpack(expect, bits), codes)


@pytest.mark.parametrize("bits", BITS)
def test_dequant_closed_form_every_code_scale_zero(bits):
    """w = scale*(q - zero) for every code value x every integer zero x a sweep of fp16 scales (incl. subnormal)."""
    qmax = (1 << bits) - 1
    scales = np.array([2.0 ** -24, 3 * 2.0 ** -24, 6.1e-5, 0.00731, 0.0123, 1.0, 1.999, 0.333, 65504.0 / 256],
                      dtype=np.float16)
    zs = range(0, qmax + 1) if bits < 8 else (0, 1, 127, 128, 254, 255)
    g = 32
    for z, s in itertools.product(zs, scales):
        K = ((qmax + 1 + g - 1) // g) * g
        codes = (np.arange(K) % (qmax + 1)).astype(np.uint8)[:, None]
        sc = np.full((K // g, 1), s, dtype=np.float16)
        zp = np.full((K // g, 1), z, dtype=np.float16)
        W = orc.dequant(orc.pack(codes, bits), sc, zp, bits, g)
        for k in range(K):
            assert W[0, k] == float(s) * (int(codes[k, 0]) - z)   # exact in binary64
        # the canonical bf16 is a single nearest-even rounding of that value: check against a rational rounding
        wb = orc.bf16_bits_to_f64(orc.dequant_bf16_bits(orc.pack(codes, bits), sc, zp, bits, g))
        for k in range(K):
            exact = float(s) * (int(codes[k, 0]) - z)
            if exact == 0:
                assert wb[0, k] == 0
                continue
            # |rounded - exact| <= half an ulp of an 8-bit significand
            e = np.floor(np.log2(abs(exact)))
            assert abs(wb[0, k] - exact) <= 2.0 ** (e - 8) * (1 + 1e-12)


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is halfway between 1 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 is halfway -> 1 + 2^-6 (even mantissa)
    x = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20, -(1 + 2.0 ** -8), 0.0])
    got = orc.bf16_bits_to_f64(orc.round_to_bf16_bits(x))
    assert list(got) == [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, -1.0, 0.0]


def test_groups_are_contiguous_along_k():
    bits, g, K = 4, 32, 96
    codes = np.full((K, 2), 5, dtype=np.uint8)
    sc = np.array([[1, 10], [2, 20], [4, 40]], dtype=np.float16)
    zp = np.array([[0, 1], [1, 2], [2, 3]], dtype=np.float16)
    W = orc.dequant(orc.pack(codes, bits), sc, zp, bits, g)
    assert W.shape == (2, K)
    assert np.all(W[0, :32] == 5) and np.all(W[0, 32:64] == 8) and np.all(W[0, 64:] == 12)
    assert np.all(W[1, :32] == 40) and np.all(W[1, 32:64] == 60) and np.all(W[1, 64:] == 80)


def test_dequant_rejects_bad_shapes():
    codes = np.zeros((64, 2), dtype=np.uint8)
    Q = orc.pack(codes, 4)
    with pytest.raises(ValueError):
        orc.dequant(Q, np.ones((3, 2), np.float16), np.ones((3, 2), np.float16), 4, 32)
    with pytest.raises(ValueError):
        orc.pack(np.full((32, 1), 16, np.uint8), 4)
    with pytest.raises(ValueError):
        orc.pack(codes[:33], 4)


def test_dequant_with_activation_order_index():
    """g_idx[k] = k // g gives the contiguous-group dequant; a scattered g_idx matches loops written from the index form;
    and permuting the code rows by a stable sort of g_idx turns it into a contiguous-group matrix with permuted columns
    (the identity the CUDA library's activation-order recipe rests on)."""
    rng = np.random.default_rng(9)
    bits, K, N, g = 3, 96, 8, 32
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    scales = rng.uniform(0.01, 0.1, size=(K // g, N)).astype(np.float16)
    zeros = rng.integers(0, 1 << bits, size=(K // g, N)).astype(np.float16)
    Q = orc.pack(codes, bits)
    assert np.array_equal(orc.dequant_gidx(Q, scales, zeros, bits, np.arange(K) // g), orc.dequant(Q, scales, zeros, bits, g))
    g_idx = rng.permutation(np.arange(K) // g)
    W = orc.dequant_gidx(Q, scales, zeros, bits, g_idx)
    for n in range(N):
        for k in range(K):
            assert W[n, k] == float(scales[g_idx[k], n]) * (int(codes[k, n]) - float(zeros[g_idx[k], n]))
    perm = np.argsort(g_idx, kind="stable")
    assert np.array_equal(g_idx[perm], np.arange(K) // g)
    Wp = orc.dequant(orc.pack(codes[perm], bits), scales, zeros, bits, g)
    assert np.array_equal(Wp, W[:, perm])
