"""Bit-exact parity of the library's pack / unpack / dequant kernels with the oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
from oracle import qlora_oracle as orc
from gpu_util import f16_to_dev

pytestmark = pytest.mark.gpu

SHAPES = [(32, 8), (96, 40), (256, 512), (4096, 264), (352, 4096)]


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("K,N", SHAPES)
def test_pack_unpack_bit_exact(bits, K, N):
    rng = np.random.default_rng(bits * 1000 + K + N)
    for codes in (rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8),
                  ((np.arange(K)[:, None] + 3 * np.arange(N)[None, :]) % (1 << bits)).astype(np.uint8)):
        want_Q = orc.pack(codes, bits)
        d_codes = torch.from_numpy(codes).cuda()
        d_Q = torch.full((K * bits // 32, N), -1, dtype=torch.int32, device="cuda")
        ql.qlora_pack(bits, K, N, d_codes, d_Q)
        assert np.array_equal(d_Q.cpu().numpy(), want_Q)
        d_back = torch.full((K, N), 0xFF, dtype=torch.uint8, device="cuda")
        ql.qlora_unpack(bits, K, N, torch.from_numpy(want_Q).cuda(), d_back)
        assert np.array_equal(d_back.cpu().numpy(), orc.unpack(want_Q, bits))
        assert np.array_equal(d_back.cpu().numpy(), codes)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_unpack_random_words_bit_exact(bits):
    rng = np.random.default_rng(77 + bits)
    K, N = 384, 72
    Q = rng.integers(0, 1 << 32, size=(K * bits // 32, N), dtype=np.uint64).astype(np.uint32).view(np.int32)
    d_codes = torch.empty((K, N), dtype=torch.uint8, device="cuda")
    ql.qlora_unpack(bits, K, N, torch.from_numpy(Q).cuda(), d_codes)
    assert np.array_equal(d_codes.cpu().numpy(), orc.unpack(Q, bits))
    d_Q = torch.empty_like(torch.from_numpy(Q)).cuda()
    ql.qlora_pack(bits, K, N, d_codes, d_Q)
    assert np.array_equal(d_Q.cpu().numpy(), Q)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("g", [32, 64, 128, 512])
def test_dequant_bit_exact_all_codes(bits, g):
    """Every code value against every integer zero-point with scales over several binades, subnormals included."""
    rng = np.random.default_rng(bits * 10 + g)
    K, N = 512, 264
    qmax = (1 << bits) - 1
    codes = ((np.arange(K)[:, None] + np.arange(N)[None, :]) % (qmax + 1)).astype(np.uint8)
    zeros = (rng.integers(0, qmax + 1, size=(K // g, N))).astype(np.float16)
    mant = rng.integers(1024, 2048, size=(K // g, N)).astype(np.float32) / 1024
    scales = (mant * np.exp2(rng.integers(-14, 2, size=(K // g, N)).astype(np.float32))).astype(np.float16)
    scales[0, :8] = np.array([2.0 ** -24, 3 * 2.0 ** -24, 2.0 ** -15, 1023 * 2.0 ** -24, 1.0, 2.0, 0.5, 1.999], np.float16)
    Q = orc.pack(codes, bits)
    want = orc.dequant_bf16_bits(Q, scales, zeros, bits, g)
    d_W = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    ql.qlora_dequant(ql.desc(bits, g, K, N, 0, 0.0), torch.from_numpy(Q).cuda(), f16_to_dev(scales), f16_to_dev(zeros), d_W)
    got = d_W.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want)


def test_dequant_random_codes_llama_shape():
    rng = np.random.default_rng(5)
    bits, g, K, N = 4, 128, 4096, 1024
    codes = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    zeros = rng.integers(0, 16, size=(K // g, N)).astype(np.float16)
    scales = rng.uniform(0.002, 0.02, size=(K // g, N)).astype(np.float16)
    Q = orc.pack(codes, bits)
    d_W = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    ql.qlora_dequant(ql.desc(bits, g, K, N, 0, 0.0), torch.from_numpy(Q).cuda(), f16_to_dev(scales), f16_to_dev(zeros), d_W)
    got = d_W.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, orc.dequant_bf16_bits(Q, scales, zeros, bits, g))
