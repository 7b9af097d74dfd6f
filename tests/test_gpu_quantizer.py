"""The on-device min-max round-to-nearest quantizer against the oracle's statement of it: codes, scales and zero-points
must be the same bits (integers decided in float32 on both sides)."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from oracle import qlora_oracle as orc

pytestmark = pytest.mark.gpu


def run_gpu(W, bits, g):
    N, K = W.shape
    d = ql.desc(bits, g, K, N, 0, 1.0)
    Wd = torch.from_numpy(W).cuda()
    Q = torch.full((K * bits // 32, N), -1, dtype=torch.int32, device="cuda")
    s = torch.full((K // g, N), float("nan"), dtype=torch.float16, device="cuda")
    z = torch.full((K // g, N), float("nan"), dtype=torch.float16, device="cuda")
    ql.qlora_quantize_rtn(d, Wd, Q, s, z)
    codes = torch.empty((K, N), dtype=torch.uint8, device="cuda")
    ql.qlora_unpack(bits, K, N, Q, codes)
    torch.cuda.synchronize()
    return Q.cpu().numpy(), codes.cpu().numpy(), s.cpu().numpy(), z.cpu().numpy()


def check(W, bits, g):
    Q, codes, s, z = run_gpu(W, bits, g)
    rc, rs, rz = orc.quantize_rtn(W, bits, g)
    assert np.array_equal(s.view(np.uint16), rs.view(np.uint16)), "scales differ"
    assert np.array_equal(z, rz), "zero-points differ"
    assert np.array_equal(codes, rc), f"{int((codes != rc).sum())} codes differ"
    assert np.array_equal(Q, orc.pack(rc, bits))


@pytest.mark.parametrize("bits,g", [(4, 128), (2, 64), (3, 128), (8, 128), (4, 32), (3, 32), (2, 512), (8, 512)])
def test_config1_shape(bits, g):
    check(qi.gaussian_weight(bits + g, 512, 512, 0.02), bits, g)


@pytest.mark.parametrize("which", ["gate", "down"])
def test_config3_outliers_int2_g64(which):
    """The MLP shapes of configs[2] (0.1 % outliers at 10 sigma), 256 output features of each."""
    K = qi.CONFIG3_SHAPES[which][0]
    check(qi.gaussian_weight(5, 256, K, 0.02, outlier_frac=0.001, outlier_mag=0.2), 2, 64)


@pytest.mark.parametrize("N,K,g", [(8, 32, 32), (40, 96, 96), (72, 1408, 64), (264, 352, 32)])
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_ragged_shapes_and_special_rows(N, K, g, bits):
    W = qi.gaussian_weight(N + K + bits, N, K, 0.05, outlier_frac=0.01)
    W[0] = 0.0                           # scale 0 -> 1
    W[1] = np.abs(W[1])                  # one-sided groups
    W[2] = -np.abs(W[2])
    W[3, :] = np.float32(0.5)            # a constant group
    W[4, ::2] = np.float32(1.0); W[4, 1::2] = np.float32(-2.0)      # exact ties at bits = 2 (scale 1: 0.5 steps do not occur) ...
    W[5] = (np.arange(K) % 7 - 3).astype(np.float32) * np.float32(0.5)   # ... and here: multiples of half the scale
    check(W, bits, g)


def test_quantized_layer_runs_through_the_library():
    """Quantize on the device, then run the layer on the result: the same Y as with the oracle-quantized layer."""
    layer = qi.make_layer(K=512, N=512, bits=4, group_size=128, r=8, alpha=16.0, M=64, seed=0)
    W = qi.gaussian_weight(0, 512, 512, 0.02)
    Q, codes, s, z = run_gpu(W, 4, 128)
    assert np.array_equal(codes, layer["codes"]) and np.array_equal(s, layer["scales"]) and np.array_equal(z, layer["zeros"])
