"""Parity of the few-token kernels (M <= 16: raw-code mma.sync streaming, contraction split over a cluster) with the
CPU oracle: every bit width, group sizes from 32 to K, ranks that are fused (8, 16) and ranks that are not (0, 24,
64), ragged column / feature tiles, contraction lengths that need more than one activation slice, and activations
whose sum does not cancel (the zero-point is applied through the sum of the activations of a group)."""
import numpy as np
import pytest
import torch

import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import GpuLayer, bf16_from_bits, to_f64
from helpers import REL_TOL, rel_err
from test_gpu_layer import check_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M", [1, 5, 8, 9, 16])
@pytest.mark.parametrize("bits,g", [(2, 64), (2, 128), (3, 32), (3, 128), (4, 32), (4, 64), (4, 128), (8, 32), (8, 128), (4, 512), (3, 256)])
def test_bits_groups_tokens(M, bits, g):
    errs, _, _ = check_layer(qi.random_codes_layer(K=512, N=768, bits=bits, group_size=g, r=8, alpha=16.0, M=M, seed=7 * M + bits + g))
    assert errs["Y"] < 1e-2 and errs["dX"] < 1e-2


@pytest.mark.parametrize("r", [0, 8, 16, 24, 64])
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_ranks(r, bits):
    check_layer(qi.random_codes_layer(K=1024, N=512, bits=bits, group_size=128, r=r, alpha=2.0 * max(r, 1), M=13, seed=r + bits))


@pytest.mark.parametrize("K,N", [(32, 8), (96, 40), (352, 520), (2048, 264), (64, 4096), (1408, 72), (11008, 256), (256, 11008)])
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_ragged_and_long_shapes(K, N, bits):
    g = 32 if K % 64 else 64
    check_layer(qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=16, alpha=32.0, M=11, seed=K + N + bits))


@pytest.mark.parametrize("bits,M", [(3, 16), (8, 1), (4, 16), (2, 7)])
def test_llama_q_proj_shape(bits, M):
    layer = qi.make_layer(K=4096, N=4096, bits=bits, group_size=128 if bits != 2 else 64, r=8, alpha=16.0, M=M, seed=bits)
    errs, _, _ = check_layer(layer)
    assert errs["Y"] < 1e-2 and errs["dX"] < 1e-2


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_activations_that_do_not_cancel(bits):
    """All-positive activations of very different magnitudes per token: sum_k X (128 + q) and (128 + z) sum_k X are then
    large against their difference, which is the quantity wanted."""
    layer = qi.random_codes_layer(K=1024, N=256, bits=bits, group_size=128, r=8, alpha=16.0, M=16, seed=bits)
    rng = np.random.default_rng(bits)
    X = np.abs(rng.standard_normal((16, 1024))).astype(np.float32) * (10.0 ** rng.integers(-3, 4, size=(16, 1)))
    dY = (np.abs(rng.standard_normal((16, 256))) + 1.0).astype(np.float32)
    layer["X"] = qi.f32_to_bf16_bits(X)
    layer["dY"] = qi.f32_to_bf16_bits(dY)
    errs, _, _ = check_layer(layer)
    assert errs["Y"] < 1e-2 and errs["dX"] < 1e-2


def test_same_bits_on_every_run_and_in_a_graph():
    layer = qi.config4(3, 16, seed=2)
    _, first, gl = check_layer(layer)
    import paper_2306_08162_b200 as ql
    M = gl.M
    Y = torch.empty_like(first["Y"]); dX = torch.empty_like(first["dX"])
    H = torch.empty_like(first["H"]); G = torch.empty_like(first["G"])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for _ in range(3):
                ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, H, gl.ws)
                ql.qlora_bwd_input(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, dX, G, gl.ws)
    for _ in range(2):
        for t in (Y, dX):
            t.view(torch.int16).fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        for got, key in ((Y, "Y"), (dX, "dX")):
            assert torch.equal(got.view(torch.int16), first[key].view(torch.int16)), key
        assert torch.equal(H, first["H"]) and torch.equal(G, first["G"])


def test_adapters_rewritten_in_stream_right_before_the_call():
    """A and B are trainable: an optimizer kernel rewrites them in the stream immediately before the next call, which
    is launched with programmatic stream serialization.  Every call must see the new values."""
    import paper_2306_08162_b200 as ql
    for bits, M in ((4, 1), (3, 16), (8, 5)):
        layer = qi.random_codes_layer(K=1024, N=1024, bits=bits, group_size=128, r=8, alpha=16.0, M=M, seed=31 + M)
        gl = GpuLayer(layer)
        A0 = qi.bf16_bits_to_f32(layer["A"]).astype(np.float64)
        B0 = qi.bf16_bits_to_f32(layer["B"]).astype(np.float64)
        Y = torch.empty((M, gl.N), dtype=torch.bfloat16, device="cuda")
        dX = torch.empty((M, gl.K), dtype=torch.bfloat16, device="cuda")
        outs = []
        for step in range(50):
            # the increments are exact in bf16 arithmetic on these magnitudes only by luck, so the reference re-reads A, B
            gl.A.add_(0.03125 * ((step % 3) - 1.0))
            gl.B.mul_(-1.0 if step % 2 else 1.25)
            ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, None, gl.ws)
            ql.qlora_bwd_input(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, dX, None, gl.ws)
            outs.append((gl.A.clone(), gl.B.clone(), Y.clone(), dX.clone()))
        torch.cuda.synchronize()
        for step in (0, 1, 2, 17, 48, 49):
            A, B, Yg, dXg = outs[step]
            lay = dict(layer)
            lay["A"] = A.view(torch.int16).cpu().numpy().view(np.uint16)
            lay["B"] = B.view(torch.int16).cpu().numpy().view(np.uint16)
            ref = orc.layer_reference(lay)
            assert rel_err(to_f64(Yg), ref["Y"]) <= REL_TOL, (bits, M, step)
            assert rel_err(to_f64(dXg), ref["dX"]) <= REL_TOL, (bits, M, step)
        assert not np.array_equal(A0, to_f64(outs[-1][0])) or not np.array_equal(B0, to_f64(outs[-1][1]))


@pytest.mark.parametrize("M", [16, 64, 1100])
def test_weights_repacked_in_stream_right_before_the_call(M):
    """The packed matrix is the one tensor the kernels read ahead of their dependency wait.  A kernel of the library that
    rewrites it (qlora_pack) must therefore hold its dependents back until it is done: two code matrices are packed
    into the SAME buffer in turn, each time immediately before a forward and a backward call in the same stream, on
    the few-token path (16 tokens), the single-CTA tensor-core path (64) and the CTA-pair path (1100)."""
    import paper_2306_08162_b200 as ql
    bits = 4
    la = qi.random_codes_layer(K=1024, N=1024, bits=bits, group_size=128, r=8, alpha=16.0, M=M, seed=71)
    lb = dict(la)
    lb["codes"] = qi.random_codes_layer(K=1024, N=1024, bits=bits, group_size=128, r=8, alpha=16.0, M=M, seed=72)["codes"]
    gl = GpuLayer(la)
    codes = [torch.from_numpy(la["codes"]).cuda(), torch.from_numpy(lb["codes"]).cuda()]
    Y = torch.empty((M, gl.N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, gl.K), dtype=torch.bfloat16, device="cuda")
    outs = []
    for step in range(20):
        ql.qlora_pack(bits, gl.K, gl.N, codes[step % 2], gl.Q)
        ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, None, gl.ws)
        ql.qlora_bwd_input(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, dX, None, gl.ws)
        outs.append((Y.clone(), dX.clone()))
    torch.cuda.synchronize()
    assert ql.qlora_device_status() == 0
    rows = np.unique(np.concatenate([np.arange(min(M, 8)), np.arange(max(M - 8, 0), M)]))
    refs = [orc.layer_reference(la, rows=rows), orc.layer_reference(lb, rows=rows)]
    rows_t = torch.from_numpy(rows).cuda()
    for step, (Yg, dXg) in enumerate(outs):
        ref = refs[step % 2]
        assert rel_err(to_f64(Yg[rows_t]), ref["Y"]) <= REL_TOL, (M, step)
        assert rel_err(to_f64(dXg[rows_t]), ref["dX"]) <= REL_TOL, (M, step)
    # the two code matrices give different results, so a stale read would have shown
    assert rel_err(to_f64(outs[0][0][rows_t]), refs[1]["Y"]) > REL_TOL
