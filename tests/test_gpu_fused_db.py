"""qlora_bwd_input_db: the backward call that also produces dB = s dY^T H, so that dY is read once (Figure 1: the
gradient of the second LoRA block leaves the same dY that flows back through the frozen weight).  With many tokens and
r = 8 the SM pairs that stream dY to form G inside the backward kernel form dB on the same pass; other shapes fall back
to the gradient kernels.  Every route is compared with the oracle; dX and G must be bit-identical to qlora_bwd_input's."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import GpuLayer, to_f64
from helpers import REL_TOL, rel_err

pytestmark = pytest.mark.gpu


def run_db(gl, accumulate=0, dB0=None):
    M, dev = gl.M, gl.X.device
    Y = torch.empty((M, gl.N), dtype=torch.bfloat16, device=dev)
    H = torch.empty((M, gl.r), dtype=torch.float32, device=dev)
    ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, H, gl.ws)
    out = {}
    for route in ("plain", "db"):
        dX = torch.empty((M, gl.K), dtype=torch.bfloat16, device=dev)
        G = torch.empty((M, gl.r), dtype=torch.float32, device=dev)
        dA = torch.empty((gl.r, gl.K), dtype=torch.float32, device=dev)
        dB = torch.full((gl.N, gl.r), 3.0, dtype=torch.float32, device=dev) if dB0 is None else dB0.clone()
        if route == "plain":
            ql.qlora_bwd_input(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, dX, G, gl.ws)
            ql.qlora_bwd_lora(gl.desc, M, gl.X, gl.dY, gl.A, gl.B, H, G, dA, dB, accumulate, gl.ws)
        else:
            ql.qlora_bwd_input_db(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, H, dX, G, dB, accumulate, gl.ws)
            ql.qlora_bwd_lora(gl.desc, M, gl.X, None, gl.A, gl.B, None, G, dA, None, 0, gl.ws)
        torch.cuda.synchronize()
        out[route] = dict(dX=dX, G=G, dA=dA, dB=dB)
    assert ql.qlora_device_status() == 0
    return out


@pytest.mark.parametrize("K,N,M,bits,g,r", [
    (1024, 1024, 1536, 4, 128, 8),      # CTA-pair kernel, 12 tiles on 74 pairs: producer clusters take dB on
    (1024, 6656, 1536, 2, 64, 8),       # 78 tiles in the forward, 12 in the backward
    (6656, 1024, 1400, 3, 128, 8),      # backward with a split last wave (producers half a tile ahead only: falls back), ragged rows
    (1024, 1024, 1400, 3, 128, 8),      # producers with ragged token rows
    (1024, 1024, 1536, 4, 128, 16),     # two rank tiles: three row blocks per producer CTA
    (1024, 1024, 4096, 4, 128, 16),     # ... which 32 tiles leave too few idle pairs for: falls back to the gradient kernels
    (2048, 1024, 2000, 8, 128, 24),     # three rank tiles: falls back
    (512, 768, 64, 4, 128, 8),          # single-CTA tensor-core kernel: falls back
    (512, 768, 9, 8, 128, 8),           # few-token kernels: falls back
    (96, 40, 300, 4, 32, 8),            # CUDA-core kernel: falls back
])
def test_db_from_the_backward_call_matches_the_oracle(K, N, M, bits, g, r):
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * r, M=M, seed=K + N + M)
    gl = GpuLayer(layer)
    ref = orc.layer_reference(layer)
    out = run_db(gl)
    for route in ("plain", "db"):
        assert rel_err(to_f64(out[route]["dB"]), ref["dB"]) <= REL_TOL, route
        assert rel_err(to_f64(out[route]["dA"]), ref["dA"]) <= REL_TOL, route
    # the frozen-weight path and G do not depend on who computes dB (dA alone is cut into finer row slices than dA with
    # dB, so its bits may differ in the last places between the routes)
    assert torch.equal(out["plain"]["dX"].view(torch.int16), out["db"]["dX"].view(torch.int16))
    assert torch.equal(out["plain"]["G"], out["db"]["G"])
    # same bits on a second run of either route
    again = run_db(gl)
    for route in ("plain", "db"):
        assert torch.equal(out[route]["dB"], again[route]["dB"]) and torch.equal(out[route]["dA"], again[route]["dA"]), route


def test_db_accumulates_into_existing_gradients():
    layer = qi.random_codes_layer(K=1024, N=1024, bits=4, group_size=128, r=8, alpha=16.0, M=1536, seed=77)
    gl = GpuLayer(layer)
    ref = orc.layer_reference(layer)
    base = torch.from_numpy(np.random.default_rng(5).standard_normal((gl.N, gl.r)).astype(np.float32)).cuda()
    out = run_db(gl, accumulate=1, dB0=base)
    want = ref["dB"] + base.cpu().numpy().astype(np.float64)
    for route in ("plain", "db"):
        assert rel_err(to_f64(out[route]["dB"]), want) <= REL_TOL, route


def test_config2_shape_db_and_step_outputs():
    """The headline shape (4096 x 4096, INT4 g128, r = 8, 2048 tokens): dB from the ten idle SM pairs of the backward
    kernel against the oracle."""
    layer = qi.config2()
    gl = GpuLayer(layer)
    ref = orc.layer_reference(layer, rows=[0, 1, 2047])
    out = run_db(gl)
    assert rel_err(to_f64(out["db"]["dB"]), ref["dB"]) <= REL_TOL
    assert rel_err(to_f64(out["db"]["dA"]), ref["dA"]) <= REL_TOL
    assert torch.equal(out["plain"]["dX"].view(torch.int16), out["db"]["dX"].view(torch.int16))


@pytest.mark.parametrize("r", [8, 16])
def test_producer_route_is_the_one_that_runs(r):
    """With the whole workspace the producer clusters form dB; with a workspace one byte short of the optional area for
    their parts the same call hands dB to the gradient kernels.  Both are right, and they group the sum over tokens
    differently, so their bits differ: equal bits would mean the producer route never ran."""
    layer = qi.random_codes_layer(K=1024, N=1024, bits=4, group_size=128, r=r, alpha=2.0 * r, M=1536, seed=90 + r)
    gl = GpuLayer(layer)
    ref = orc.layer_reference(layer)
    M, dev = gl.M, gl.X.device
    Y = torch.empty((M, gl.N), dtype=torch.bfloat16, device=dev)
    H = torch.empty((M, gl.r), dtype=torch.float32, device=dev)
    ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, H, gl.ws)
    need = ql.qlora_workspace_bytes(gl.desc, M)
    got = {}
    for name, nbytes in (("producers", need), ("gradient kernels", need - 1)):
        dX = torch.empty((M, gl.K), dtype=torch.bfloat16, device=dev)
        G = torch.empty((M, gl.r), dtype=torch.float32, device=dev)
        dB = torch.empty((gl.N, gl.r), dtype=torch.float32, device=dev)
        ql.qlora_bwd_input_db(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, H, dX, G, dB, 0, gl.ws, workspace_bytes=nbytes)
        torch.cuda.synchronize()
        assert rel_err(to_f64(dB), ref["dB"]) <= REL_TOL, name
        got[name] = dB
    assert ql.qlora_device_status() == 0
    assert not torch.equal(got["producers"], got["gradient kernels"])


@pytest.mark.parametrize("K,N,M,bits,g,r", [(1024, 1024, 1536, 4, 128, 8),      # dB on the producers
                                            (1024, 6656, 1536, 4, 128, 8),      # ... with a split last wave in the forward
                                            (6656, 1024, 1536, 2, 64, 16)])     # split last wave in the backward, dB by the gradient kernels
def test_replayed_graph_gives_the_eager_bits(K, N, M, bits, g, r):
    """A whole step (forward, backward with dB, gradient call for dA) captured in a CUDA graph and replayed three times:
    the counters in the workspace are zeroed by a captured launch, so every replay must reproduce the eager results bit
    for bit, split tiles and producer clusters included."""
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * r, M=M, seed=K + N + r)
    gl = GpuLayer(layer)
    dev = gl.X.device

    def buffers():
        return dict(Y=torch.empty((M, N), dtype=torch.bfloat16, device=dev), H=torch.empty((M, r), dtype=torch.float32, device=dev),
                    dX=torch.empty((M, K), dtype=torch.bfloat16, device=dev), G=torch.empty((M, r), dtype=torch.float32, device=dev),
                    dA=torch.empty((r, K), dtype=torch.float32, device=dev), dB=torch.empty((N, r), dtype=torch.float32, device=dev))

    def step(b):
        ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, b["Y"], b["H"], gl.ws)
        ql.qlora_bwd_input_db(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, b["H"], b["dX"], b["G"], b["dB"], 0, gl.ws)
        ql.qlora_bwd_lora(gl.desc, M, gl.X, None, gl.A, gl.B, None, b["G"], b["dA"], None, 0, gl.ws)

    eager = buffers()
    step(eager)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    captured = buffers()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step(captured)
    for _ in range(3):
        for t in captured.values():
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for key in eager:
            a, b = eager[key], captured[key]
            assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a, b.view(torch.int16) if b.dtype == torch.bfloat16 else b), key
    assert ql.qlora_device_status() == 0
    ref = orc.layer_reference(layer, rows=[0, 1, M - 1])
    assert rel_err(to_f64(captured["dB"]), ref["dB"]) <= REL_TOL and rel_err(to_f64(captured["dA"]), ref["dA"]) <= REL_TOL
