"""Calls given different workspaces may overlap on the GPU (the header's rule): two layers stepped on two streams at the
same time, each with its own workspace (hence its own counters, exchange area and parts of dB), must give the bits they
give when stepped one after the other."""
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from gpu_util import GpuLayer

pytestmark = pytest.mark.gpu


def make(K, N, M, bits, g, r, seed):
    gl = GpuLayer(qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * r, M=M, seed=seed))
    dev = gl.X.device
    gl.out = dict(Y=torch.empty((M, N), dtype=torch.bfloat16, device=dev), H=torch.empty((M, r), dtype=torch.float32, device=dev),
                  dX=torch.empty((M, K), dtype=torch.bfloat16, device=dev), G=torch.empty((M, r), dtype=torch.float32, device=dev),
                  dA=torch.empty((r, K), dtype=torch.float32, device=dev), dB=torch.empty((N, r), dtype=torch.float32, device=dev))
    return gl


def step(gl, stream=None):
    o, M = gl.out, gl.M
    ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, o["Y"], o["H"], gl.ws, stream=stream)
    ql.qlora_bwd_input_db(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, o["H"], o["dX"], o["G"], o["dB"], 0, gl.ws, stream=stream)
    ql.qlora_bwd_lora(gl.desc, M, gl.X, None, gl.A, gl.B, None, o["G"], o["dA"], None, 0, gl.ws, stream=stream)


def snapshot(gl):
    return {k: v.clone() for k, v in gl.out.items()}


def test_two_streams_two_workspaces():
    a = make(1024, 1024, 1536, 4, 128, 8, seed=201)       # producer clusters with dB, 12 tiles
    b = make(1024, 6656, 1536, 2, 64, 8, seed=202)        # 78 tiles forward: split last wave
    step(a); step(b)
    torch.cuda.synchronize()
    want_a, want_b = snapshot(a), snapshot(b)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    sa.wait_stream(torch.cuda.current_stream()); sb.wait_stream(torch.cuda.current_stream())
    for _ in range(6):
        for t in list(a.out.values()) + list(b.out.values()):
            t.zero_()
        torch.cuda.synchronize()
        step(a, stream=sa.cuda_stream)
        step(b, stream=sb.cuda_stream)
        step(a, stream=sa.cuda_stream)
        torch.cuda.synchronize()
        assert ql.qlora_device_status() == 0
        for gl, want in ((a, want_a), (b, want_b)):
            for key, ref in want.items():
                got = gl.out[key]
                same = torch.equal(got.view(torch.int16), ref.view(torch.int16)) if got.dtype == torch.bfloat16 else torch.equal(got, ref)
                assert same, key
