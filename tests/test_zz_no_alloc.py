"""qlora_bwd_lora_static: the LoRA-gradient call for hosts that may not allocate device memory when they call the
library (everything is owned by their own memory pool, or allocation calls are banned inside their step loop because
they synchronise the device).  It takes no workspace; its scratch is a fixed array inside the library.

The check: through the C ABI, its dA / dB equal those of qlora_bwd_lora (same kernels, so bit for bit, and in any case
within the parity tolerance of the other GPU tests) on two calls in a row -- the second call finds the first one's
leftovers in the shared array -- for saved and for recomputed H / G, with and without accumulation.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from gpu_util import GpuLayer, to_f64
from helpers import REL_TOL, rel_err


def test_static_limit_is_refused_on_the_host():
    """A shape whose scratch need exceeds the built-in array is rejected before anything is launched (no GPU needed)."""
    from paper_2306_08162_b200 import build as qbuild
    qbuild.build_library()
    d = ql.desc(4, 128, 11008, 11008, 64, 128.0)
    assert ql.qlora_workspace_bytes(d, 4096) > ql.STATIC_SCRATCH_BYTES
    ok = 0x1000   # aligned, non-NULL, never dereferenced: the size check comes first
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_bwd_lora_static(d, 4096, ok, ok, ok, ok, None, None, ok, ok, 0, stream=0)
    assert e.value.status == -7
    assert "built-in" in ql.qlora_status_string(-7)


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [dict(K=512, N=512, bits=4, group_size=128, r=8, alpha=16.0, M=64),
                                   dict(K=1024, N=2048, bits=2, group_size=64, r=16, alpha=32.0, M=300)])
def test_static_scratch_matches_workspace_call_twice_in_a_row(shape):
    layer = qi.random_codes_layer(seed=21, **shape)
    gl = GpuLayer(layer)
    assert ql.qlora_workspace_bytes(gl.desc, gl.M) <= ql.STATIC_SCRATCH_BYTES
    want = gl.run()                                   # qlora_fwd / qlora_bwd_input / qlora_bwd_lora with a workspace
    H, G = want["H"], want["G"]
    for call in range(2):                             # the second call reuses the array the first one left dirty
        for saved in (True, False):
            dA = torch.full_like(want["dA"], float("nan"))
            dB = torch.full_like(want["dB"], float("nan"))
            ql.qlora_bwd_lora_static(gl.desc, gl.M, gl.X, gl.dY, gl.A, gl.B, H if saved else None, G if saved else None,
                                     dA, dB, 0)
            torch.cuda.synchronize()
            assert rel_err(to_f64(dA), to_f64(want["dA"])) <= REL_TOL, (call, saved)
            assert rel_err(to_f64(dB), to_f64(want["dB"])) <= REL_TOL, (call, saved)
            assert torch.equal(dA, want["dA"]) and torch.equal(dB, want["dB"]), (call, saved)
    # accumulate = 1 adds to what is there
    dA = torch.full_like(want["dA"], 1.5)
    dB = torch.full_like(want["dB"], -0.5)
    ql.qlora_bwd_lora_static(gl.desc, gl.M, gl.X, gl.dY, gl.A, gl.B, H, G, dA, dB, 1)
    torch.cuda.synchronize()
    assert torch.equal(dA, 1.5 + want["dA"]) and torch.equal(dB, -0.5 + want["dB"])
    assert ql.qlora_device_status() == 0
