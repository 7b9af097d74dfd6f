"""Parity of the fused LREC loss kernel with the oracle (needs a B200).  Logits are bf16 on both sides; the loss is compared
per token, the gradient with the layer tests' error measure (|got - ref| / max(|ref|, rms(ref)) <= 2e-2: the gradient is
stored in bf16)."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import bf16_from_bits, to_f64
from helpers import REL_TOL, rel_err

pytestmark = pytest.mark.gpu


def run_case(T, V, lkl, lce, seed, with_grad=True, scale=1.0, spread=3.0):
    z_bits = qi.normal_bf16(seed, 0, (T, V), spread)
    t_bits = qi.normal_bf16(seed, 1, (T, V), spread)
    labels = np.random.default_rng(seed).integers(-1, V, size=T).astype(np.int32)
    z, t = bf16_from_bits(z_bits), bf16_from_bits(t_bits)
    loss = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    grad = torch.full((T, V), float("nan"), dtype=torch.bfloat16, device="cuda") if with_grad else None
    ql.qlora_lrec_loss(z, t, torch.from_numpy(labels).cuda(), lkl, lce, scale, loss, grad)
    torch.cuda.synchronize()
    want_loss, want_grad = orc.lrec_loss(orc.bf16_bits_to_f64(z_bits), orc.bf16_bits_to_f64(t_bits), labels, lkl, lce)
    assert np.allclose(loss.cpu().numpy(), want_loss, rtol=2e-4, atol=2e-5)
    if with_grad:
        assert rel_err(to_f64(grad), scale * want_grad) <= REL_TOL
    return loss


@pytest.mark.parametrize("T,V", [(7, 32000), (64, 32768), (33, 4096), (5, 8), (300, 1000), (2, 12296)])
def test_loss_and_gradient_match_the_oracle(T, V):
    run_case(T, V, 0.8, 1.2, seed=T + V, scale=1.0 / T)


def test_loss_only_and_pure_terms_and_determinism():
    a = run_case(16, 32000, 1.0, 0.0, seed=1, with_grad=False)
    run_case(16, 32000, 0.0, 1.0, seed=2)
    b = run_case(16, 32000, 1.0, 0.0, seed=1, with_grad=False)
    assert torch.equal(a, b)
    run_case(8, 2048, 0.5, 0.5, seed=3, spread=12.0)        # peaked distributions: large logit range


def test_rejected_shapes():
    z = torch.zeros((2, 12), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_lrec_loss(z, z, None, 1.0, 1.0, 1.0, out, None)          # V % 8 != 0
    assert e.value.status == -2
