"""Chained decoder-block projection sets (the shape of configs[4]: q, k, v, o 4096x4096; gate, up 4096->11008; down
11008->4096; INT2 group 64, r = 8, M = 4096 tokens), forward through the chain and then backward, on a B200.

Chaining: q, k, v read the block input; o reads q's output; gate and up read o's output; down reads gate's output; down's
output is the next block's input (no attention, no non-linearity).  Backward mirrors it along down -> gate -> o -> q; k, v
and up get seeded upstream gradients.  Every projection is checked on its own against the oracle fed that projection's
ACTUAL device inputs (copied back), so errors do not compound; Y / dX on sampled token rows, dA / dB in full.
Two blocks are run (the full 32 only repeat the same seven shapes)."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import bf16_from_bits, f16_to_dev, to_f64
from helpers import REL_TOL, rel_err

pytestmark = pytest.mark.gpu
BLOCKS = 2


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


class Proj:
    def __init__(self, layer):
        self.layer = layer
        K, N, bits = layer["K"], layer["N"], layer["bits"]
        self.K, self.N, self.r = K, N, layer["r"]
        self.desc = ql.desc(bits, layer["group_size"], K, N, self.r, layer["alpha"])
        self.Q = torch.empty((K * bits // 32, N), dtype=torch.int32, device="cuda")
        ql.qlora_pack(bits, K, N, torch.from_numpy(layer["codes"]).cuda(), self.Q)
        self.scales, self.zeros = f16_to_dev(layer["scales"]), f16_to_dev(layer["zeros"])
        self.A, self.B = bf16_from_bits(layer["A"]), bf16_from_bits(layer["B"])


def test_two_chained_blocks_match_the_oracle_projection_by_projection():
    M = qi.CONFIG5_M
    rows = sorted(set(np.random.default_rng(5).choice(M, size=28, replace=False).tolist()) | {0, 1, M - 2, M - 1})
    names = [p[0] for p in qi.CONFIG5_PROJECTIONS]
    x_in = bf16_from_bits(qi.config5_tokens())
    ws = None
    saved = []          # per block: dict name -> (Proj, X, Y, H)
    for blk in range(BLOCKS):
        acts = {}
        for name in names:
            pr = Proj(qi.config5_projection(blk, name))
            need = ql.qlora_workspace_bytes(pr.desc, M)
            if ws is None or ws.numel() < need:
                ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            X = {"q": x_in, "k": x_in, "v": x_in, "o": acts.get("q", (None,) * 3)[2], "gate": acts.get("o", (None,) * 3)[2],
                 "up": acts.get("o", (None,) * 3)[2], "down": acts.get("gate", (None,) * 3)[2]}[name]
            Y = torch.empty((M, pr.N), dtype=torch.bfloat16, device="cuda")
            H = torch.empty((M, pr.r), dtype=torch.float32, device="cuda")
            ql.qlora_fwd(pr.desc, M, X, pr.Q, pr.scales, pr.zeros, pr.A, pr.B, Y, H, ws)
            acts[name] = (pr, X, Y, H)
        saved.append(acts)
        x_in = acts["down"][2]
    torch.cuda.synchronize()
    assert ql.qlora_device_status() == 0
    assert torch.isfinite(x_in.float()).all()

    grad_in = None      # gradient w.r.t. the block output, from the block after
    for blk in reversed(range(BLOCKS)):
        acts = saved[blk]
        grads = {}
        for name in ("down", "up", "gate", "o", "v", "k", "q"):
            pr, X, Y, H = acts[name]
            if name == "down":
                dY = grad_in if grad_in is not None else bf16_from_bits(qi.config5_seed_grad(blk, name, pr.N))
            elif name in ("up", "v", "k"):
                dY = bf16_from_bits(qi.config5_seed_grad(blk, name, pr.N))
            else:
                dY = grads[{"gate": "down", "o": "gate", "q": "o"}[name]]
            dX = torch.empty((M, pr.K), dtype=torch.bfloat16, device="cuda")
            G = torch.empty((M, pr.r), dtype=torch.float32, device="cuda")
            dA = torch.empty((pr.r, pr.K), dtype=torch.float32, device="cuda")
            dB = torch.empty((pr.N, pr.r), dtype=torch.float32, device="cuda")
            ql.qlora_bwd_input(pr.desc, M, dY, pr.Q, pr.scales, pr.zeros, pr.A, pr.B, dX, G, ws)
            ql.qlora_bwd_lora(pr.desc, M, X, dY, pr.A, pr.B, H, G, dA, dB, 0, ws)
            torch.cuda.synchronize()
            grads[name] = dX
            # oracle on this projection's actual inputs
            layer = dict(pr.layer, X=bits_of(X), dY=bits_of(dY))
            ref = orc.layer_reference(layer, rows=rows)
            errs = {"Y": rel_err(to_f64(Y)[rows], ref["Y"]), "dX": rel_err(to_f64(dX)[rows], ref["dX"]),
                    "dA": rel_err(to_f64(dA), ref["dA"]), "dB": rel_err(to_f64(dB), ref["dB"])}
            for key, e in errs.items():
                assert e <= REL_TOL, (blk, name, key, e, errs)
            del layer, ref
        grad_in = grads["q"]
    assert ql.qlora_device_status() == 0
