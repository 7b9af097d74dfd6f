"""All 32 chained decoder-block projection sets of configs[4] (q, k, v, o 4096x4096; gate, up 4096->11008; down
11008->4096; INT2 group 64, r = 8, M = 4096 tokens): forward through the 224 projections, then backward, on a B200.

Chaining: q, k, v read the block input; o reads q's output; gate and up read o's output; down reads gate's output; down's
output is the next block's input (no attention, no non-linearity), so the activations grow about 4.4x per block and reach
~1e20 by the last one; the gradients grow the same way on the way back.  Backward mirrors the chain along
down -> gate -> o -> q; k, v and up get seeded upstream gradients.

The weights are drawn on the host (N(0, 0.02^2)) and quantized on the device by qlora_quantize_rtn.  Every projection is
checked on its own against the oracle fed that projection's ACTUAL device inputs (copied back), so errors do not compound.
To keep the host time bounded the oracle works on sub-layers, which is exact because the quantizer and the layer are
independent per (output feature, group): Y on sampled token rows x 64 sampled output features (all K), dX on sampled
rows x two sampled groups of input features (all N); the oracle quantizes those sub-blocks of W itself.  Rows, features
and groups rotate with the block.  dA / dB (sums over all 4096 tokens) are checked on the same sub-blocks for every
projection of blocks 0, 1, 15, 31 and for one rotating projection of every other block."""
import numpy as np
import pytest
import torch

import paper_2306_08162_b200 as ql
import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import bf16_from_bits, to_f64
from helpers import REL_TOL, rel_err

pytestmark = pytest.mark.gpu
BLOCKS = qi.CONFIG5_LAYERS
BITS, GROUP, RANK, ALPHA = 2, 64, 8, 16.0
NAMES = [p[0] for p in qi.CONFIG5_PROJECTIONS]


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f64_of(t: torch.Tensor) -> np.ndarray:
    return orc.bf16_bits_to_f64(bits_of(t))


class Proj:
    """One projection: host weight W [N, K] (kept as the oracle's input), device Q / scales / zeros from the library's
    quantizer, adapters from the seeded generator."""

    def __init__(self, blk, name):
        _, K, N = qi.CONFIG5_PROJECTIONS[NAMES.index(name)]
        seed = 5000 + 10 * blk + NAMES.index(name)
        self.K, self.N, self.r, self.seed = K, N, RANK, seed
        self.desc = ql.desc(BITS, GROUP, K, N, RANK, ALPHA)
        W = qi.gaussian_weight(seed, N, K, 0.02)
        self.Q = torch.empty((K * BITS // 32, N), dtype=torch.int32, device="cuda")
        self.scales = torch.empty((K // GROUP, N), dtype=torch.float16, device="cuda")
        self.zeros = torch.empty((K // GROUP, N), dtype=torch.float16, device="cuda")
        ql.qlora_quantize_rtn(self.desc, torch.from_numpy(W).cuda(), self.Q, self.scales, self.zeros)
        self.A_bits = qi.uniform_bf16(seed, qi._T_A, (RANK, K), 1.0 / np.sqrt(K))
        self.B_bits = qi.normal_bf16(seed, qi._T_B, (N, RANK), 0.01)
        self.A, self.B = bf16_from_bits(self.A_bits), bf16_from_bits(self.B_bits)
        # the oracle's sub-blocks of W: 64 output features (all K) and two groups of input features (all N)
        rng = np.random.default_rng(seed)
        self.cols = np.sort(rng.choice(N // 8, size=8, replace=False))[:, None] * 8 + np.arange(8)[None, :]
        self.cols = self.cols.reshape(-1)
        self.groups = np.sort(rng.choice(K // GROUP, size=2, replace=False))
        self.ks = (self.groups[:, None] * GROUP + np.arange(GROUP)[None, :]).reshape(-1)
        self.W_cols = np.ascontiguousarray(W[self.cols, :])
        self.W_ks = np.ascontiguousarray(W[:, self.ks])

    def oracle_weights(self):
        """float64 weights of the two sub-layers, from the oracle's own quantizer, packer and dequantizer."""
        c, s, z = orc.quantize_rtn(self.W_cols, BITS, GROUP)
        Wc = orc.dequant(orc.pack(c, BITS), s, z, BITS, GROUP)             # [64, K]
        c, s, z = orc.quantize_rtn(self.W_ks, BITS, GROUP)
        Wk = orc.dequant(orc.pack(c, BITS), s, z, BITS, GROUP)             # [N, 128]
        return Wc, Wk


def test_thirty_two_chained_blocks_match_the_oracle_projection_by_projection():
    M = qi.CONFIG5_M
    x_in = bf16_from_bits(qi.config5_tokens())
    ws = None
    saved = []          # per block: dict name -> (Proj, X, Y, H)
    for blk in range(BLOCKS):
        acts = {}
        for name in NAMES:
            pr = Proj(blk, name)
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
    assert float(x_in.float().abs().max()) > 1e15           # the chain really reaches the large magnitudes

    s = ALPHA / RANK
    grad_in = None      # gradient w.r.t. the block output, from the block after
    for blk in reversed(range(BLOCKS)):
        acts = saved[blk]
        grads = {}
        rows = np.sort(np.random.default_rng(100 + blk).choice(M, size=16, replace=False))
        rows[0], rows[-1] = (0, M - 1) if blk % 2 else (1, M - 2)
        rows_t = torch.from_numpy(rows).cuda()
        full_grads = blk in (0, 1, 15, 31)
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
            # ---- the oracle on this projection's actual inputs, sub-layer by sub-layer ----
            Wc, Wk = pr.oracle_weights()
            A, B = orc.bf16_bits_to_f64(pr.A_bits), orc.bf16_bits_to_f64(pr.B_bits)
            cols_t, ks_t = torch.from_numpy(pr.cols).cuda(), torch.from_numpy(pr.ks).cuda()
            Xr, dYr = f64_of(X[rows_t]), f64_of(dY[rows_t])
            Y_ref, H_ref = orc.forward(Xr, Wc, A, B[pr.cols], ALPHA)                      # [rows, 64 features]
            dX_ref, _, _, G_ref = orc.backward(Xr[:, pr.ks], dYr, Wk, A[:, pr.ks], B, ALPHA)   # [rows, 128 features]
            errs = {"Y": rel_err(to_f64(Y[rows_t][:, cols_t]), Y_ref), "dX": rel_err(to_f64(dX[rows_t][:, ks_t]), dX_ref),
                    "H": rel_err(to_f64(H[rows_t]), H_ref), "G": rel_err(to_f64(G[rows_t]), G_ref)}
            if full_grads or NAMES.index(name) == blk % 7:
                Xf, dYf = f64_of(X), f64_of(dY)                                            # all 4096 tokens
                dA_ref = s * ((dYf @ B).T @ Xf[:, pr.ks])                                  # [r, 128]
                dB_ref = s * (dYf[:, pr.cols].T @ (Xf @ A.T))                              # [64, r]
                errs["dA"] = rel_err(to_f64(dA[:, ks_t]), dA_ref)
                errs["dB"] = rel_err(to_f64(dB[cols_t]), dB_ref)
                del Xf, dYf
            for key, e in errs.items():
                assert e <= REL_TOL, (blk, name, key, e, errs)
        grad_in = grads["q"]
        saved[blk] = None
    assert ql.qlora_device_status() == 0
