"""Helpers for the GPU parity tests: upload a synthetic layer, run the three C-ABI calls, fetch results."""
import numpy as np
import torch

import paper_2306_08162_b200 as ql

CANARY = 0x7B


def bf16_from_bits(bits16: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits16).view(np.int16)).to(device).view(torch.bfloat16)


def f16_to_dev(x: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).to(device)


def guarded(shape, dtype, device="cuda", pad_bytes=256):
    """A tensor with canary bytes on both sides, to catch out-of-bounds writes.  Returns (view, raw buffer)."""
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    n_al = (n + 255) // 256 * 256
    raw = torch.full((pad_bytes + n_al + pad_bytes,), CANARY, dtype=torch.uint8, device=device)
    view = raw[pad_bytes:pad_bytes + n].view(dtype).view(*shape)
    return view, raw


def canaries_intact(raw, shape, dtype, pad_bytes=256) -> bool:
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    head = raw[:pad_bytes]
    tail = raw[pad_bytes + n:]
    return bool((head == CANARY).all().item() and (tail == CANARY).all().item())


class GpuLayer:
    """Device copies of one projection's inputs; packing is done by the library's own qlora_pack."""

    def __init__(self, layer: dict, device="cuda"):
        self.layer = layer
        self.K, self.N, self.r, self.M = layer["K"], layer["N"], layer["r"], layer["M"]
        self.bits, self.g = layer["bits"], layer["group_size"]
        self.desc = ql.desc(self.bits, self.g, self.K, self.N, self.r, layer["alpha"])
        codes = torch.from_numpy(layer["codes"]).to(device)
        self.Q = torch.empty((self.K * self.bits // 32, self.N), dtype=torch.int32, device=device)
        ql.qlora_pack(self.bits, self.K, self.N, codes, self.Q)
        self.scales = f16_to_dev(layer["scales"], device)
        self.zeros = f16_to_dev(layer["zeros"], device)
        self.A = bf16_from_bits(layer["A"], device) if self.r else None
        self.B = bf16_from_bits(layer["B"], device) if self.r else None
        self.X = bf16_from_bits(layer["X"], device) if "X" in layer else None
        self.dY = bf16_from_bits(layer["dY"], device) if "dY" in layer else None
        self.ws = torch.empty(max(ql.qlora_workspace_bytes(self.desc, self.M), 256), dtype=torch.uint8, device=device)

    def run(self, X=None, dY=None, save_hg=True, accumulate=0, dA=None, dB=None, check_canaries=True):
        X = self.X if X is None else X
        dY = self.dY if dY is None else dY
        M = X.shape[0]
        dev = X.device
        Y, Yraw = guarded((M, self.N), torch.bfloat16, dev)
        dX, dXraw = guarded((M, self.K), torch.bfloat16, dev)
        H = torch.empty((M, self.r), dtype=torch.float32, device=dev) if (save_hg and self.r) else None
        G = torch.empty((M, self.r), dtype=torch.float32, device=dev) if (save_hg and self.r) else None
        if dA is None:
            dA = torch.full((self.r, self.K), float("nan"), dtype=torch.float32, device=dev)
        if dB is None:
            dB = torch.full((self.N, self.r), float("nan"), dtype=torch.float32, device=dev)
        ql.qlora_fwd(self.desc, M, X, self.Q, self.scales, self.zeros, self.A, self.B, Y, H, self.ws)
        ql.qlora_bwd_input(self.desc, M, dY, self.Q, self.scales, self.zeros, self.A, self.B, dX, G, self.ws)
        ql.qlora_bwd_lora(self.desc, M, X, dY, self.A, self.B, H, G, dA, dB, accumulate, self.ws)
        torch.cuda.synchronize()
        assert ql.qlora_device_status() == 0
        if check_canaries:
            assert canaries_intact(Yraw, (M, self.N), torch.bfloat16), "write outside Y"
            assert canaries_intact(dXraw, (M, self.K), torch.bfloat16), "write outside dX"
        return dict(Y=Y, dX=dX, dA=dA, dB=dB, H=H, G=G)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()
