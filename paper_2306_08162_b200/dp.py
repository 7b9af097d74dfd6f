"""Token-sharded data parallelism for the layer: the one exchange step it needs.

Every rank holds a replica of the frozen packed weights and of the LoRA pairs and runs the layer on its own slice of
the token rows.  Y and dX are then rank-local; dA and dB are sums over tokens, so the ranks' partial gradients have to
be added once per step (r * (K + N) fp32 per adapted projection: 256 KiB at r = 8, K = N = 4096).  This module does
that with torch.distributed (NCCL over NVLink on GPUs, gloo on CPU): gradients of many projections are packed into a
few flat fp32 buckets so that the collective's launch latency, not its bandwidth, is amortised.  No kernel of the
library is involved; the single-GPU hot path is unchanged.
"""
from __future__ import annotations

from typing import Iterable, List

import torch
import torch.distributed as dist


def allreduce_lora_grads(grads: Iterable[torch.Tensor], group=None, bucket_bytes: int = 32 << 20) -> None:
    """Sum the fp32 gradient tensors `grads` (dA / dB of any number of projections) over the process group, in place.

    Tensors are copied into flat buckets of at most `bucket_bytes`, each bucket is all-reduced (SUM) once, and the
    result is copied back.  The order of `grads` must be the same on every rank.  A single-process run is a no-op."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    pending: List[torch.Tensor] = []
    size = 0

    def flush():
        nonlocal pending, size
        if not pending:
            return
        flat = torch.cat([t.reshape(-1) for t in pending])
        dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
        off = 0
        for t in pending:
            n = t.numel()
            t.copy_(flat[off:off + n].view_as(t))
            off += n
        pending, size = [], 0

    for t in grads:
        if t.dtype != torch.float32:
            raise TypeError("LoRA gradients are fp32")
        nbytes = t.numel() * 4
        if pending and (size + nbytes > bucket_bytes or t.device != pending[0].device):
            flush()
        pending.append(t)
        size += nbytes
    flush()
