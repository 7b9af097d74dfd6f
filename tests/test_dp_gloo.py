"""Token-sharded data parallelism, two `gloo` ranks on the CPU: each rank's LoRA gradients over its half of the tokens
(computed here with the oracle: this is a test of the exchange step, not of the kernels), summed by
allreduce_lora_grads, equal the full-batch gradients; Y and dX need no exchange."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import qlora_inputs as qi
    from oracle import qlora_oracle as orc
    from paper_2306_08162_b200.dp import allreduce_lora_grads
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layers = [qi.make_layer(K=64, N=32, bits=4, group_size=32, r=8, alpha=16.0, M=24, seed=s) for s in (1, 2, 3)]
    grads, want = [], []
    for L in layers:
        ref = orc.layer_reference(L)
        rows = np.arange(rank, L["M"], world)                  # this rank's token shard
        shard = dict(L, X=L["X"][rows], dY=L["dY"][rows], M=len(rows))
        mine = orc.layer_reference(shard)
        # rank-local outputs are already the full-batch rows
        assert np.allclose(mine["Y"], ref["Y"][rows], rtol=1e-12, atol=1e-12)
        assert np.allclose(mine["dX"], ref["dX"][rows], rtol=1e-12, atol=1e-12)
        grads += [torch.from_numpy(mine["dA"].astype(np.float32)), torch.from_numpy(mine["dB"].astype(np.float32))]
        want += [ref["dA"], ref["dB"]]
    allreduce_lora_grads(grads, bucket_bytes=3000)             # small buckets: several collectives, uneven packing
    ok = all(np.allclose(g.numpy(), w, rtol=1e-5, atol=1e-6) for g, w in zip(grads, want))
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write("1" if ok else "0")
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_gradients_sum_to_the_full_batch(tmp_path):
    world, port = 2, 29547
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        assert (tmp_path / f"ok{rank}").read_text() == "1"


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_2306_08162_b200.dp import allreduce_lora_grads
    g = torch.ones(4, 4)
    allreduce_lora_grads([g])
    assert torch.equal(g, torch.ones(4, 4))
