"""Multi-process path on CPU (gloo, world size 2): the batch split used for N > 1 GPUs.

Samples are independent under the per-sample stopping test (Algorithm 1 applied per sequence), so a
multi-GPU run is a plain batch split with replicated weights and no exchange on the data path.  Two
gloo ranks each decode their shard with the CPU oracle; the gathered result must equal the
single-process result bit for bit, the shards must tile the batch, and the max-over-ranks reduction
bench.py uses for its timing must behave.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case():
    cfg = synth.micro_config(H=2, W=4, n_blocks=2, width=16, n_heads=2, B=5)
    blocks = synth.make_weights(cfg, seed=3, head_scale=0.4)
    z = synth.make_latents(cfg, 77)
    return cfg, blocks, z


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg, blocks, z = _case()
        lo, hi = synth.shard_batch(cfg["B"], rank, world)
        x, it = O.model_inverse(blocks, z[lo:hi], None, cfg, [0, 1], 1e-6, synth.seq_len(cfg) + 1)
        # gather ragged shards: pad to the largest shard
        pad = (cfg["B"] + world - 1) // world
        buf = torch.zeros((pad,) + x.shape[1:], dtype=torch.float64)
        buf[: hi - lo] = torch.from_numpy(x)
        got = [torch.zeros_like(buf) for _ in range(world)]
        dist.all_gather(got, buf)
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        if rank == 0:
            parts = []
            for r in range(world):
                a, b = synth.shard_batch(cfg["B"], r, world)
                parts.append(got[r][: b - a].numpy())
            np.save(os.path.join(out_dir, "x.npy"), np.concatenate(parts, axis=0))
            np.save(os.path.join(out_dir, "tmax.npy"), t.numpy())
    finally:
        dist.destroy_process_group()


def test_shards_tile_the_batch():
    for B in (1, 5, 64, 257):
        for world in (1, 2, 3, 8):
            spans = [synth.shard_batch(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def test_two_gloo_ranks_reproduce_the_single_process_result(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    cfg, blocks, z = _case()
    want, _ = O.model_inverse(blocks, z, None, cfg, [0, 1], 1e-6, synth.seq_len(cfg) + 1)
    got = np.load(os.path.join(str(tmp_path), "x.npy"))
    assert got.shape == want.shape and np.array_equal(got, want)
    assert np.load(os.path.join(str(tmp_path), "tmax.npy"))[0] == float(world)
