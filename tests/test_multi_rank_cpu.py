"""World-size-2 test of the data-parallel host logic on CPU (gloo): blocks are split across
ranks, every rank computes its shard (here with the float64 oracle standing in for the GPU
kernels), grad_codebook is all-reduced, and the result equals the single-process one."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2605_10655_b200 import shard, synth


def test_block_range_partitions_exactly():
    for nb in (0, 1, 5, 64, 237568):
        for world in (1, 2, 3, 8):
            spans = [shard.block_range(nb, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == nb
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.block_range(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = synth.tiny()
        W, c, g = wl.weights(), wl.codebook(), wl.upstream()
        a, b = shard.block_range(W.shape[0], rank, world)
        part = oracle.backward(W[a:b], c, g[a:b], wl.Lb, wl.k, wl.T)
        gc = torch.from_numpy(part["grad_codebook"].copy())
        shard.allreduce_grad_codebook(gc)
        np.save(os.path.join(out_dir, f"gc_{rank}.npy"), gc.numpy())
        np.save(os.path.join(out_dir, f"gw_{rank}.npy"), part["grad_W"])
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo_match_single_process(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = synth.tiny()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    ref = oracle.backward(W, c, g, wl.Lb, wl.k, wl.T)
    gcs = [np.load(tmp_path / f"gc_{r}.npy") for r in range(world)]
    np.testing.assert_allclose(gcs[0], gcs[1], rtol=0, atol=0)          # every rank holds the sum
    np.testing.assert_allclose(gcs[0], ref["grad_codebook"], rtol=0, atol=1e-11)
    gw = np.concatenate([np.load(tmp_path / f"gw_{r}.npy") for r in range(world)])
    np.testing.assert_allclose(gw, ref["grad_W"], rtol=0, atol=1e-13)


def test_allreduce_is_a_noop_without_a_group():
    t = torch.arange(4.0)
    assert torch.equal(shard.allreduce_grad_codebook(t.clone()), t)
