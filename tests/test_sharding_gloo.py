"""Batch sharding over ranks (world size 2, gloo, CPU): shards cover the batch, per-entry
results do not depend on the split, and the all-reduced relation gradient equals the
full-batch one.  The oracle stands in for the kernels here (no GPU in this test)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import bpt_oracle as orc
from paper_1911_04070_b200 import shard, synth


def test_batch_shard_covers_the_batch():
    for B in (0, 1, 2, 5, 8, 33):
        for world in (1, 2, 3, 8):
            spans = [shard.batch_shard(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c and 0 <= b - a <= (B + world - 1) // world
    with pytest.raises(ValueError):
        shard.batch_shard(4, 2, 2)


def _worker(rank, world, port, B, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n, k, H, d = 16, 2, 2, 8
    g = orc.enumerate_graph(n, k, 0)
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=3, std_qkv=1.0, std_rel=0.3, bf16=False)
    a, b = shard.batch_shard(B, rank, world)
    sl = slice(a, b)
    dq, dk, dv, dr = orc.attn_bwd(g, x["q"][sl], x["k"][sl], x["v"][sl], x["rel_emb"], 0.3, x["d_out"][sl])
    dr_t = torch.from_numpy(dr.copy())
    shard.allreduce_d_rel(dr_t)
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), dq=dq, dr=dr_t.numpy(), a=a, b=b)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_full_batch(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    B, world = 3, 2
    mp.spawn(_worker, args=(world, port, B, str(tmp_path)), nprocs=world, join=True)
    n, k, H, d = 16, 2, 2, 8
    g = orc.enumerate_graph(n, k, 0)
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=3, std_qkv=1.0, std_rel=0.3, bf16=False)
    dq, dk, dv, dr = orc.attn_bwd(g, x["q"], x["k"], x["v"], x["rel_emb"], 0.3, x["d_out"])
    for rank in range(world):
        r = np.load(os.path.join(str(tmp_path), "rank%d.npz" % rank))
        np.testing.assert_allclose(r["dr"], dr, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(r["dq"], dq[int(r["a"]):int(r["b"])], rtol=1e-12, atol=1e-14)
