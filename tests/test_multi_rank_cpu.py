"""World-size-2 check of the multi-GPU form on CPU (gloo): the batch is split by request,
each rank works on its slice alone, and the gathered result equals the whole-batch result.
The per-rank work is done by the CPU oracle here; the point is the sharding and that the
data path needs no collective."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_10803_b200 import synth
from paper_2411_10803_b200.sharding import shard_range

W = synth.WORKLOADS["c1_tiny"].with_(batch=5, n_vis=40, n_txt=6, n_heads=2, hidden=256, n_salient=2,
                                     key_cnt=3, budget=8)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_path):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = shard_range(W.batch, rank, world)
    d = synth.make_batch(W, requests=range(lo, hi))
    G, I = oracle.score(d["q_text"], d["k"], W.vis_start, W.n_vis, W.txt_start)
    kept, cnt, _, _ = oracle.select(G, I, W.seq_len, d["key_idx"], d["key_cnt"], budget=W.budget)
    # gather only to compare; the filter itself exchanged nothing
    mine = torch.full((3, W.budget), -1, dtype=torch.int32)        # ceil(5/2) rows per rank
    mine[: hi - lo] = torch.from_numpy(kept)
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    sizes = torch.tensor([hi - lo], dtype=torch.int64)
    all_sizes = [torch.empty_like(sizes) for _ in range(world)]
    dist.all_gather(all_sizes, sizes)
    if rank == 0:
        rows = [g[: int(s)] for g, s in zip(gathered, all_sizes)]
        np.save(out_path, torch.cat(rows).numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_whole_batch(tmp_path):
    import oracle
    out = str(tmp_path / "kept.npy")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    d = synth.make_batch(W)
    G, I = oracle.score(d["q_text"], d["k"], W.vis_start, W.n_vis, W.txt_start)
    kept, _, _, _ = oracle.select(G, I, W.seq_len, d["key_idx"], d["key_cnt"], budget=W.budget)
    assert np.array_equal(np.load(out), kept)
