"""Data-parallel host logic on CPU: two gloo ranks split a batch by user, each computes its shard (the oracle
stands in for the GPU here), the results are gathered in rank order and must equal the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import laser_oracle
from paper_2602_11562_b200.sharding import shard_batch_arrays, user_shard
from workloads import make_custom


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _make():
    w = make_custom(U=5, C=3, L=40, d=16, H=2, S=8, M=2, dtype="f32", seed=77, d_qh=4, lengths=[40, 0, 17, 33, 8])
    w.cand_offsets = np.array([0, 4, 4, 9, 12, 15], dtype=np.int32)     # uneven candidate counts
    return w


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = _make()
    s = w.spec
    items, lengths, cands, offs, (c0, c1) = shard_batch_arrays(w.items, w.lengths, w.cands, w.cand_offsets, rank, world)
    _, z = laser_oracle.forward(items, lengths, cands, offs, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, w.gamma, w.tau)
    # gather variable-sized shards: pad to the largest shard
    n_loc = torch.tensor([z.shape[0]])
    sizes = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(sizes, n_loc)
    mx = int(max(int(x) for x in sizes))
    buf = torch.zeros(mx, s.d, dtype=torch.float64)
    buf[:z.shape[0]] = torch.from_numpy(z)
    parts = [torch.zeros_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    full = torch.cat([p[:int(n)] for p, n in zip(parts, sizes)]).numpy()
    if rank == 0:
        np.save(os.path.join(out_dir, "z.npy"), full)
    dist.barrier()
    dist.destroy_process_group()


def test_user_shard_partitions_exactly():
    for n, world in [(0, 2), (5, 2), (7, 3), (4096, 8), (3, 4)]:
        seen = []
        for r in range(world):
            seen.extend(user_shard(n, r, world))
        assert seen == list(range(n))
        sizes = [len(user_shard(n, r, world)) for r in range(world)]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        user_shard(4, 2, 2)


def test_two_rank_gloo_split_matches_unsharded(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    w = _make()
    s = w.spec
    _, z_ref = laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                    w.gamma, w.tau)
    z = np.load(tmp_path / "z.npy")
    np.testing.assert_allclose(z, z_ref, atol=1e-14)
