"""The N > 1 path on CPU: two gloo ranks shard a batch by rows, each verifies its shard (with the
oracle standing in for the device path, which needs a GPU), and the gathered outputs equal the
unsharded result row for row -- batch rows are independent, so no data-path collective is needed.
Also checks the timing reduction (MAX over ranks) and the shard arithmetic."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2604_25925_b200 import sharding, workloads


def test_shard_rows_partition_every_batch_exactly_once():
    for B in (0, 1, 2, 7, 8, 64, 257):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                a, b = sharding.shard_rows(B, r, world)
                assert 0 <= a <= b <= B
                seen += list(range(a, b))
            assert seen == list(range(B))
            sizes = [sharding.shard_rows(B, r, world)[1] - sharding.shard_rows(B, r, world)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_rows(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = workloads.VerifyConfig("mr", B=7, K=3, gamma=3, V=600, temperature=0.9, alpha=0.8, seed=77)
        inp = workloads.make_inputs(cfg)          # every rank builds the same seeded global batch
        a, b = sharding.shard_rows(cfg.B, rank, world)
        res = oracle.verify(inp.target_logits[a:b].numpy(), inp.draft_logits[a:b].numpy(),
                            inp.draft_tokens[a:b].numpy(), inp.uniforms[a:b].numpy(), cfg.temperature)
        mine = torch.from_numpy(np.concatenate([res.tau[:, None], res.f[:, None], res.tokens], axis=1).astype(np.int64))
        # outputs stay with their shard in production; here they are gathered only to be checked
        pad = torch.full((cfg.B, mine.shape[1]), -9, dtype=torch.int64)
        pad[: b - a] = mine
        got = [torch.empty_like(pad) for _ in range(world)]
        dist.all_gather(got, pad)
        slow = sharding.max_over_ranks(1.0 + rank)           # rank r "took" 1 + r
        total = sharding.sum_over_ranks(float(b - a))
        if rank == 0:
            rows = []
            for r in range(world):
                ra, rb = sharding.shard_rows(cfg.B, r, world)
                rows.append(got[r][: rb - ra])
            np.save(os.path.join(out_dir, "gathered.npy"), torch.cat(rows).numpy())
            np.save(os.path.join(out_dir, "scalars.npy"), np.array([slow, total]))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_result(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = workloads.VerifyConfig("mr", B=7, K=3, gamma=3, V=600, temperature=0.9, alpha=0.8, seed=77)
    inp = workloads.make_inputs(cfg)
    ref = oracle.verify(inp.target_logits.numpy(), inp.draft_logits.numpy(), inp.draft_tokens.numpy(),
                        inp.uniforms.numpy(), cfg.temperature)
    want = np.concatenate([ref.tau[:, None], ref.f[:, None], ref.tokens], axis=1).astype(np.int64)
    got = np.load(tmp_path / "gathered.npy")
    assert np.array_equal(got, want)
    slow, total = np.load(tmp_path / "scalars.npy")
    assert slow == 2.0 and total == cfg.B
