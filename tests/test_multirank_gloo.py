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


# ---- vocabulary-sharded step: the exchanges between the four local phases ------------------------------------------

def test_shard_bounds_cover_the_vocabulary_in_rank_order():
    from paper_2604_25925_b200 import sharded
    for V in (1, 16, 3001, 32000, 128256, 151936):
        for R in (1, 2, 3, 8):
            b = sharded.shard_bounds(V, R)
            assert len(b) == R and b[0][0] == 0 and b[-1][1] == V
            assert all(lo <= hi for lo, hi in b) and all(b[r][1] == b[r + 1][0] for r in range(R - 1))
            assert all(lo % 8 == 0 for lo, hi in b if lo < V)


class _RecordingPhases:
    """Stands in for the C ABI's four phases (which need a GPU): every output is tagged with the rank that made it,
    and every phase checks that what the exchange handed it is every rank's output in rank order."""
    _dtype_code = staticmethod(lambda t: 0)

    def __init__(self, rank, world):
        self.rank, self.world, self.calls = rank, world, []

    def sgbv_shard_workspace_bytes(self, B, K, gamma, Vs, code):
        return 256

    def sgbv_shard_stats(self, zq, zp, tok, v_begin, V, T):
        self.calls.append("stats")
        B, K, g1, _ = zq.shape
        return torch.full((B, K, g1, 8), float(self.rank), dtype=torch.float32)

    def sgbv_shard_sums(self, zq, zp, T, stats_all, ws):
        self.calls.append("sums")
        assert stats_all.shape[0] == self.world and stats_all.is_contiguous()
        for r in range(self.world):
            assert (stats_all[r] == float(r)).all()
        B, K, g1, _ = zq.shape
        return torch.full((B, K, g1 - 1, 3), 10.0 + self.rank, dtype=torch.float64)

    def sgbv_shard_decide(self, tok, u, Vs, T, stats_all, sums_all, ws):
        self.calls.append("decide")
        for r in range(self.world):
            assert (sums_all[r] == 10.0 + r).all()
        from paper_2604_25925_b200.binding import VerifyOutput
        B, K, g = tok.shape
        return VerifyOutput(torch.ones(B, dtype=torch.int32), torch.zeros(B, dtype=torch.int32),
                            torch.full((B, g + 1), -1, dtype=torch.int32))

    def sgbv_shard_draw(self, zq, zp, v_begin, T, rank, ws, tokens):
        self.calls.append("draw")
        assert rank == self.rank
        tokens[rank::self.world, 1] = v_begin + 5     # this rank "owns" every world-th batch row


def _shard_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2604_25925_b200 import sharded
        fake = _RecordingPhases(rank, world)
        sharded.binding = fake
        ex = sharded.TorchExchange()
        assert (ex.rank, ex.world_size) == (rank, world)
        B, K, g, V = 5, 2, 3, 64
        lo, hi = sharded.shard_bounds(V, world)[rank]
        zq, zp = torch.zeros(B, K, g + 1, hi - lo), torch.zeros(B, K, g, hi - lo)
        out = sharded.verify(zq, zp, torch.zeros(B, K, g, dtype=torch.int32), torch.zeros(B, K * g + 1), 1.0, lo, V, ex)
        assert fake.calls == ["stats", "sums", "decide", "draw"]
        np.save(os.path.join(out_dir, f"tokens{rank}.npy"), out.tokens.numpy())
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_exchange_the_shard_phases_in_rank_order(tmp_path):
    world = 2
    mp.spawn(_shard_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    t0, t1 = np.load(tmp_path / "tokens0.npy"), np.load(tmp_path / "tokens1.npy")
    assert np.array_equal(t0, t1)                       # the max-all-reduce leaves every rank with every owner's token
    assert list(t0[:, 1]) == [5, 37, 5, 37, 5] and (t0[:, [0, 2, 3]] == -1).all()
